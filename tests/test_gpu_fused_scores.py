"""hilore_coeffs_exposure (coefficients computed inside the exposure reduction): bit for bit the results of
hilore_grpo_coeffs followed by hilore_unit_exposure, and within 1e-5 of the oracle's own chain."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def fused(ro, rms, sl, beta=0.0, row_shift=0, N=None):
    n_rows, T = sl.stop - sl.start, ro.T
    U, ld = rms.shape
    nws = api.hilore_workspace_bytes(U, n_rows * T)
    ws, omega, E, sw = G.Guarded(nws), G.Guarded(n_rows * T * 4), G.Guarded(U * 4), G.Guarded(4)
    api.hilore_coeffs_exposure(G.dev(ro.rewards), ro.n_resp, ro.G, sl.start, n_rows, T, G.dev(ro.logp_new[sl]), G.dev(ro.logp_old[sl]),
                               G.dev(ro.logp_ref[sl]) if beta else None, G.dev(ro.mask[sl]), ro.n_valid if N is None else N, None,
                               0.2, beta, 1e-6, G.dev(rms), U, ld, row_shift, 1e-8, omega.ptr(), E.ptr(), sw.ptr(), ws.ptr(), nws)
    ws.numpy(np.uint8, (nws,))
    return omega.numpy(np.float32, (n_rows, T)), E.numpy(np.float32, (U,)), float(sw.numpy(np.float32, (1,))[0])


@pytest.mark.parametrize("P,G_,T,U,lengths,beta,row_shift", [
    (4, 8, 256, 2, "full", 0.0, 0),            # the tiny configuration
    (1, 8, 1024, 84, "full", 0.0, 0),          # one microbatch of the 1.5B-shaped configuration
    (2, 4, 4096, 5, "uniform", 1e-3, 0),       # padding, KL term
    (3, 4, 52, 3, "uniform", 0.0, 1),          # short rows, many responses per tile, shifted rows
    (16, 16, 2048, 9, "uniform", 0.0, 0),      # 2^19 slots: the call runs the two passes in turn
    (64, 8, 16, 4, "full", 0.0, 0),            # 64 responses per 1024 slots: too many rows per tile for one sweep
])
def test_one_sweep_equals_the_two_calls_and_the_oracle(P, G_, T, U, lengths, beta, row_shift):
    ro = synth.rollout(51, P, G_, T, lengths=lengths, min_len=2, rewards="uniform", mask_first_column=bool(row_shift))
    ro.logp_old[:] = ro.logp_new + np.random.default_rng(3).normal(0, 0.1, ro.logp_new.shape).astype(np.float32)
    sl = slice(0, ro.n_resp)
    rms = np.random.default_rng(4).random((U, ro.n_resp * T + 8), dtype=np.float32) + np.float32(0.25)
    omega, E, sw = fused(ro, rms, sl, beta=beta, row_shift=row_shift)
    two = G.grpo_coeffs(ro, N_norm=ro.n_valid, beta=beta, extras=False)["omega"]
    E2, sw2 = G.unit_exposure(two, ro.mask, rms, row_shift=row_shift)
    assert omega.tobytes() == two.tobytes() and E.tobytes() == E2.tobytes() and sw == sw2
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, r, _ = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, ro.logp_ref if beta else None, ro.mask, N_norm=ro.n_valid, beta=beta)
    oE, osw = oracle.unit_exposure(w, ro.mask, rms, row_shift=row_shift)
    assert G.rel_err(E, oE).max() <= 1e-5 and abs(sw - osw) <= 1e-5 * osw


def test_microbatch_slice_of_a_rollout_batch():
    ro = synth.rollout(52, 4, 16, 512, rewards="bernoulli", equal_group_fraction=0.25)
    sl = slice(24, 40)                                        # straddles two prompt groups
    rms = np.random.default_rng(5).random((7, 16 * 512), dtype=np.float32) + np.float32(0.5)
    omega, E, _ = fused(ro, rms, sl)
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, _, _ = oracle.grpo_coeffs(adv[sl], ro.logp_new[sl], ro.logp_old[sl], None, ro.mask[sl], N_norm=ro.n_valid)
    oE, _ = oracle.unit_exposure(w, ro.mask[sl], rms)
    assert G.rel_err(omega, w).max() <= 1e-5 and G.rel_err(E, oE).max() <= 1e-5


def test_argument_errors():
    z = torch.zeros(64, device="cuda")
    m = torch.zeros(64, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    call = lambda **k: api.hilore_coeffs_exposure(z, k.get("n_resp", 4), k.get("G", 4), 0, 4, k.get("T", 16), z, z, None, m,
                                                  k.get("N", 3), None, 0.2, k.get("beta", 0.0), 1e-6, z, 1, 64, 0, 1e-8,
                                                  k.get("omega", z), z, None, ws, k.get("nws", 4096), check=False)
    assert call() == api.OK
    assert call(omega=None) == api.INVALID_ARG and call(N=0) == api.ZERO_NORM and call(beta=0.5) == api.INVALID_ARG
    assert call(T=18) == api.SHAPE and call(n_resp=5) == api.SHAPE and call(nws=8) == api.WORKSPACE


def scores_plan(ro, rms, sl, shapes, kappa, ebar, tau, avail, beta=0.0, row_shift=0, fmt=None):
    """hilore_scores_plan on rows `sl` of a rollout: -> omega, E, sum|omega|, psi, action, recompute, retained bytes."""
    n_rows, T = sl.stop - sl.start, ro.T
    U, ld = rms.shape
    fmt = [api.FMT_E4M3FN_BLK] * U if fmt is None else fmt
    units = [dict(rows=r, cols=c, fmt=f, block=64 if f else 0) for (r, c), f in zip(shapes, fmt)]
    udev, _ = api.make_unit_table(units, "cuda")
    nws = api.hilore_scores_plan_workspace_bytes(U, n_rows * T)
    ws, omega, E, sw = G.Guarded(nws, fill=0xA5), G.Guarded(n_rows * T * 4), G.Guarded(U * 4), G.Guarded(4)
    psi, act, rec, ret = G.Guarded(U * 4), G.Guarded(U), G.Guarded(U), G.Guarded(U * 8)
    api.hilore_scores_plan(G.dev(ro.rewards), ro.n_resp, ro.G, sl.start, n_rows, T, G.dev(ro.logp_new[sl]), G.dev(ro.logp_old[sl]),
                           G.dev(ro.logp_ref[sl]) if beta else None, G.dev(ro.mask[sl]), ro.n_valid, None, 0.2, beta, 1e-6,
                           G.dev(rms), U, ld, row_shift, 1e-8, omega.ptr(), E.ptr(), sw.ptr(), udev, G.dev(kappa), G.dev(ebar),
                           tau[0], tau[1], G.dev(avail), act.ptr(), psi.ptr(), rec.ptr(), ret.ptr(), ws.ptr(), nws)
    ws.numpy(np.uint8, (nws,))
    return (omega.numpy(np.float32, (n_rows, T)), E.numpy(np.float32, (U,)), float(sw.numpy(np.float32, (1,))[0]),
            psi.numpy(np.float32, (U,)), act.numpy(np.uint8, (U,)), rec.numpy(np.uint8, (U,)), ret.numpy(np.uint64, (U,)))


@pytest.mark.parametrize("P,G_,T,U,lengths,beta,row_shift", [
    (1, 8, 1024, 84, "full", 0.0, 0),          # one microbatch of the 1.5B-shaped configuration
    (1, 8, 2048, 84, "uniform", 0.0, 0),       # one microbatch of the 7B-shaped configuration, padded
    (2, 4, 4096, 5, "uniform", 1e-3, 0),       # KL term
    (3, 4, 52, 3, "uniform", 0.0, 1),          # short rows, shifted rows
    (16, 16, 2048, 9, "uniform", 0.0, 0),      # 2^19 slots: coefficient pass first, then reduction + plan in one launch
])
def test_single_launch_refresh_equals_the_separate_calls_and_the_oracle(P, G_, T, U, lengths, beta, row_shift, monkeypatch):
    ro = synth.rollout(71, P, G_, T, lengths=lengths, min_len=2, rewards="uniform", mask_first_column=bool(row_shift))
    ro.logp_old[:] = ro.logp_new + np.random.default_rng(5).normal(0, 0.1, ro.logp_new.shape).astype(np.float32)
    sl = slice(0, ro.n_resp)
    rng = np.random.default_rng(6)
    rms = rng.random((U, ro.n_resp * T), dtype=np.float32) + np.float32(0.25)
    shapes = [(ro.n_resp * T, int(c)) for c in rng.choice([1536, 3584, 8960, 18944], U)]
    fmt = [int(f) for f in rng.choice([api.FMT_E4M3FN_RAW, api.FMT_E4M3FN_BLK], U)]
    kappa = rng.uniform(0.5, 2.0, U).astype(np.float32)
    ebar = rng.uniform(0.01, 0.03, U).astype(np.float32)
    avail = rng.choice([api.ACT_R, api.ACT_H, api.ACT_H, api.ACT_L], U).astype(np.uint8)
    # thresholds from the separate calls' psi, between order statistics
    omega2, E2, sw2 = fused(ro, rms, sl, beta=beta, row_shift=row_shift)
    p2 = (kappa * E2).astype(np.float32) * ebar
    srt = np.sort(p2)
    tau = (float((srt[U // 2 - 1] + srt[U // 2]) / 2), float((srt[-(U // 3) - 1] + srt[-(U // 3)]) / 2)) if U >= 3 else (0.0, 1.0)
    omega, E, sw, psi, act, rec, ret = scores_plan(ro, rms, sl, shapes, kappa, ebar, tau, avail, beta, row_shift, fmt)
    assert omega.tobytes() == omega2.tobytes() and E.tobytes() == E2.tobytes() and sw == sw2
    # the plan of the separate DECIDE call on the same exposure, and of the oracle
    oa, opsi, orec, oret = oracle.plan(E2, kappa, ebar, tau[0], tau[1], avail, [s[0] for s in shapes], [s[1] for s in shapes], fmt,
                                       [64 if f else 0 for f in fmt])
    assert np.array_equal(act, oa) and np.array_equal(rec, orec) and np.array_equal(ret, oret)
    assert psi.tobytes() == opsi.tobytes()
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, _, _ = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, ro.logp_ref if beta else None, ro.mask, N_norm=ro.n_valid, beta=beta)
    oE, _ = oracle.unit_exposure(w, ro.mask, rms, row_shift=row_shift)
    assert G.rel_err(E, oE).max() <= 1e-5
    # twice in a row on the same workspace: the finished-CTA counter is left clean
    again = scores_plan(ro, rms, sl, shapes, kappa, ebar, tau, avail, beta, row_shift, fmt)
    assert again[1].tobytes() == E.tobytes() and np.array_equal(again[4], act)
    # without thread-block clusters (the counter form of the single launch; workspace forms of the separate calls)
    monkeypatch.setenv("HILORE_DISABLE_CLUSTER_LAUNCH", "1")
    plain = scores_plan(ro, rms, sl, shapes, kappa, ebar, tau, avail, beta, row_shift, fmt)
    assert plain[0].tobytes() == omega.tobytes() and plain[1].tobytes() == E.tobytes() and plain[3].tobytes() == psi.tobytes()
    assert np.array_equal(plain[4], act) and np.array_equal(plain[6], ret)
    omega3, E3, sw3 = fused(ro, rms, sl, beta=beta, row_shift=row_shift)
    assert omega3.tobytes() == omega.tobytes() and E3.tobytes() == E.tobytes() and sw3 == sw


def test_single_launch_refresh_argument_errors():
    z = torch.zeros(64, device="cuda")
    m = torch.zeros(64, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    udev, _ = api.make_unit_table([dict(rows=64, cols=64, fmt=1, block=64)], "cuda")
    call = lambda **k: api.hilore_scores_plan(z, 4, 4, 0, 4, k.get("T", 16), z, z, None, m, k.get("N", 3), None, 0.2, 0.0, 1e-6, z,
                                              k.get("U", 1), 64, 0, 1e-8, z, z, None, k.get("units", udev), z, z, 0.0, 1.0,
                                              k.get("avail", m), m, None, None, None, ws, k.get("nws", 4096), check=False)
    assert call() == api.OK
    assert call(units=None) == api.INVALID_ARG and call(avail=None) == api.INVALID_ARG and call(U=0) == api.INVALID_ARG
    assert call(N=0) == api.ZERO_NORM and call(T=18) == api.SHAPE
    assert call(nws=api.hilore_workspace_bytes(1, 64)) == api.WORKSPACE       # no room for the counter
