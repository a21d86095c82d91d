"""Parity of the omega diagnostics and the score variants with the oracle: counts exact; top-decile share and
sum |omega| within 1e-9 relative (same fp32 values, fp64 sums); variants within 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def diag_gpu(adv, ratio, mask, omega, clip_eps=0.2):
    n_rows, T = omega.shape
    nws = api.hilore_omega_diagnostics_workspace_bytes()
    ws, counts, share, total = G.Guarded(nws), G.Guarded(40), G.Guarded(8), G.Guarded(8)
    api.hilore_omega_diagnostics(G.dev(adv), G.dev(ratio), G.dev(mask), G.dev(omega), n_rows, T, clip_eps, counts.ptr(),
                                 share.ptr(), total.ptr(), ws.ptr(), nws)
    ws.numpy(np.uint8, (nws,))
    return counts.numpy(np.int64, (5,)), float(share.numpy(np.float64, (1,))[0]), float(total.numpy(np.float64, (1,))[0])


def coeffs(ro, beta=0.0, variant=None):
    t = G.dev
    n_rows, T = ro.logp_new.shape
    adv, omega, ratio, chi = G.Guarded(n_rows * 4), G.Guarded(n_rows * T * 4), G.Guarded(n_rows * T * 4), G.Guarded(n_rows * T)
    args = (t(ro.rewards), ro.n_resp, ro.G, 0, n_rows, T, t(ro.logp_new), t(ro.logp_old), t(ro.logp_ref) if beta else None,
            t(ro.mask), ro.n_valid, None, 0.2, beta, 1e-6)
    if variant is None:
        api.hilore_grpo_coeffs(*args, adv.ptr(), omega.ptr(), ratio.ptr(), chi.ptr())
    else:
        api.hilore_grpo_coeffs_variant(*args, variant, adv.ptr(), omega.ptr(), ratio.ptr(), chi.ptr())
    return (adv.numpy(np.float32, (n_rows,)), omega.numpy(np.float32, (n_rows, T)), ratio.numpy(np.float32, (n_rows, T)),
            chi.numpy(np.uint8, (n_rows, T)))


def oracle_record(ro):
    """adv, omega, ratio of a rollout from the oracle (host inputs only)."""
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, r, _ = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask, N_norm=ro.n_valid)
    return adv, w, r


@pytest.mark.parametrize("P,G_,T,lengths", [(4, 8, 256, "full"), (64, 8, 1024, "uniform"), (3, 4, 52, "uniform")])
def test_diagnostics_match_oracle(P, G_, T, lengths):
    """The same record (written by the oracle from host inputs) through both diagnostics: counts exact."""
    ro = synth.rollout(7, P, G_, T, rewards="bernoulli", lengths=lengths, min_len=8)
    ro.logp_old[:] = ro.logp_new + np.random.default_rng(1).normal(0, 0.15, ro.logp_new.shape).astype(np.float32)
    adv, omega, ratio = oracle_record(ro)
    counts, share, total = diag_gpu(adv, ratio, ro.mask, omega)
    oc, oshare, ototal = oracle.omega_diagnostics(adv, ratio, ro.mask, omega)
    assert counts.tolist() == oc.tolist()
    assert share == pytest.approx(oshare, rel=1e-9) and total == pytest.approx(ototal, rel=1e-9)
    assert counts[3] == counts[0] + counts[1] + counts[2]                 # Remark 1 accounting at beta = 0
    a = diag_gpu(adv, ratio, ro.mask, omega)
    assert a[1] == share and a[2] == total                                  # deterministic


def test_diagnostics_of_the_gpu_record_end_to_end():
    """GPU coefficients -> GPU diagnostics against oracle coefficients -> oracle diagnostics.  The log-ratios keep a
    distance from the clip bounds, so that the two chains classify every slot alike."""
    ro = synth.rollout(9, 32, 8, 512, rewards="bernoulli", lengths="uniform", min_len=8)
    d = np.random.default_rng(2).normal(0, 0.15, ro.logp_new.shape).astype(np.float32)
    for bound in (np.log(1.2), np.log(0.8)):
        close = np.abs(d - bound) < 1e-3
        d[close] += np.float32(4e-3)
    ro.logp_old[:] = ro.logp_new - d
    adv_g, omega_g, ratio_g, _ = coeffs(ro)
    counts, share, total = diag_gpu(adv_g, ratio_g, ro.mask, omega_g)
    adv, omega, ratio = oracle_record(ro)
    oc, oshare, ototal = oracle.omega_diagnostics(adv, ratio, ro.mask, omega)
    assert counts.tolist() == oc.tolist()
    assert share == pytest.approx(oshare, rel=1e-5) and total == pytest.approx(ototal, rel=1e-5)


def test_diagnostics_ties_and_degenerate_records():
    n_rows, T = 4, 25
    adv, ratio, mask = np.ones(n_rows, np.float32), np.ones((n_rows, T), np.float32), np.ones((n_rows, T), np.uint8)
    for w in (np.full((n_rows, T), 0.5, np.float32),                        # all tied: the decile carries 10 %
              np.zeros((n_rows, T), np.float32),
              np.where(np.arange(100).reshape(n_rows, T) % 7 == 0, -2.0, 1e-3).astype(np.float32)):
        counts, share, total = diag_gpu(adv, ratio, mask, w)
        oc, oshare, ototal = oracle.omega_diagnostics(adv, ratio, mask, w)
        assert counts.tolist() == oc.tolist() and share == pytest.approx(oshare, rel=1e-12, abs=1e-15)
        assert total == pytest.approx(ototal, rel=1e-12, abs=1e-15)
    # the strict clipping test of the diagnostics: r exactly on a bound is not clipped
    ratio2 = np.full((n_rows, T), np.float32(1.0) + np.float32(0.2), np.float32)
    counts, _, _ = diag_gpu(adv, ratio2, mask, np.ones((n_rows, T), np.float32))
    assert counts[2] == 0
    counts, _, _ = diag_gpu(adv, np.nextafter(ratio2, np.float32(2)), mask, np.ones((n_rows, T), np.float32))
    assert counts[2] == n_rows * T


@pytest.mark.parametrize("beta", [0.0, 1e-3])
def test_score_variants(beta):
    ro = synth.rollout(8, 16, 8, 512, lengths="uniform")
    adv_o = oracle.group_advantages(ro.rewards, 8)
    for variant in (0, 1, 2):
        adv, omega, ratio, chi = coeffs(ro, beta=beta, variant=variant)
        w, r, c = oracle.grpo_coeffs_variant(adv_o, ro.logp_new, ro.logp_old, ro.logp_ref if beta else None, ro.mask,
                                             ro.n_valid, 0.2, beta, variant)
        hi, lo = np.float32(1.2), np.float32(0.8)
        near = (np.abs(r - hi) <= 4 * np.spacing(hi)) | (np.abs(r - lo) <= 4 * np.spacing(lo))
        ok = ~near if variant == 0 else np.ones_like(near)
        err = G.rel_err(omega[ok], w[ok])
        # where the policy and K3 terms cancel, allow 1e-5 of the larger term
        kl = beta * ro.mask / ro.n_valid * (1 - np.exp(ro.logp_ref.astype(np.float64) - ro.logp_new))
        floor = 1e-5 * np.maximum(np.abs(w.astype(np.float64) - kl), np.abs(kl))[ok]
        assert np.all((err <= 1e-5) | (np.abs(omega[ok].astype(np.float64) - w[ok]) <= floor))
        assert G.rel_err(ratio, r).max() <= 1e-5
    base = coeffs(ro, beta=beta)[1]
    assert np.array_equal(base, coeffs(ro, beta=beta, variant=0)[1])
    # advantage-only exposure through the ordinary exposure call
    adv, sig, _, _ = coeffs(ro, beta=beta, variant=2)
    rms = (np.random.default_rng(2).random((3, ro.n_resp * ro.T), dtype=np.float32) + np.float32(0.5))
    E, _ = G.unit_exposure(sig, ro.mask, rms)
    oE, _ = oracle.unit_exposure((ro.mask * adv_o[:, None]).astype(np.float32), ro.mask, rms)
    assert G.rel_err(E, oE).max() <= 1e-5
