"""Parity of hilore_mask_count / hilore_grpo_coeffs / hilore_unit_exposure with the CPU oracle.

fp32 outputs: 1e-5 relative (signed zeros equal).  The clip indicator is an integer decided by an
fp32 compare of r = exp(s - s_old); the oracle rounds a double exp, the kernel evaluates
ex2.approx(d * log2 e), whose relative error is bounded by |d| * 2^-24 + 2^-22 (2.4e-7 plus 6e-8 per
unit of |d|: about 3 ulp of a ratio near the clip bounds 0.8 and 1.2, and below 6e-6 up to |d| = 80), so
a slot whose oracle ratio lies within 4 ulp of a clip bound may legitimately differ and is excused (and
counted).  All calls go through the C ABI.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def check_coeffs(ro, got, *, resp_offset=0, N=None, beta=0.0, clip_eps=0.2):
    n_rows = got["omega"].shape[0]
    sl = slice(resp_offset, resp_offset + n_rows)
    adv_all = oracle.group_advantages(ro.rewards, ro.G)
    N = ro.n_valid if N is None else N
    w, r, chi = oracle.grpo_coeffs(adv_all[sl], ro.logp_new[sl], ro.logp_old[sl], ro.logp_ref[sl], ro.mask[sl],
                                   N_norm=N, clip_eps=clip_eps, beta=beta)
    assert G.rel_err(got["adv"], adv_all[sl]).max() <= RTOL
    assert np.array_equal(got["adv"] == 0, adv_all[sl] == 0)
    hi, lo = np.float32(1) + np.float32(clip_eps), np.float32(1) - np.float32(clip_eps)
    near = (np.abs(r - hi) <= 4 * np.spacing(hi)) | (np.abs(r - lo) <= 4 * np.spacing(lo))
    if "chi" in got:
        bad = got["chi"] != chi
        assert not np.any(bad & ~near), "clip indicator differs away from the clip bounds"
        assert G.rel_err(got["ratio"], r).max() <= RTOL
    ok = ~near
    err = G.rel_err(got["omega"][ok], w[ok])
    if beta != 0:
        # where the policy and K3 terms cancel, allow 1e-5 of the larger term (reported, not hidden)
        kl = beta * ro.mask[sl] / N * (1 - np.exp(ro.logp_ref[sl].astype(np.float64) - ro.logp_new[sl]))
        floor = RTOL * np.maximum(np.abs(w.astype(np.float64) - kl), np.abs(kl))[ok]
        assert np.all((err <= RTOL) | (np.abs(got["omega"][ok].astype(np.float64) - w[ok]) <= floor))
    else:
        assert err.max(initial=0) <= RTOL, err.max()
    assert np.all(got["omega"][ro.mask[sl] == 0] == 0)
    return int(near.sum())


def test_config1_tiny():
    """4 prompts x G=8 x 256 tokens, Bernoulli rewards, all slots valid."""
    ro = synth.rollout(0, 4, 8, 256)
    check_coeffs(ro, G.grpo_coeffs(ro, N_norm=ro.n_valid))


def test_config2_rollout_batch_and_microbatches():
    """64 prompts x 8 x 1024 in one call, and as 64 microbatches of 8 responses with resp_offset."""
    ro = synth.rollout(0, 64, 8, 1024)
    whole = G.grpo_coeffs(ro, N_norm=ro.n_valid)
    check_coeffs(ro, whole)
    for mb in (0, 17, 63):
        part = G.grpo_coeffs(ro, resp_offset=mb * 8, n_rows=8, N_norm=ro.n_valid)
        check_coeffs(ro, part, resp_offset=mb * 8)
        assert np.array_equal(part["omega"], whole["omega"][mb * 8:mb * 8 + 8])


def test_group_straddles_microbatches():
    """G=16 with microbatches of 8 responses: a prompt group spans two calls."""
    ro = synth.rollout(1, 8, 16, 512)
    for off in (0, 8, 24, 120):
        check_coeffs(ro, G.grpo_coeffs(ro, resp_offset=off, n_rows=8, N_norm=ro.n_valid), resp_offset=off)


def test_variable_length_masks_and_equal_groups():
    """Lengths U{128..T}, rewards U[0,1), 5% of the groups all-equal (non-dyadic values): omega exactly 0."""
    ro = synth.rollout(0, 64, 8, 2048, rewards="uniform", lengths="uniform", equal_group_fraction=0.05)
    got = G.grpo_coeffs(ro, N_on_device=True)
    assert got["N"] == ro.n_valid
    check_coeffs(ro, got)
    Rg = ro.rewards.reshape(-1, 8)
    eq = np.where((Rg.max(axis=1) == Rg.min(axis=1)))[0]
    assert len(eq) == 3
    for g in eq:
        assert np.all(got["omega"][g * 8:(g + 1) * 8] == 0) and np.all(got["adv"][g * 8:(g + 1) * 8] == 0)


@pytest.mark.parametrize("beta", [1e-3, 0.5])
def test_k3_regulariser(beta):
    ro = synth.rollout(2, 16, 8, 512, lengths="uniform")
    ro.rewards[8:16] = 1.0       # zero-advantage group keeps its K3 contribution
    got = G.grpo_coeffs(ro, N_norm=ro.n_valid, beta=beta)
    check_coeffs(ro, got, beta=beta)
    live = ro.mask[8:16] == 1
    assert np.all(got["omega"][8:16][live] != 0)


def test_without_optional_outputs_and_other_clip_radius():
    ro = synth.rollout(3, 8, 8, 1280)      # T not a multiple of the 1024-slot tile
    a = G.grpo_coeffs(ro, N_norm=12345, extras=False, clip_eps=0.05)
    b = G.grpo_coeffs(ro, N_norm=12345, extras=True, clip_eps=0.05)
    assert np.array_equal(a["omega"], b["omega"])
    assert (b["chi"] == 0).mean() > 0.05
    check_coeffs(ro, b, N=12345, clip_eps=0.05)


def test_ratio_one_gives_minus_adv_over_N():
    ro = synth.rollout(4, 4, 8, 256)
    ro.logp_old[:] = ro.logp_new
    got = G.grpo_coeffs(ro, N_norm=ro.n_valid)
    assert np.all(got["ratio"] == 1) and np.all(got["chi"] == 1)
    adv = oracle.group_advantages(ro.rewards, 8).astype(np.float64)
    assert G.rel_err(got["omega"], -adv[:, None] / ro.n_valid * np.ones((1, 256))).max() <= RTOL


def test_mask_count_sizes_and_alignment():
    import torch
    rng = np.random.default_rng(0)
    for n in (0, 1, 15, 16, 17, 4097, 1 << 20):
        m = (rng.random(n + 3) < 0.4).astype(np.uint8)
        d = G.dev(m)
        out = torch.full((1,), -7, dtype=torch.int64, device="cuda")
        api.hilore_mask_count(d, n, out)
        assert int(out.item()) == int(m[:n].sum())
        api.hilore_mask_count(d[1:], n, out)       # unaligned base
        assert int(out.item()) == int(m[1:n + 1].sum())


def _rms_for(ro, U, seed):
    rng = np.random.default_rng(seed)
    return (rng.random((U, ro.n_resp * ro.T), dtype=np.float32) * np.float32(2) + np.float32(0.25))


def oracle_omega(ro):
    """Coefficients of a rollout from the oracle (host inputs only): the common input of both exposure paths."""
    adv = oracle.group_advantages(ro.rewards, ro.G)
    return oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask, N_norm=ro.n_valid)[0]


@pytest.mark.parametrize("U", [1, 2, 9, 84])
def test_exposure_config1(U):
    ro = synth.rollout(0, 4, 8, 256)
    omega = oracle_omega(ro)
    rms = _rms_for(ro, U, 1)
    E, sw = G.unit_exposure(omega, ro.mask, rms)
    oE, osw = oracle.unit_exposure(omega, ro.mask, rms)
    assert G.rel_err(E, oE).max() <= RTOL and abs(sw - osw) <= RTOL * osw


def test_exposure_masked_microbatch_and_row_shift():
    """Microbatch of 4 responses x 4096 slots with padding; both row conventions."""
    ro = synth.rollout(0, 1, 4, 4096, rewards="uniform", lengths="uniform", mask_first_column=True)
    omega = oracle_omega(ro)
    rms = _rms_for(ro, 5, 2)
    rms[:, ro.mask.reshape(-1) == 0] = 1e9          # padded rows must not contribute
    for shift in (0, 1):
        r = rms.copy()
        if shift:
            r = np.roll(rms.reshape(5, 4, 4096), -1, axis=2).reshape(5, -1).copy()
        E, sw = G.unit_exposure(omega, ro.mask, r, row_shift=shift)
        oE, osw = oracle.unit_exposure(omega, ro.mask, r, row_shift=shift)
        assert G.rel_err(E, oE).max() <= RTOL and abs(sw - osw) <= RTOL * osw
    E0, _ = G.unit_exposure(omega, ro.mask, rms, row_shift=0)
    E1, _ = G.unit_exposure(omega, ro.mask, np.roll(rms.reshape(5, 4, 4096), -1, axis=2).reshape(5, -1).copy(), row_shift=1)
    assert G.rel_err(E1, E0).max() <= RTOL


def test_exposure_degenerate_cases():
    ro = synth.rollout(5, 2, 4, 64)
    omega = oracle_omega(ro)
    rms = _rms_for(ro, 3, 3)
    E, sw = G.unit_exposure(np.zeros_like(omega), ro.mask, rms)
    assert np.all(E == 0) and sw == 0                       # all coefficients zero
    E, sw = G.unit_exposure(omega, np.zeros_like(ro.mask), rms)
    assert np.all(E == 0) and sw == 0                       # empty T_b
    odd = omega.reshape(-1)[:501].reshape(3, 167).copy()    # sizes that defeat the vector path
    m = (np.random.default_rng(1).random((3, 167)) < 0.7).astype(np.uint8)
    r = _rms_for(ro, 3, 4)[:, :501].copy()
    E, sw = G.unit_exposure(odd, m, r)
    oE, osw = oracle.unit_exposure(odd, m, r)
    assert G.rel_err(E, oE).max() <= RTOL
    a, b = G.unit_exposure(omega, ro.mask, rms), G.unit_exposure(omega, ro.mask, rms)
    assert a[0].tobytes() == b[0].tobytes()                 # fixed reduction order


def test_exposure_from_fused_token_rms():
    """End of the chain on the device (coefficients and token RMS as the kernels wrote them feed
    hilore_unit_exposure) against the oracle's own chain."""
    ro = synth.rollout(0, 4, 8, 256)
    omega = G.grpo_coeffs(ro, N_norm=ro.n_valid)["omega"]
    rng = np.random.default_rng(0)
    units = [synth.activation_unit(rng, 8192, 896) for _ in range(2)]
    rms = np.stack([G.compress(x, api.FMT_E4M3FN_BLK)[2] for x in units])
    E, _ = G.unit_exposure(omega, ro.mask, rms)
    o_rms = np.stack([oracle.row_rms(x) for x in units])
    oE, _ = oracle.unit_exposure(oracle_omega(ro), ro.mask, o_rms)
    assert G.rel_err(E, oE).max() <= RTOL


def test_ratio_over_the_whole_exponent_range():
    """Log-ratio from -80 to +80 (r from 1e-35 to 5e34): ratio and omega stay within 1e-5 of the oracle."""
    ro = synth.rollout(41, 4, 4, 1024, rewards="uniform")
    d = np.linspace(-80.0, 80.0, ro.logp_new.size, dtype=np.float32).reshape(ro.logp_new.shape)
    ro.logp_old[:] = ro.logp_new - d
    got = G.grpo_coeffs(ro, N_norm=ro.n_valid)
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, r, chi = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask, N_norm=ro.n_valid)
    assert G.rel_err(got["ratio"], r).max() <= RTOL
    hi, lo = np.float32(1.2), np.float32(0.8)
    near = (np.abs(r - hi) <= 4 * np.spacing(hi)) | (np.abs(r - lo) <= 4 * np.spacing(lo))
    assert np.array_equal(got["chi"][~near], chi[~near])
    assert G.rel_err(got["omega"][~near], w[~near]).max() <= RTOL


@pytest.mark.parametrize("seed", range(4))
def test_random_rollouts_and_microbatch_slices(seed):
    """Random group sizes, lengths, rewards, clip radii, KL weights and microbatch slices against the oracle."""
    rng = np.random.default_rng(500 + seed)
    for _ in range(4):
        Gs = int(rng.choice([1, 2, 4, 8, 16, 32, 48]))
        P = int(rng.integers(1, 9))
        T = 4 * int(rng.integers(1, 600))
        ro = synth.rollout(int(rng.integers(0, 1 << 30)), P, Gs, T, rewards=str(rng.choice(["bernoulli", "uniform"])),
                           lengths=str(rng.choice(["full", "uniform"])), min_len=1,
                           equal_group_fraction=float(rng.choice([0.0, 0.5])))
        ro.logp_old[:] = ro.logp_new + rng.normal(0, float(rng.choice([0.01, 0.1, 0.4])), ro.logp_new.shape).astype(np.float32)
        beta = float(rng.choice([0.0, 1e-3, 0.3]))
        clip = float(rng.choice([0.1, 0.2, 0.28]))
        off = int(rng.integers(0, ro.n_resp))
        n_rows = int(rng.integers(1, ro.n_resp - off + 1))
        got = G.grpo_coeffs(ro, resp_offset=off, n_rows=n_rows, N_norm=ro.n_valid, clip_eps=clip, beta=beta)
        check_coeffs(ro, got, resp_offset=off, beta=beta, clip_eps=clip)


def test_k3_term_alone_over_a_wide_range_of_log_ratios():
    """Zero advantages (equal rewards): omega is the K3 term only, beta/N * (1 - exp(s_ref - s)); it must hold 1e-5
    relative from |s_ref - s| = 1e-6 (no cancellation) to 30 (no overflow), on both sides of the 0.5 switch."""
    ro = synth.rollout(43, 2, 4, 1024, rewards="uniform", equal_group_fraction=1.0)
    mag = np.logspace(-6, np.log10(30.0), ro.logp_new.size // 2, dtype=np.float64)
    d = np.concatenate([mag, -mag]).astype(np.float32).reshape(ro.logp_new.shape)
    d.reshape(-1)[[0, 1, 2, 3]] = np.float32([0.5, -0.5, np.nextafter(np.float32(0.5), np.float32(1)), 0.0])
    ro.logp_ref[:] = ro.logp_new + d
    got = G.grpo_coeffs(ro, N_norm=ro.n_valid, beta=0.25)
    adv = oracle.group_advantages(ro.rewards, ro.G)
    assert np.all(adv == 0)
    w, _, _ = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, ro.logp_ref, ro.mask, N_norm=ro.n_valid, beta=0.25)
    assert G.rel_err(got["omega"], w).max() <= RTOL


def test_normaliser_of_this_call_matches_the_oracles_zero_rule():
    """The oracle takes N_norm = 0 as "the sum of the mask over this call".  The library keeps no scratch of its own,
    so the same rule is two stream-ordered calls: hilore_mask_count of the call's mask into a device word, which the
    coefficient kernel reads (no host synchronisation); a host N_norm <= 0 without that word is refused."""
    ro = synth.rollout(51, 4, 8, 512, rewards="uniform", lengths="uniform")
    off, n_rows = 8, 16
    sl = slice(off, off + n_rows)
    R, ln, lo, mk = G.dev(ro.rewards), G.dev(ro.logp_new[sl]), G.dev(ro.logp_old[sl]), G.dev(ro.mask[sl])
    omega = G.Guarded(n_rows * ro.T * 4)
    for bad in (0, -5):
        st = api.hilore_grpo_coeffs(R, ro.n_resp, ro.G, off, n_rows, ro.T, ln, lo, None, mk, bad, None, 0.2, 0.0, 1e-6, None,
                                    omega.ptr(), None, None, check=False)
        assert st == api.ZERO_NORM
    ndev = torch.full((1,), -7, dtype=torch.int64, device="cuda")
    api.hilore_mask_count(mk, mk.numel(), ndev)
    api.hilore_grpo_coeffs(R, ro.n_resp, ro.G, off, n_rows, ro.T, ln, lo, None, mk, 0, ndev, 0.2, 0.0, 1e-6, None, omega.ptr(),
                           None, None)
    got = omega.numpy(np.float32, (n_rows, ro.T))
    adv = oracle.group_advantages(ro.rewards, ro.G)
    w, r, _ = oracle.grpo_coeffs(adv[sl], ro.logp_new[sl], ro.logp_old[sl], None, ro.mask[sl], N_norm=0)
    assert int(ndev.item()) == int(ro.mask[sl].sum())
    hi, lo_b = np.float32(1.2), np.float32(0.8)
    near = (np.abs(r - hi) <= 4 * np.spacing(hi)) | (np.abs(r - lo_b) <= 4 * np.spacing(lo_b))
    assert G.rel_err(got[~near], w[~near]).max() <= RTOL
    # a call whose mask is empty: the oracle refuses (no normaliser), the device word is 0 and every coefficient is 0
    empty = np.zeros_like(ro.mask[sl])
    with pytest.raises(oracle.OracleError) as e:
        oracle.grpo_coeffs(adv[sl], ro.logp_new[sl], ro.logp_old[sl], None, empty, N_norm=0)
    assert e.value.status == oracle.ZERO_NORM
    mk0 = G.dev(empty)
    api.hilore_mask_count(mk0, mk0.numel(), ndev)
    api.hilore_grpo_coeffs(R, ro.n_resp, ro.G, off, n_rows, ro.T, ln, lo, None, mk0, 0, ndev, 0.2, 0.0, 1e-6, None, omega.ptr(),
                           None, None)
    assert int(ndev.item()) == 0 and np.all(omega.numpy(np.float32, (n_rows, ro.T)) == 0)


def test_coefficients_at_the_top_of_the_sweep_every_slot():
    """2^24 slots at G = 16, T = 1024 (16 384 responses, the largest point of the bandwidth sweep), with and without
    the K3 term: every slot and every advantage against the oracle."""
    ro = synth.rollout(61, 1024, 16, 1024)
    R, ln, lo, lr, mk = (G.dev(a) for a in (ro.rewards, ro.logp_new, ro.logp_old, ro.logp_ref, ro.mask))
    for beta in (0.0, 1e-3):
        omega = torch.full((ro.n_resp, ro.T), 7.0, dtype=torch.float32, device="cuda")
        a_out = torch.full((ro.n_resp,), 7.0, dtype=torch.float32, device="cuda")
        api.hilore_grpo_coeffs(R, ro.n_resp, ro.G, 0, ro.n_resp, ro.T, ln, lo, lr if beta else None, mk, ro.n_valid, None, 0.2,
                               beta, 1e-6, a_out, omega, None, None)
        check_coeffs(ro, dict(adv=a_out.cpu().numpy(), omega=omega.cpu().numpy()), N=ro.n_valid, beta=beta)


def test_exposure_shifted_rows_with_a_valid_first_slot():
    """row_shift = 1 and the first slot of every response in T_b: the slot has no activation row and carries no weight
    (neither in the mean nor in the sum); dense and packed layouts against the oracle."""
    ro = synth.rollout(81, 3, 4, 96, rewards="uniform", lengths="uniform", min_len=5)
    assert ro.mask[:, 0].all()
    rng = np.random.default_rng(82)
    omega = (rng.standard_normal((ro.n_resp, ro.T)) * 1e-4).astype(np.float32) * ro.mask
    rms = rng.random((5, ro.n_resp * ro.T), dtype=np.float32) + np.float32(0.25)
    E, sw = G.unit_exposure(omega, ro.mask, rms, row_shift=1)
    oE, osw = oracle.unit_exposure(omega, ro.mask, rms, row_shift=1)
    assert G.rel_err(E, oE).max() <= RTOL and abs(sw - osw) <= RTOL * osw
    const = np.where(ro.mask != 0, np.float32(2e-4), 0).astype(np.float32)       # mean-one weights over the slots with a row
    Ec, _ = G.unit_exposure(const, ro.mask, rms, row_shift=1, eps_alpha=0.0)
    assert G.rel_err(Ec, np.full(5, 2e-4 * int(ro.mask[:, 1:].sum()))).max() <= RTOL
    # packed: every sequence starts with its first response token (no prompt), so the same slots lack a row
    pk = synth.pack_rollout(ro, 83, max_prompt=0, min_prompt=0)
    om_p = np.concatenate([omega[i, :ro.lengths[i]] for i in range(ro.n_resp)]).astype(np.float32)
    rms_p = rng.random((5, pk.n_tok), dtype=np.float32) + np.float32(0.25)
    nws = api.hilore_workspace_bytes(5, pk.n_tok)
    ws, Eg = G.Guarded(nws), G.Guarded(5 * 4)
    api.hilore_unit_exposure_packed(G.dev(om_p), G.dev(pk.mask), pk.n_tok, G.dev(pk.cu_seqlens), len(pk.rows), G.dev(rms_p), 5,
                                    pk.n_tok, 1, 1e-8, Eg.ptr(), None, ws.ptr(), nws)
    oEp, _ = oracle.unit_exposure_packed(om_p, pk.mask, pk.cu_seqlens, rms_p, row_shift=1)
    assert G.rel_err(Eg.numpy(np.float32, (5,)), oEp).max() <= RTOL


@pytest.mark.parametrize("beta", [0.0, 0.02])
def test_fast_and_generic_coefficient_paths_give_the_same_bits(beta):
    """T % 8 == 0 and 32-byte alignment select the warp-per-tile kernel (256-bit accesses, packed fp32 pairs), anything
    else the 128-bit one: the same inputs at 32-byte and at 16-byte aligned addresses must give identical omega, ratio
    and clip indicator, masked slots included."""
    ro = synth.rollout(91, 6, 8, 1096, rewards="uniform", lengths="uniform", min_len=3)
    ro.logp_ref[:] = ro.logp_new + np.random.default_rng(92).normal(0, 0.2, ro.logp_new.shape).astype(np.float32)
    n, T = ro.n_resp, ro.T

    def run(shift):                                   # shift in elements: 0 -> 32-byte aligned, 4 -> only 16-byte
        pad = lambda a, dt: torch.cat([torch.zeros(shift, dtype=dt, device="cuda"), torch.from_numpy(a.reshape(-1)).cuda()])[shift:]
        big = lambda dt: torch.zeros(n * T + 8, dtype=dt, device="cuda")[shift:shift + n * T]
        ln, lo, lr = (pad(a, torch.float32) for a in (ro.logp_new, ro.logp_old, ro.logp_ref))
        mk = torch.cat([torch.zeros(2 * shift, dtype=torch.uint8, device="cuda"), torch.from_numpy(ro.mask.reshape(-1)).cuda()])[2 * shift:]
        omega, ratio, chi = big(torch.float32), big(torch.float32), torch.zeros(n * T + 16, dtype=torch.uint8, device="cuda")[2 * shift:2 * shift + n * T]
        assert ln.data_ptr() % 32 == (16 if shift else 0)
        api.hilore_grpo_coeffs(G.dev(ro.rewards), n, ro.G, 0, n, T, ln, lo, lr if beta else None, mk, ro.n_valid, None, 0.2, beta,
                               1e-6, None, omega, ratio, chi)
        return omega.cpu().numpy(), ratio.cpu().numpy(), chi.cpu().numpy()

    fast, generic = run(0), run(4)
    for a, b in zip(fast, generic):
        assert a.tobytes() == b.tobytes()


@pytest.mark.parametrize("tiles", [1, 2, 3, 4, 7, 8, 15, 16, 17, 33])
def test_exposure_forms_give_the_same_bits_at_every_tile_count(tiles, monkeypatch):
    """1, 2, 4, 8 and 16 tiles of 1024 tokens take the one-launch form (a thread-block cluster per group of eight units),
    the other counts the workspace and a second kernel; with HILORE_DISABLE_CLUSTER_LAUNCH set every count does.  The
    exposure scores are the oracle's to 1e-5 and the same bits in both forms; U = 11: a full and a partial unit group;
    the last tile is ragged."""
    T = 256
    n_rows = 4 * tiles - 1
    rng = np.random.default_rng(tiles)
    omega = (rng.normal(0, 1e-5, (n_rows, T)) * (rng.random((n_rows, T)) < 0.7)).astype(np.float32)
    mask = (rng.random((n_rows, T)) < 0.8).astype(np.uint8)
    omega *= mask
    rms = (rng.random((11, n_rows * T), dtype=np.float32) + np.float32(0.25))
    E, sw = G.unit_exposure(omega, mask, rms)
    oE, osw = oracle.unit_exposure(omega, mask, rms)
    assert G.rel_err(E, oE).max() <= RTOL and abs(sw - osw) <= RTOL * osw
    monkeypatch.setenv("HILORE_DISABLE_CLUSTER_LAUNCH", "1")
    E2, sw2 = G.unit_exposure(omega, mask, rms)
    assert E2.tobytes() == E.tobytes() and sw2 == sw
