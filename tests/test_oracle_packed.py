"""Pins of the packed-layout oracle functions: hand-worked records, and the dense functions (pinned elsewhere)
on the same tokens laid out with padding."""
import numpy as np
import pytest

import oracle
from paper_2609_33570_b200 import synth

f32 = np.float32


def test_hand_worked_two_sequences():
    # seq 0: prompt, resp, resp (A = +1);  seq 1: prompt, resp (A = -1);  r = 1 everywhere, N = 3
    cu = np.array([0, 3, 5], np.int32)
    s = np.array([-1.0, -2.0, -0.5, -3.0, -1.5], f32)
    mask = np.array([0, 1, 1, 0, 1], np.uint8)
    w, r, chi = oracle.grpo_coeffs_packed(np.array([1, -1], f32), cu, s, s.copy(), None, mask)
    assert np.array_equal(w, np.array([0, -1 / 3, -1 / 3, 0, 1 / 3], f32))
    assert np.array_equal(r, np.ones(5, f32)) and chi.tolist() == [1] * 5
    # r = 2 at token 2 (positive advantage: clipped, omega = 0) and at token 4 (negative advantage: kept, +2/3)
    s_old = s.copy()
    s_old[[2, 4]] -= f32(np.log(2.0))
    w, r, chi = oracle.grpo_coeffs_packed(np.array([1, -1], f32), cu, s, s_old, None, mask)
    assert chi.tolist() == [1, 1, 0, 1, 1] and w[2] == 0
    assert w[4] == pytest.approx(2 / 3, rel=1e-6) and w[1] == f32(-1 / 3)
    # K3 part alone (A = 0): beta / N * (1 - exp(s_ref - s)) at valid tokens
    s_ref = s + f32(0.25)
    w, _, _ = oracle.grpo_coeffs_packed(np.zeros(2, f32), cu, s, s, s_ref, mask, beta=0.5)
    want = 0.5 / 3 * (1 - np.exp(np.float64(f32(0.25))))
    assert w[[0, 3]].tolist() == [0, 0]
    assert np.allclose(w[[1, 2, 4]], want, rtol=1e-6, atol=0)


def test_zero_length_sequences_and_errors():
    cu = np.array([0, 2, 2, 5, 5], np.int32)
    s = np.linspace(-2, -1, 5).astype(f32)
    mask = np.array([0, 1, 0, 1, 1], np.uint8)
    adv = np.array([2.0, 99.0, -1.0, 77.0], f32)       # sequences 1 and 3 own no token: their advantage is unused
    w, _, _ = oracle.grpo_coeffs_packed(adv, cu, s, s.copy(), None, mask)
    assert np.array_equal(w, np.array([0, -2 / 3, 0, 1 / 3, 1 / 3], f32))
    with pytest.raises(oracle.OracleError):
        oracle.grpo_coeffs_packed(adv, np.array([0, 3, 2, 5, 5], np.int32), s, s, None, mask)
    with pytest.raises(oracle.OracleError):
        oracle.grpo_coeffs_packed(adv, cu, s, s, None, np.zeros(5, np.uint8))   # N = 0


@pytest.mark.parametrize("beta", [0.0, 1e-3])
def test_packed_equals_dense_on_the_same_tokens(beta):
    ro = synth.rollout(21, 6, 4, 96, lengths="uniform", min_len=5, rewards="uniform")
    pk = synth.pack_rollout(ro, 3, max_prompt=9)
    adv = oracle.group_advantages(ro.rewards, ro.G)
    N = ro.n_valid
    wd, rd, cd = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, ro.logp_ref if beta else None, ro.mask, N_norm=N,
                                    beta=beta)
    wp, rp, cp = oracle.grpo_coeffs_packed(adv[pk.rows], pk.cu_seqlens, pk.logp_new, pk.logp_old,
                                           pk.logp_ref if beta else None, pk.mask, N_norm=N, beta=beta)
    seq = np.repeat(np.arange(len(pk.rows)), np.diff(pk.cu_seqlens))
    resp = pk.dense_t >= 0
    i, t = pk.rows[seq[resp]], pk.dense_t[resp]
    assert np.array_equal(wp[resp], wd[i, t]) and np.array_equal(rp[resp], rd[i, t]) and np.array_equal(cp[resp], cd[i, t])
    assert np.all(wp[~resp] == 0)
    assert int(resp.sum()) == N
    # N_norm = 0 counts the mask of the packed microbatch itself
    w0, _, _ = oracle.grpo_coeffs_packed(adv[pk.rows], pk.cu_seqlens, pk.logp_new, pk.logp_old, None, pk.mask)
    assert np.array_equal(w0[resp], oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask)[0][i, t])


def test_exposure_hand_worked_first_token_rule():
    cu = np.array([0, 2, 4], np.int32)
    omega = np.array([1, -1, 1, -1], f32)
    mask = np.ones(4, np.uint8)
    rms = np.array([[1, 2, 3, 4]], f32)
    E0, sw = oracle.unit_exposure_packed(omega, mask, cu, rms, row_shift=0, eps_alpha=0.0)
    assert E0[0] == pytest.approx(4.0, rel=1e-7) and sw == 4.0          # mean-one weights: E = sum |omega|
    # row_shift = 1: tokens 0 and 2 have no source row inside their sequence and carry no weight; tokens 1, 3 read
    # rows 0, 2 (a = 1, 3): mean 2, E = (1 * 1 + 1 * 3) / 2 -- the two weights 1/2 and 3/2 average to one
    E1, sw1 = oracle.unit_exposure_packed(omega, mask, cu, rms, row_shift=1, eps_alpha=0.0)
    assert E1[0] == pytest.approx((1 + 3) / ((1 + 3) / 2), rel=1e-7) and sw1 == 4.0
    # one long sequence: only token 0 is skipped; a = 1, 2, 3 with mean 2
    E2, _ = oracle.unit_exposure_packed(omega, mask, np.array([0, 4], np.int32), rms, row_shift=1, eps_alpha=0.0)
    assert E2[0] == pytest.approx((1 + 2 + 3) / ((1 + 2 + 3) / 3), rel=1e-7)


@pytest.mark.parametrize("row_shift", [0, 1])
def test_exposure_packed_equals_dense_of_padded_sequences(row_shift):
    ro = synth.rollout(5, 3, 4, 40, lengths="uniform", min_len=3)
    pk = synth.pack_rollout(ro, 9, max_prompt=6, min_prompt=0)
    rng = np.random.default_rng(0)
    n_seq, n_tok = len(pk.rows), pk.n_tok
    omega = (rng.standard_normal(n_tok).astype(f32) * pk.mask).astype(f32)
    rms = (rng.random((3, n_tok), dtype=f32) + f32(0.25))
    # the same record as whole sequences padded to the longest one
    lens = np.diff(pk.cu_seqlens)
    Tm = int(lens.max())
    om_d, mk_d, rms_d = np.zeros((n_seq, Tm), f32), np.zeros((n_seq, Tm), np.uint8), np.zeros((3, n_seq * Tm), f32)
    for i in range(n_seq):
        a, b = pk.cu_seqlens[i], pk.cu_seqlens[i + 1]
        om_d[i, :b - a], mk_d[i, :b - a] = omega[a:b], pk.mask[a:b]
        rms_d[:, i * Tm:i * Tm + b - a] = rms[:, a:b]
    Ed, swd = oracle.unit_exposure(om_d, mk_d, rms_d, row_shift=row_shift)
    Ep, swp = oracle.unit_exposure_packed(omega, pk.mask, pk.cu_seqlens, rms, row_shift=row_shift)
    assert np.allclose(Ep, Ed, rtol=1e-6, atol=0) and swp == pytest.approx(swd, rel=1e-6)
