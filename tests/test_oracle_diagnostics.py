"""Pins for the oracle's omega diagnostics (structural sparsity, top-decile concentration) and score variants."""
import numpy as np
import pytest

import oracle
from paper_2609_33570_b200 import synth


def test_hand_worked_record():
    # two responses x five slots; eps = 0.2
    adv = np.array([1.0, -2.0], np.float32)
    ratio = np.array([[1.0, 1.3, 1.2, 0.5, 9.0], [0.7, 0.8, 1.5, 1.0, 1.0]], np.float32)
    mask = np.array([[1, 1, 1, 1, 0], [1, 1, 1, 0, 0]], np.uint8)
    omega = np.array([[-.1, 0, -.12, -.05, 0], [0, .16, .3, 0, 0]], np.float32)
    counts, share, total = oracle.omega_diagnostics(adv, ratio, mask, omega)
    # padding: 3; zero advantage: 0; clipped: (A>0, r=1.3) and (A<0, r=0.7) -> 2 (r = 1.2 = 1+eps is not clipped)
    assert counts.tolist() == [3, 0, 2, 5, 10]
    assert total == pytest.approx(0.1 + 0.12 + 0.05 + 0.16 + 0.3, rel=1e-6)
    assert share == pytest.approx(0.3 / total, rel=1e-6)            # ceil(0.1 * 10) = 1 slot: the largest


def test_remark1_accounting_on_a_rollout():
    """beta = 0: the slots with zero coefficient are exactly padding + zero advantage + flat clipped branch."""
    ro = synth.rollout(3, 16, 8, 256, rewards="bernoulli", lengths="uniform", min_len=16)
    ro.rewards[8:16] = 1.0                                         # one zero-advantage group
    ro.logp_old[:] = ro.logp_new + np.random.default_rng(0).normal(0, 0.2, ro.logp_new.shape).astype(np.float32)
    adv = oracle.group_advantages(ro.rewards, 8)
    w, r, chi = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, None, ro.mask)
    counts, share, total = oracle.omega_diagnostics(adv, r, ro.mask, w)
    assert counts[0] == (ro.mask == 0).sum() and counts[4] == ro.mask.size
    assert counts[1] == ro.mask[adv == 0].sum() and counts[2] > 0
    assert counts[3] == counts[0] + counts[1] + counts[2]
    assert counts[2] == ((chi == 0) & (ro.mask == 1) & (adv[:, None] != 0)).sum()
    aw = np.sort(np.abs(w).reshape(-1).astype(np.float64))[::-1]
    k = -(-aw.size // 10)
    assert share == pytest.approx(aw[:k].sum() / aw.sum(), rel=1e-9) and total == pytest.approx(aw.sum(), rel=1e-9)


def test_top_decile_closed_forms():
    n_rows, T = 4, 25
    adv, ratio, mask = np.ones(n_rows, np.float32), np.ones((n_rows, T), np.float32), np.ones((n_rows, T), np.uint8)
    _, share, _ = oracle.omega_diagnostics(adv, ratio, mask, np.full((n_rows, T), 0.5, np.float32))
    assert share == pytest.approx(0.1)                              # uniform coefficients: the decile carries 10 %
    w = np.zeros((n_rows, T), np.float32)
    w[2, 7] = -3.0
    _, share, total = oracle.omega_diagnostics(adv, ratio, mask, w)
    assert share == 1.0 and total == 3.0                            # one-hot
    _, share, total = oracle.omega_diagnostics(adv, ratio, mask, np.zeros((n_rows, T), np.float32))
    assert share == 0.0 and total == 0.0


def test_score_variants():
    ro = synth.rollout(4, 4, 8, 64, lengths="uniform", min_len=8)
    adv = oracle.group_advantages(ro.rewards, 8)
    N = ro.n_valid
    base, r, chi = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_old, ro.logp_ref, ro.mask, N_norm=N, beta=1e-3)
    w1, r1, c1 = oracle.grpo_coeffs_variant(adv, ro.logp_new, ro.logp_old, ro.logp_ref, ro.mask, N, 0.2, 1e-3, variant=1)
    assert np.array_equal(r, r1) and np.array_equal(chi, c1)
    kl = 1e-3 * ro.mask / N * (1 - np.exp(ro.logp_ref.astype(np.float64) - ro.logp_new))
    np.testing.assert_allclose(w1, -(ro.mask * adv[:, None].astype(np.float64)) / N + kl, rtol=1e-6, atol=1e-12)
    w2, _, _ = oracle.grpo_coeffs_variant(adv, ro.logp_new, ro.logp_old, ro.logp_ref, ro.mask, N, 0.2, 1e-3, variant=2)
    assert np.array_equal(w2, (ro.mask * adv[:, None]).astype(np.float32))
    w0, _, _ = oracle.grpo_coeffs_variant(adv, ro.logp_new, ro.logp_old, ro.logp_ref, ro.mask, N, 0.2, 1e-3, variant=0)
    assert np.array_equal(w0, base)
    # with s = s_old (ratio 1, nothing clipped) removing ratio/clipping changes nothing
    w_a, _, _ = oracle.grpo_coeffs(adv, ro.logp_new, ro.logp_new, None, ro.mask, N_norm=N)
    w_b, _, _ = oracle.grpo_coeffs_variant(adv, ro.logp_new, ro.logp_new, None, ro.mask, N, 0.2, 0.0, variant=1)
    assert np.array_equal(w_a, w_b)
