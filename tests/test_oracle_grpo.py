"""Pins for the oracle's GRPO quantities (advantages, ratio, clip indicator, omega).

Every check here compares the oracle with something the paper or the mathematics fixes:
hand-worked values (tests/golden/grpo_hand_worked.txt), the Bernoulli closed form of the
group statistics, the exact-zero rule for equal-reward groups, central finite differences
of the printed objective (Prop. 1: omega = dL/ds), the r = 1 special case of the setup
paragraph, and the invariants of Remark 1.
"""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "grpo_hand_worked.txt")


def _golden(kind):
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = [x.strip() for x in line.split("|")]
        if f[0] == kind:
            out.append(f[1:])
    return out


@pytest.mark.parametrize("rewards,expected", _golden("advantage"))
def test_advantage_hand_worked(rewards, expected):
    R = np.array([float(x) for x in rewards.split(",")], np.float32)
    want = np.array([float(x) for x in expected.split(",")])
    got = oracle.group_advantages(R, G=len(R))
    np.testing.assert_allclose(got.astype(np.float64), want, rtol=2e-7, atol=0)


@pytest.mark.parametrize("G", [2, 8, 16])
def test_advantage_bernoulli_closed_form(G):
    # k successes of G: mean p = k/G, population std sqrt(p(1-p)); success (1-p)/(std+eps), failure -p/(std+eps)
    for k in range(G + 1):
        R = np.zeros(G, np.float32)
        R[:k] = 1.0
        R = np.roll(R, 3)
        got = oracle.group_advantages(R, G).astype(np.float64)
        p = k / G
        if k in (0, G):
            assert np.all(got == 0.0)
            continue
        den = math.sqrt(p * (1 - p)) + 1e-6
        want = np.where(R > 0, (1 - p) / den, -p / den)
        np.testing.assert_allclose(got, want, rtol=2e-7)


def test_advantage_equal_rewards_exactly_zero():
    # 0.7 is not a dyadic rational: a naive fp32 mean of eight copies differs from 0.7f.
    for val in (0.7, 0.1, 1.0, -3.3, 0.0):
        for G in (1, 2, 8, 16):
            got = oracle.group_advantages(np.full(G * 3, val, np.float32), G)
            assert got.tobytes() == np.zeros(G * 3, np.float32).tobytes()


def test_advantage_invariants_random_groups():
    rng = np.random.default_rng(1)
    G = 8
    R = rng.random(G * 200, dtype=np.float32)
    A = oracle.group_advantages(R, G).astype(np.float64).reshape(-1, G)
    Rg = R.astype(np.float64).reshape(-1, G)
    sigma = Rg.std(axis=1)
    np.testing.assert_allclose(A.sum(axis=1), 0.0, atol=2e-6)
    np.testing.assert_allclose(A.var(axis=1), (sigma / (sigma + 1e-6)) ** 2, rtol=1e-6)
    # advantages are an increasing affine function of the rewards inside a group
    assert np.all(np.argsort(A, axis=1, kind="stable") == np.argsort(Rg, axis=1, kind="stable"))
    # groups are independent and consecutive: shuffling other groups does not change group 5
    R2 = R.copy()
    R2[: 5 * G] = rng.random(5 * G, dtype=np.float32)
    A2 = oracle.group_advantages(R2, G).reshape(-1, G)
    assert np.array_equal(A2[5:], A.astype(np.float32)[5:])


def test_advantage_shape_errors():
    with pytest.raises(oracle.OracleError) as e:
        oracle.group_advantages(np.zeros(7, np.float32), 4)
    assert e.value.status == oracle.SHAPE


@pytest.mark.parametrize("A,r,m,beta,d,chi,omega", _golden("coeff"))
def test_coeff_hand_worked(A, r, m, beta, d, chi, omega):
    A, r, beta, d, omega = float(A), float(r), float(beta), float(d), float(omega)
    m, chi = int(m), int(chi)
    N = 4
    s_new = np.array([[-1.0]], np.float32)
    s_old = (s_new.astype(np.float64) - math.log(r)).astype(np.float32)
    s_ref = (s_new.astype(np.float64) + d).astype(np.float32)
    mask = np.array([[m]], np.uint8)
    w, rr, c = oracle.grpo_coeffs(np.array([A], np.float32), s_new, s_old, s_ref, mask, N_norm=N, clip_eps=0.2,
                                  beta=beta)
    assert int(c[0, 0]) == chi
    assert rr[0, 0] == pytest.approx(r, rel=2e-7)
    assert float(w[0, 0]) == pytest.approx(omega, rel=3e-7, abs=1e-12)


def _random_case(seed, n_rows=6, T=40, G=3, beta=0.0, spread=0.15):
    rng = np.random.default_rng(seed)
    R = rng.random(n_rows, dtype=np.float32)
    adv = oracle.group_advantages(R, G)
    s = (rng.standard_normal((n_rows, T)) * 0.5 - 1.5).astype(np.float32)
    s_old = (s + rng.standard_normal((n_rows, T)).astype(np.float32) * np.float32(spread)).astype(np.float32)
    s_ref = (s + rng.standard_normal((n_rows, T)).astype(np.float32) * np.float32(0.05)).astype(np.float32)
    mask = (rng.random((n_rows, T)) < 0.8).astype(np.uint8)
    return adv, s, s_old, s_ref, mask


@pytest.mark.parametrize("beta", [0.0, 1e-3, 0.5])
def test_coeff_is_derivative_of_objective(beta):
    """Prop. 1: omega_t = dL/ds_t.  Central differences of the printed objective, in fp64."""
    adv, s, s_old, s_ref, mask = _random_case(3, beta=beta)
    N = int(mask.sum())
    w, r, chi = oracle.grpo_coeffs(adv, s, s_old, s_ref, mask, N_norm=N, clip_eps=0.2, beta=beta)
    assert (chi == 0).any() and (chi == 1).any()          # both branches are exercised
    s64 = s.astype(np.float64)
    h = 1e-6
    checked = 0
    for i in range(s.shape[0]):
        for t in range(s.shape[1]):
            if min(abs(r[i, t] - 1.2), abs(r[i, t] - 0.8)) < 1e-3:
                continue                                  # the derivative is not defined at the kink
            sp, sm = s64.copy(), s64.copy()
            sp[i, t] += h
            sm[i, t] -= h
            fd = (oracle.grpo_objective(adv, sp, s_old, s_ref, mask, N, 0.2, beta)
                  - oracle.grpo_objective(adv, sm, s_old, s_ref, mask, N, 0.2, beta)) / (2 * h)
            assert fd == pytest.approx(float(w[i, t]), rel=2e-5, abs=2e-9), (i, t)
            checked += 1
    assert checked > 200


def test_coeff_ratio_one_special_case():
    """With s = s_old the ratio is 1, clipping is inactive and omega = -m A / N."""
    adv, s, _, s_ref, mask = _random_case(4)
    N = 1234
    w, r, chi = oracle.grpo_coeffs(adv, s, s.copy(), None, mask, N_norm=N)
    assert np.all(r == 1.0) and np.all(chi == 1)
    want = -(mask.astype(np.float64) * adv.astype(np.float64)[:, None]) / N
    np.testing.assert_allclose(w, want, rtol=1e-7, atol=0)


def test_coeff_remark1_zero_contributions():
    """beta = 0: masked slots, zero-advantage rows and flat clipped branches have omega = 0."""
    adv, s, s_old, s_ref, mask = _random_case(5, spread=0.3)
    adv[1] = 0.0
    w, r, chi = oracle.grpo_coeffs(adv, s, s_old, None, mask)
    assert np.all(w[mask == 0] == 0.0)
    assert np.all(w[1] == 0.0)
    assert np.all(w[chi == 0] == 0.0)
    live = (mask == 1) & (chi == 1) & (adv[:, None] != 0)
    assert np.all(w[live] != 0.0)
    # with K3 regularisation unmasked zero-advantage slots keep a contribution, masked ones stay zero
    w2, _, _ = oracle.grpo_coeffs(adv, s, s_old, s_ref, mask, beta=1e-3)
    assert np.all(w2[mask == 0] == 0.0)
    assert np.any(w2[1][mask[1] == 1] != 0.0)


def test_coeff_clip_indicator_definition():
    """chi against the printed indicator evaluated independently, incl. the inclusive boundaries."""
    hi, lo = np.float32(1.0) + np.float32(0.2), np.float32(1.0) - np.float32(0.2)
    # ratios exactly on the fp32 boundaries: pick s - s_old = 0 and patch r through eps
    adv = np.array([1.0, -1.0], np.float32)
    s = np.zeros((2, 3), np.float32)
    s_old = -np.log(np.array([[1.0, float(hi) * 1.001, float(lo) * 0.999]] * 2)).astype(np.float32)
    mask = np.ones((2, 3), np.uint8)
    _, r, chi = oracle.grpo_coeffs(adv, s, s_old, None, mask)
    want = np.stack([(r[0] <= hi), (r[1] >= lo)]).astype(np.uint8)
    assert np.array_equal(chi, want)
    assert chi.tolist() == [[1, 0, 1], [1, 1, 0]]


def test_coeff_normaliser():
    adv, s, s_old, _, mask = _random_case(6)
    w_auto, _, _ = oracle.grpo_coeffs(adv, s, s_old, None, mask, N_norm=0)
    w_n, _, _ = oracle.grpo_coeffs(adv, s, s_old, None, mask, N_norm=int(mask.sum()))
    assert np.array_equal(w_auto, w_n)
    w_2n, _, _ = oracle.grpo_coeffs(adv, s, s_old, None, mask, N_norm=2 * int(mask.sum()))
    np.testing.assert_allclose(w_2n * 2, w_n, rtol=2e-7)
    with pytest.raises(oracle.OracleError) as e:
        oracle.grpo_coeffs(adv, s, s_old, None, np.zeros_like(mask))
    assert e.value.status == oracle.ZERO_NORM
