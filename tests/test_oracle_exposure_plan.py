"""Pins for the oracle's token weights, update exposure, risk score and H/L/R gating."""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import ACT_H, ACT_L, ACT_R


def bf16_bits(x):
    return torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_row_rms_hand_values():
    x = bf16_bits([[3, 4, 0, 0], [1, 1, 1, 1], [0, 0, 0, 0], [-2, 2, -2, 2]])
    got = oracle.row_rms(x)
    np.testing.assert_allclose(got, [2.5, 1.0, 0.0, 2.0], rtol=1e-7)
    # leading dimension: trailing padding is ignored
    wide = np.concatenate([x, np.full((4, 4), 0x7FC0, np.uint16)], axis=1)
    assert np.array_equal(oracle.row_rms(wide, cols=4), got)


def test_row_rms_against_numpy_fp64():
    rng = np.random.default_rng(0)
    x = bf16_bits(rng.standard_normal((37, 896)) * 3)
    xf = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    np.testing.assert_allclose(oracle.row_rms(x), np.sqrt((xf ** 2).mean(axis=1)), rtol=1e-7)


def _case(seed, n_rows=4, T=50, U=3):
    rng = np.random.default_rng(seed)
    omega = (rng.standard_normal((n_rows, T)) * 1e-4).astype(np.float32)
    lengths = rng.integers(5, T + 1, n_rows)
    mask = (np.arange(T)[None, :] < lengths[:, None]).astype(np.uint8)
    omega[mask == 0] = 0
    rms = (rng.random((U, n_rows * T)) + 0.5).astype(np.float32)
    return omega, mask, rms


def test_exposure_hand_example():
    """4 valid tokens, 2 units, by hand.  a = (1,2,3,2) -> mean 2 -> alpha = (.5,1,1.5,1)."""
    omega = np.array([[0.1, -0.2, 0.3, 0.4, 9.0]], np.float32)
    mask = np.array([[1, 1, 1, 1, 0]], np.uint8)
    rms = np.array([[1, 2, 3, 2, 100], [5, 5, 5, 5, 0]], np.float32)
    E, sw = oracle.unit_exposure(omega, mask, rms)
    assert sw == pytest.approx(1.0, rel=1e-6)
    assert E[0] == pytest.approx(0.1 * 0.5 + 0.2 * 1 + 0.3 * 1.5 + 0.4 * 1, rel=1e-6)
    assert E[1] == pytest.approx(1.0, rel=1e-6)              # equal rows: alpha = 1, E = sum |omega|


def test_exposure_weights_have_mean_one():
    """Constant |omega| = c gives E = c |T_b| because the weights average to one over T_b."""
    omega, mask, rms = _case(1)
    c = np.float32(3e-5)
    om = np.where(mask == 1, c, 0).astype(np.float32) * np.where(np.arange(omega.size).reshape(omega.shape) % 2, -1, 1).astype(np.float32)
    E, sw = oracle.unit_exposure(om, mask, rms)
    np.testing.assert_allclose(E, float(c) * int(mask.sum()), rtol=1e-6)


def test_exposure_scale_invariance_and_cor1():
    omega, mask, rms = _case(2)
    E1, _ = oracle.unit_exposure(omega, mask, rms)
    E2, _ = oracle.unit_exposure(omega, mask, (rms * np.float32(64.0)).astype(np.float32))
    np.testing.assert_allclose(E1, E2, rtol=1e-6)             # the unit's overall activation scale drops out
    E0, sw0 = oracle.unit_exposure(np.zeros_like(omega), mask, rms)
    assert np.all(E0 == 0) and sw0 == 0                        # all coefficients zero => zero exposure
    En, _ = oracle.unit_exposure(omega, np.zeros_like(mask), rms)
    assert np.all(En == 0)                                     # empty T_b: no division


def test_exposure_ignores_padded_rows_and_matches_numpy():
    omega, mask, rms = _case(3)
    rms2 = rms.copy()
    rms2[:, mask.reshape(-1) == 0] = 1e6                        # garbage at padded slots
    om2 = omega.copy()
    om2[mask == 0] = 7.0
    E1, _ = oracle.unit_exposure(omega, mask, rms)
    E2, _ = oracle.unit_exposure(om2, mask, rms2)
    assert np.array_equal(E1, E2)
    m = mask.reshape(-1).astype(bool)
    a = rms.astype(np.float64)[:, m]
    alpha = (a + 1e-8) / (a.mean(axis=1, keepdims=True) + 1e-8)
    np.testing.assert_allclose(alpha.mean(axis=1), 1.0, rtol=1e-12)
    want = (np.abs(omega.astype(np.float64)).reshape(-1)[m][None, :] * alpha).sum(axis=1)
    np.testing.assert_allclose(E1, want, rtol=2e-7)


def test_exposure_row_shift_uses_previous_position():
    omega, mask, rms = _case(4)
    mask[:, 0] = 0
    omega[:, 0] = 0
    n_rows, T = omega.shape
    shifted = np.roll(rms.reshape(rms.shape[0], n_rows, T), 1, axis=2).reshape(rms.shape[0], -1).copy()
    E_shift, _ = oracle.unit_exposure(omega, mask, rms, row_shift=1)
    E_ref, _ = oracle.unit_exposure(omega, mask, shifted, row_shift=0)
    np.testing.assert_allclose(E_shift, E_ref, rtol=1e-7)


def test_exposure_row_shift_weights_average_to_one_over_the_slots_that_have_a_row():
    """row_shift = 1 with the first slot of every response valid: that slot has no source row inside the grid and
    carries no weight; over the remaining slots of T_b the weights average to one (Eq. activation-token-weights), so
    constant |omega| = c gives E = c * (number of valid slots with t >= 1), whatever the activation magnitudes; and
    the result equals the exposure of the same record with the first column masked out."""
    omega, mask, rms = _case(7)
    mask[:, 0] = 1
    n_rows, T = omega.shape
    c = np.float32(3e-4)
    const = np.where(mask != 0, c, 0).astype(np.float32)
    E, sw = oracle.unit_exposure(const, mask, rms, row_shift=1, eps_alpha=0.0)
    with_row = int(mask[:, 1:].sum())
    np.testing.assert_allclose(E, np.float64(c) * with_row, rtol=1e-6)
    assert sw == pytest.approx(float(c) * int(mask.sum()), rel=1e-6)          # sum |omega| is over all of T_b
    mask2 = mask.copy()
    mask2[:, 0] = 0
    E_a, _ = oracle.unit_exposure(omega * (mask != 0), mask, rms, row_shift=1)
    E_b, _ = oracle.unit_exposure(omega * (mask2 != 0), mask2, rms, row_shift=1)
    np.testing.assert_allclose(E_a, E_b, rtol=1e-6)


def _avail_table():
    """Eq. "available-recovery-actions": q = H -> {H, L, R}; q = L -> {L, R}; q = R -> {R}."""
    return {ACT_H: {ACT_H, ACT_L, ACT_R}, ACT_L: {ACT_L, ACT_R}, ACT_R: {ACT_R}}


def test_plan_availability_table_exhaustive():
    tbl = _avail_table()
    for want, q in itertools.product((ACT_R, ACT_H, ACT_L), repeat=2):
        a, _, rec, ret = oracle.plan(None, None, None, 0.0, 0.0, [q], [128], [256], [1], [64], action_in=[want])
        expect = want if want in tbl[q] else ACT_R
        assert a[0] == expect and rec[0] == (expect == ACT_R)
        bytes_ = {ACT_H: 128 * 256 * 2, ACT_L: 128 * 256 + 4 * 128 * 256 // 64, ACT_R: 0}[expect]
        assert ret[0] == bytes_
    a, _, _, ret = oracle.plan(None, None, None, 0, 0, [ACT_H], [128], [256], [0], [0], action_in=[ACT_L])
    assert ret[0] == 128 * 256                                  # unscaled format stores no scales


def test_plan_threshold_example():
    E = np.array([1, 2, 3, 4, 5, 6, 7, 8, 9, 10], np.float32)
    kappa = np.full(10, 0.5, np.float32)
    ebar = np.full(10, 0.02, np.float32)
    psi_want = (kappa * E) * ebar
    avail = [ACT_H] * 10
    avail[0] = ACT_R        # wants L, only R available
    avail[9] = ACT_L        # wants H, only L/R available -> R
    avail[8] = ACT_L
    a, psi, rec, ret = oracle.plan(E, kappa, ebar, 0.045, 0.075, avail, [8] * 10, [64] * 10, [1] * 10, [64] * 10)
    assert np.array_equal(psi, psi_want)
    # psi = .01 .02 .03 .04 | .05 .06 .07 | .08 .09 .10  -> L L L L R R R H H H before availability
    assert a.tolist() == [ACT_R, ACT_L, ACT_L, ACT_L, ACT_R, ACT_R, ACT_R, ACT_H, ACT_R, ACT_R]
    assert rec.tolist() == [1, 0, 0, 0, 1, 1, 1, 0, 1, 1]
    assert ret.tolist() == [0, 544, 544, 544, 0, 0, 0, 1024, 0, 0]
    # NaN risk falls to R (exact and always available)
    E[3] = np.nan
    a, *_ = oracle.plan(E, kappa, ebar, 0.045, 0.075, avail, [8] * 10, [64] * 10, [1] * 10, [64] * 10)
    assert a[3] == ACT_R


def test_fit_kappa_closed_form_against_grid_search():
    """kappa = argmin_{kappa >= 0} sum (y - kappa x)^2 (Eq. "susceptibility")."""
    rng = np.random.default_rng(0)
    x = rng.uniform(0, 1, 50)
    assert oracle.fit_kappa(x, 2.5 * x) == pytest.approx(2.5, rel=1e-12)      # exact line
    assert oracle.fit_kappa(x, -3 * x) == 0.0                                 # constrained at zero
    assert oracle.fit_kappa(np.zeros(4), np.ones(4)) == 0.0                   # no signal
    y = 1.7 * x + rng.normal(0, 0.1, 50)
    k = oracle.fit_kappa(x, y)
    grid = np.linspace(0, 4, 40001)
    loss = ((y[None, :] - grid[:, None] * x[None, :]) ** 2).sum(axis=1)
    assert k == pytest.approx(grid[loss.argmin()], abs=2e-4)
