"""Parity of hilore_allocate (the paper's knapsack DP, on the device) with the CPU oracle: the selected
actions are compared bit for bit (same candidates order, same tie rules, same fp64 additions), on small
grids where ties are frequent and on the paper's 1025 x 1025 grid with U up to 84."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
R, H, L = api.ACT_R, api.ACT_H, api.ACT_L


def run(psi, dtau, dmem, avail, M_res, delta_b, N=1024, check=True):
    U = len(psi)
    nws = api.hilore_allocate_workspace_bytes(U, N)
    ws = G.Guarded(nws)
    act, rec, tot = G.Guarded(max(U, 1)), G.Guarded(max(U, 1)), G.Guarded(24)
    d = lambda a, t: torch.from_numpy(np.ascontiguousarray(a, t)).cuda()
    st = api.hilore_allocate(U, d(psi, np.float32), d(dtau, np.float64), d(dmem, np.float64), d(avail, np.uint8), M_res, delta_b,
                             N, act.ptr(), rec.ptr(), tot.ptr(), ws.ptr(), nws, check=check)
    if st != api.OK:
        return st
    ws.numpy(np.uint8, (nws,))
    return act.numpy(np.uint8, (max(U, 1),))[:U], rec.numpy(np.uint8, (max(U, 1),))[:U], tot.numpy(np.float64, (3,))


def case(rng, U, quantised=False):
    psi = rng.uniform(0.0, 0.004, U).astype(np.float32)
    dtau = np.zeros((U, 3))
    dmem = np.zeros((U, 3))
    dmem[:, H] = rng.uniform(20, 600, U)
    dmem[:, L] = dmem[:, H] * 0.53
    dtau[:, H] = rng.uniform(-0.5, 4.0, U)
    dtau[:, L] = dtau[:, H] - rng.uniform(0.05, 0.8, U)
    if quantised:                       # few distinct values: many exact ties
        dtau = np.round(dtau * 2) / 2
        dmem = np.round(dmem / 100) * 100
        psi = (np.round(psi * 1000) / 1000).astype(np.float32)
    avail = rng.choice([H, H, L, R], U).astype(np.uint8)
    return psi, dtau, dmem, avail


@pytest.mark.parametrize("N", [4, 16, 61])
def test_small_grids_with_ties(N):
    rng = np.random.default_rng(N)
    for _ in range(25):
        U = int(rng.integers(1, 12))
        psi, dtau, dmem, avail = case(rng, U, quantised=True)
        M_res, delta_b = float(rng.choice([300, 800, 1500])), float(rng.choice([0.002, 0.01]))
        a, rec, tot = run(psi, dtau, dmem, avail, M_res, delta_b, N)
        oa, otot = oracle.allocate(psi, dtau, dmem, avail, M_res, delta_b, N)
        assert np.array_equal(a, oa) and np.array_equal(rec, (oa == R).astype(np.uint8))
        assert tot.tolist() == otot.tolist()


@pytest.mark.parametrize("U", [1, 7, 36, 84])
def test_paper_grid(U):
    """N_B = N_delta = 1024 (1025 states per axis); U = 36 is the paper's Qwen2.5-3B case, 84 the benchmark's."""
    rng = np.random.default_rng(U)
    psi, dtau, dmem, avail = case(rng, U)
    M_res = float(dmem[:, H].sum() * 0.35)
    delta_b = float(psi.sum() * 0.3)
    a, rec, tot = run(psi, dtau, dmem, avail, M_res, delta_b)
    oa, otot = oracle.allocate(psi, dtau, dmem, avail, M_res, delta_b)
    assert np.array_equal(a, oa)
    assert tot.tolist() == otot.tolist()
    assert tot[1] <= M_res and tot[2] <= delta_b * (1 + 1e-6)            # upward rounding keeps the real budgets
    assert len(set(a.tolist())) >= (2 if U > 1 else 1)


def test_boundary_cases_and_errors():
    psi = np.array([0.001, 0.001, 0.0], np.float32)
    dtau = np.array([[0, 3.0, 2.0], [0, 3.0, 2.0], [0, 1.0, 0.5]])
    dmem = np.array([[0, 10.0, 5.0], [0, 0.0, 0.0], [0, 10.0, 0.0]])
    avail = [H, H, H]
    for M_res, delta_b in ((0.0, 0.01), (100.0, 0.0), (0.0, 0.0), (100.0, 0.01)):
        a, _, tot = run(psi, dtau, dmem, avail, M_res, delta_b)
        oa, otot = oracle.allocate(psi, dtau, dmem, avail, M_res, delta_b)
        assert np.array_equal(a, oa) and tot.tolist() == otot.tolist()
    psi2 = psi.copy()
    psi2[0] = np.nan
    a, _, _ = run(psi2, dtau, dmem, avail, 100.0, 0.01)
    oa, _ = oracle.allocate(psi2, dtau, dmem, avail, 100.0, 0.01)
    assert np.array_equal(a, oa)
    assert run(psi, dtau, dmem, avail, -1.0, 0.01, check=False) == api.INVALID_ARG
    assert run(psi, dtau, dmem, avail, 1.0, float("nan"), check=False) == api.INVALID_ARG
    d = torch.zeros(64, device="cuda", dtype=torch.float64)
    assert api.hilore_allocate(3, d, d, d, d, 1.0, 1.0, 1024, d, None, None, d, 1024, check=False) == api.WORKSPACE
    assert api.hilore_risk_budget(0.02, 4096, 16384) == pytest.approx(0.005)


def test_allocate_consumes_device_side_risk_scores():
    """psi written by hilore_plan_apply(DECIDE) feeds hilore_allocate without leaving the device; the chosen
    actions then gate the batched recover through hilore_plan_apply."""
    rng = np.random.default_rng(3)
    U = 6
    units = [dict(rows=64, cols=128, fmt=api.FMT_E4M3FN_BLK, block=64) for _ in range(U)]
    udev, uhost = api.make_unit_table(units)
    exposure = torch.from_numpy(rng.uniform(0.05, 0.3, U).astype(np.float32)).cuda()
    kappa = torch.ones(U, device="cuda")
    ebar = torch.full((U,), 0.025, device="cuda")
    avail = torch.full((U,), H, dtype=torch.uint8, device="cuda")
    action = torch.zeros(U, dtype=torch.uint8, device="cuda")
    psi = torch.zeros(U, device="cuda")
    api.hilore_plan_apply(udev, uhost, U, api.PHASE_DECIDE, exposure, kappa, ebar, 0.0, float("inf"), avail, action, psi,
                          None, None)
    dtau = np.tile(np.array([0.0, 2.0, 1.5]), (U, 1))
    dmem = np.tile(np.array([0.0, 16384.0, 8704.0]), (U, 1))
    # the oracle's own psi from the host inputs; the device's must be the same bits
    _, o_psi, _, _ = oracle.plan(exposure.cpu().numpy(), np.ones(U, np.float32), np.full(U, 0.025, np.float32), 0.0,
                                 float("inf"), [H] * U, [64] * U, [128] * U, [1] * U, [64] * U)
    assert np.array_equal(psi.cpu().numpy().view(np.uint32), o_psi.view(np.uint32))
    M_res, delta_b = 3.2 * 16384, float(o_psi.astype(np.float64).sum() * 0.5)
    nws = api.hilore_allocate_workspace_bytes(U, 1024)
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    api.hilore_allocate(U, psi, torch.from_numpy(dtau).cuda(), torch.from_numpy(dmem).cuda(), avail, M_res, delta_b, 1024,
                        action, None, None, ws, nws)
    oa, _ = oracle.allocate(o_psi, dtau, dmem, np.full(U, H, np.uint8), M_res, delta_b)
    assert np.array_equal(action.cpu().numpy(), oa)
    assert (oa == L).sum() >= 1 and (oa == H).sum() >= 1
