"""Pins for the oracle's joint H/L/R allocator (the paper's two-constraint multiple-choice knapsack DP).

The DP is an algorithm; what it must reach has a plain definition -- the best assignment of the discretised
problem -- so it is checked against exhaustive enumeration of all 3^U assignments, against the feasibility
guarantee of upward rounding, and against the tie rules and boundary cases the paper states."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import ACT_H, ACT_L, ACT_R

ALLOWED = {ACT_H: (ACT_R, ACT_H, ACT_L), ACT_L: (ACT_R, ACT_L), ACT_R: (ACT_R,)}


def int_costs(psi, dmem, M_res, delta_b, N):
    """b_u(a) = ceil(dmem / h_B), r_u(a) = ceil(d / h_delta) (Eq. "allocation-integer-costs"), None if infeasible."""
    U = len(psi)
    out = {}
    for u in range(U):
        for a in (ACT_R, ACT_H, ACT_L):
            dm = 0.0 if a == ACT_R else max(0.0, float(dmem[u][a]))
            d = float(psi[u]) if a == ACT_L else 0.0
            if M_res > 0:
                b = math.ceil(dm / (M_res / N))
            else:
                b = 0 if dm == 0 else None
            if delta_b > 0:
                r = math.ceil(d / (delta_b / N)) if d >= 0 else None
            else:
                r = None if a == ACT_L else 0
            ok = b is not None and r is not None and b <= N and r <= N
            out[u, a] = (b, r) if ok else None
    return out


def brute_force(psi, dtau, dmem, avail, M_res, delta_b, N):
    """Best utility over all assignments that fit the integer budgets."""
    U = len(psi)
    c = int_costs(psi, dmem, M_res, delta_b, N)
    best = -math.inf
    for assign in itertools.product(*[ALLOWED[int(q)] for q in avail]):
        if any(c[u, a] is None for u, a in enumerate(assign)):
            continue
        if sum(c[u, a][0] for u, a in enumerate(assign)) > N or sum(c[u, a][1] for u, a in enumerate(assign)) > N:
            continue
        util = 0.0
        for u, a in enumerate(assign):       # same order of additions as the DP
            util += 0.0 if a == ACT_R else float(dtau[u][a])
        best = max(best, util)
    return best, c


def random_case(rng, U):
    psi = rng.uniform(0.0, 0.02, U).astype(np.float32)
    dtau = np.zeros((U, 3))
    dmem = np.zeros((U, 3))
    dmem[:, ACT_H] = rng.uniform(50, 600, U)
    dmem[:, ACT_L] = dmem[:, ACT_H] * 0.53
    dtau[:, ACT_H] = rng.uniform(-0.5, 4.0, U)          # some bundles do not pay
    dtau[:, ACT_L] = dtau[:, ACT_H] - rng.uniform(0.05, 0.8, U)
    avail = rng.choice([ACT_H, ACT_H, ACT_L, ACT_R], U).astype(np.uint8)
    return psi, dtau, dmem, avail


@pytest.mark.parametrize("N", [8, 37, 1024])
def test_dp_reaches_the_enumerated_optimum(N):
    rng = np.random.default_rng(N)
    for trial in range(40):
        U = int(rng.integers(1, 8))
        psi, dtau, dmem, avail = random_case(rng, U)
        M_res = float(rng.uniform(100, 1500))
        delta_b = float(rng.uniform(0.002, 0.05))
        action, totals = oracle.allocate(psi, dtau, dmem, avail, M_res, delta_b, N)
        best, c = brute_force(psi, dtau, dmem, avail, M_res, delta_b, N)
        # the returned assignment is valid ...
        for u, a in enumerate(action):
            assert int(a) in ALLOWED[int(avail[u])] and c[u, int(a)] is not None
        assert sum(c[u, int(a)][0] for u, a in enumerate(action)) <= N
        assert sum(c[u, int(a)][1] for u, a in enumerate(action)) <= N
        # ... optimal on the grid ...
        util = sum(0.0 if a == ACT_R else dtau[u][int(a)] for u, a in enumerate(action))
        assert util == pytest.approx(best, rel=1e-12, abs=1e-12) and totals[0] == pytest.approx(best, rel=1e-12, abs=1e-12)
        # ... and, costs being rounded up, feasible for the real budgets (Eq. "allocation-grid-feasibility")
        assert totals[1] <= M_res * (1 + 1e-12) and totals[2] <= delta_b * (1 + 1e-6)
        assert totals[1] == pytest.approx(sum(dmem[u][int(a)] for u, a in enumerate(action)))


def test_all_R_is_always_admitted_and_never_worse():
    rng = np.random.default_rng(1)
    psi, dtau, dmem, avail = random_case(rng, 6)
    dtau[:, 1:] = -1.0                                      # nothing pays: the zero-cost all-R assignment wins
    action, totals = oracle.allocate(psi, dtau, dmem, avail, 500.0, 0.01)
    assert action.tolist() == [ACT_R] * 6 and totals.tolist() == [0.0, 0.0, 0.0]


def test_boundary_cases():
    psi = np.array([0.001, 0.001, 0.0], np.float32)
    dtau = np.array([[0, 3.0, 2.0], [0, 3.0, 2.0], [0, 1.0, 0.5]])
    dmem = np.array([[0, 10.0, 5.0], [0, 0.0, 0.0], [0, 10.0, 0.0]])
    avail = [ACT_H, ACT_H, ACT_H]
    # zero residual memory: only actions without memory cost (unit 1: H; unit 2: L costs no memory, no risk)
    a, t = oracle.allocate(psi, dtau, dmem, avail, 0.0, 0.01)
    assert a.tolist() == [ACT_R, ACT_H, ACT_L] and t[1] == 0.0
    # zero risk budget disables L everywhere, even where psi is zero
    a, t = oracle.allocate(psi, dtau, dmem, avail, 100.0, 0.0)
    assert ACT_L not in a.tolist() and a.tolist() == [ACT_H, ACT_H, ACT_H]
    # both zero: only free H
    a, _ = oracle.allocate(psi, dtau, dmem, avail, 0.0, 0.0)
    assert a.tolist() == [ACT_R, ACT_H, ACT_R]
    # a NaN risk score makes L unavailable for that unit only
    psi2 = psi.copy()
    psi2[0] = np.nan
    dtau2 = dtau.copy()
    dtau2[0] = [0, -1.0, 2.0]
    a, _ = oracle.allocate(psi2, dtau2, dmem, avail, 100.0, 0.01)
    assert a[0] == ACT_R
    with pytest.raises(oracle.OracleError):
        oracle.allocate(psi, dtau, dmem, avail, -1.0, 0.01)


def test_tie_rules():
    # within a state: equal utilities are resolved in the order R, H, L
    psi = np.array([0.0], np.float32)
    a, _ = oracle.allocate(psi, [[0, 0.0, 0.0]], [[0, 1.0, 1.0]], [ACT_H], 10.0, 0.01)
    assert a.tolist() == [ACT_R]
    a, _ = oracle.allocate(psi, [[0, 1.0, 1.0]], [[0, 1.0, 1.0]], [ACT_H], 10.0, 0.01)
    assert a.tolist() == [ACT_H]
    # terminal ties favour lower risk, then lower memory: H (no risk, more memory) beats L (risk, less memory)
    psi = np.array([0.005], np.float32)
    a, _ = oracle.allocate(psi, [[0, 2.0, 2.0]], [[0, 8.0, 4.0]], [ACT_H], 10.0, 0.01)
    assert a.tolist() == [ACT_H]
    # with equal risk (both zero) the lower memory state wins: two units, either may take the single H slot's
    # utility through different memory use
    psi = np.array([0.0, 0.0], np.float32)
    dtau = [[0, 2.0, 0.0], [0, 2.0, 0.0]]
    dmem = [[0, 6.0, 0.0], [0, 3.0, 0.0]]
    a, t = oracle.allocate(psi, dtau, dmem, [ACT_H, ACT_H], 8.0, 0.01)      # only one of the two fits
    assert a.tolist() == [ACT_R, ACT_H] and t[1] == 3.0


def test_conservative_rounding_can_refuse_a_tight_fit():
    """Costs are rounded up to the grid: two bundles of 5.004 each do not fit a budget of 10.008 on a coarse grid
    although they fit exactly -- feasibility is preserved, optimality is on the grid."""
    psi = np.zeros(2, np.float32)
    dtau = [[0, 1.0, 0.0]] * 2
    dmem = [[0, 5.004, 0.0]] * 2
    a, _ = oracle.allocate(psi, dtau, dmem, [ACT_H, ACT_H], 10.008, 0.01, N=1024)
    assert sorted(a.tolist()) == [ACT_R, ACT_H] or a.tolist() == [ACT_H, ACT_H]
    a, _ = oracle.allocate(psi, dtau, dmem, [ACT_H, ACT_H], 10.008, 0.01, N=3)   # step 3.336: each costs 2 of 3
    assert sorted(a.tolist()) == [ACT_R, ACT_H]


def test_risk_budget_split():
    assert oracle.risk_budget(0.02, 4096, 16384) == pytest.approx(0.005)
    assert oracle.risk_budget(0.02, 1, 0) == 0.0
    parts = [oracle.risk_budget(0.02, n, 1000) for n in (100, 400, 500)]
    assert sum(parts) == pytest.approx(0.02)
