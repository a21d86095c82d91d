"""hilore_unit_exposure_static: the exposure reduction for callers that may not allocate (its partial
sums live in a fixed array inside the library).  Checked against hilore_unit_exposure, which takes the
scratch from the caller, and against the CPU oracle, on two calls in a row -- the second call finds the
first call's partial sums still in the shared array and must not be disturbed by them.  Collected last
on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def _case(seed, n_resp_groups, G_, T, U, lengths):
    ro = synth.rollout(seed, n_resp_groups, G_, T, rewards="uniform", lengths=lengths)
    rng = np.random.default_rng(seed + 100)
    omega = (rng.standard_normal((ro.n_resp, T)) * 1e-4).astype(np.float32) * ro.mask
    rms = (rng.random((U, ro.n_resp * T), dtype=np.float32) + np.float32(0.5))
    return omega, ro.mask, rms


def _static(omega, mask, rms, row_shift=0):
    n_rows, T = omega.shape
    U, ld = rms.shape
    E, sw = G.Guarded(U * 4), G.Guarded(4)
    api.hilore_unit_exposure_static(G.dev(omega), G.dev(mask), n_rows, T, G.dev(rms), U, ld, row_shift, 1e-8,
                                    E.ptr(), sw.ptr())
    return E.numpy(np.float32, (U,)), float(sw.numpy(np.float32, (1,))[0])


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    big = _case(0, 2, 8, 1024, 84, "uniform")        # 16 384 slots, 84 units: fills many scratch slots
    small = _case(1, 1, 4, 256, 3, "full")           # then a much smaller problem on the stale array
    for omega, mask, rms in (big, small, big):
        want_E, want_sw = G.unit_exposure(omega, mask, rms)
        got_E, got_sw = _static(omega, mask, rms)
        assert G.rel_err(got_E, want_E).max() <= RTOL
        assert abs(got_sw - want_sw) <= RTOL * abs(want_sw)
        oE, osw = oracle.unit_exposure(omega, mask, rms)       # and both against the oracle's definition
        assert G.rel_err(got_E, oE).max() <= RTOL and abs(got_sw - osw) <= RTOL * abs(osw)
    # the scalar path (row_shift = 1) goes through the same array
    omega, mask, rms = small
    mask = mask.copy()
    mask[:, 0] = 0
    want_E, _ = G.unit_exposure(omega, mask, rms, row_shift=1)
    got_E, _ = _static(omega, mask, rms, row_shift=1)
    assert G.rel_err(got_E, want_E).max() <= RTOL
    assert G.rel_err(got_E, oracle.unit_exposure(omega, mask, rms, row_shift=1)[0]).max() <= RTOL


def test_static_scratch_rejects_problems_beyond_its_size():
    cap = api.hilore_static_scratch_bytes()
    assert cap == 1 << 20
    U, n_rows, T = 255, 257, 1024                      # (U + 1) * 257 tiles * 16 bytes > 1 MiB
    assert api.hilore_workspace_bytes(U, n_rows * T) > cap
    a = torch.zeros(16, device="cuda")
    st = api.hilore_unit_exposure_static(a, a, n_rows, T, a, U, n_rows * T, 0, 1e-8, a, None, check=False)
    assert st == api.WORKSPACE
    assert "workspace" in api.status_string(st)
    U, n_rows = 255, 256                               # exactly at the limit is accepted by the size check
    assert api.hilore_workspace_bytes(U, n_rows * T) == cap
