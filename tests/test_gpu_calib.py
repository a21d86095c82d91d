"""Parity of the calibration statistics with the oracle: e^L of the codec round trip (1e-6 relative: fp32 per
16 elements, fp64 beyond), the susceptibility fit (host arithmetic, exact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def rel_error_gpu(x_bits, xh_bits, cols=None):
    rows, ld = x_bits.shape
    cols = ld if cols is None else cols
    nws = api.hilore_relative_error_workspace_bytes()
    ws, e, n2 = G.Guarded(nws), G.Guarded(8), G.Guarded(16)
    api.hilore_relative_error(G.dev(x_bits), G.dev(xh_bits), rows, cols, ld, xh_bits.shape[1], e.ptr(), n2.ptr(), ws.ptr(), nws)
    ws.numpy(np.uint8, (nws,))
    return float(e.numpy(np.float64, (1,))[0]), n2.numpy(np.float64, (2,))


@pytest.mark.parametrize("fmt", [api.FMT_E4M3FN_RAW, api.FMT_E4M3FN_BLK, api.FMT_INT8_BLK])
@pytest.mark.parametrize("rows,cols", [(8192, 896), (37, 4096), (1, 64), (300, 1536)])
def test_relative_error_of_the_round_trip(fmt, rows, cols):
    x = synth.activation_unit(np.random.default_rng(rows + cols), rows, cols)
    codes, scales, _ = G.compress(x, fmt)
    xh = G.recover(codes, scales, fmt)
    e, n2 = rel_error_gpu(x, xh)
    want = oracle.relative_error(x, xh)
    assert e == pytest.approx(want, rel=1e-6)
    xf = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert n2[1] == pytest.approx((xf ** 2).sum(), rel=1e-6)
    a, _ = rel_error_gpu(x, xh)
    assert a == e                                              # fixed reduction order


def test_relative_error_expected_sizes_and_leading_dimension():
    """On N(0,1) data: unscaled E4M3FN about 0.027, block-scaled about 0.025, INT8 about 0.006-0.03 (outliers)."""
    rng = np.random.default_rng(0)
    x = synth._to_bf16_bits(rng.standard_normal((512, 1024), dtype=np.float32))
    got = {}
    for fmt in (api.FMT_E4M3FN_RAW, api.FMT_E4M3FN_BLK, api.FMT_INT8_BLK):
        codes, scales, _ = G.compress(x, fmt)
        got[fmt] = rel_error_gpu(x, G.recover(codes, scales, fmt))[0]
    assert 0.02 < got[api.FMT_E4M3FN_RAW] < 0.035 and 0.02 < got[api.FMT_E4M3FN_BLK] < 0.03 and got[api.FMT_INT8_BLK] < 0.012
    wide = np.full((512, 1088), 0x7FC0, np.uint16)
    wide[:, :1024] = x
    codes, scales, _ = G.compress(x, api.FMT_E4M3FN_BLK)
    xh = G.recover(codes, scales, api.FMT_E4M3FN_BLK)
    assert rel_error_gpu(wide, xh, cols=1024)[0] == pytest.approx(got[api.FMT_E4M3FN_BLK], rel=1e-9)
    assert rel_error_gpu(x, x)[0] == 0.0
    z = np.zeros((4, 64), np.uint16)
    assert rel_error_gpu(z, z)[0] == 0.0                      # 0 / (0 + 1e-8)


def test_fit_kappa_matches_oracle():
    rng = np.random.default_rng(1)
    x = rng.uniform(0, 1e-3, 16)
    y = 2.2 * x + rng.normal(0, 1e-4, 16)
    assert api.hilore_fit_kappa(x, y) == oracle.fit_kappa(x, y)
    assert api.hilore_fit_kappa(x, -y) == 0.0 and api.hilore_fit_kappa([0.0, 0.0], [1.0, 2.0]) == 0.0


def test_calibration_chain_on_one_unit_class():
    """ebar^L over four calibration microbatches and kappa from synthetic targets y = 1.8 x."""
    rng = np.random.default_rng(2)
    e, xs = [], []
    for b in range(4):
        x = synth.activation_unit(rng, 1024, 896)
        codes, scales, _ = G.compress(x, api.FMT_E4M3FN_RAW)
        e.append(rel_error_gpu(x, G.recover(codes, scales, api.FMT_E4M3FN_RAW))[0])
        xs.append(e[-1] * rng.uniform(0.1, 0.3))                 # x_{u,b} = exposure * e^L
    ebar = float(np.mean(e))
    assert 0.02 < ebar < 0.05
    assert api.hilore_fit_kappa(xs, [1.8 * v for v in xs]) == pytest.approx(1.8, rel=1e-12)
