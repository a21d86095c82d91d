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
    o_codes, o_scales = oracle.compress(x, fmt)[:2]           # the oracle's own round trip
    want = oracle.relative_error(x, oracle.recover(o_codes, o_scales, fmt))
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


def codec_rel_error_gpu(x_bits, fmt, cols=None):
    rows, ld = x_bits.shape
    cols = ld if cols is None else cols
    nws = api.hilore_relative_error_workspace_bytes()
    ws, e, n2 = G.Guarded(nws), G.Guarded(8), G.Guarded(16)
    api.hilore_codec_relative_error(G.dev(x_bits), rows, cols, ld, fmt, 0 if fmt == api.FMT_E4M3FN_RAW else 64, e.ptr(),
                                    n2.ptr(), ws.ptr(), nws)
    ws.numpy(np.uint8, (nws,))
    return float(e.numpy(np.float64, (1,))[0]), n2.numpy(np.float64, (2,))


@pytest.mark.parametrize("fmt", [api.FMT_E4M3FN_RAW, api.FMT_E4M3FN_BLK, api.FMT_INT8_BLK])
@pytest.mark.parametrize("rows,cols,ld", [(8192, 896, 896), (37, 4096, 4096), (1, 64, 64), (300, 1536, 1600), (5, 262144, 262144)])
def test_fused_relative_error_equals_the_round_trip(fmt, rows, cols, ld):
    """e^L computed in registers while encoding = e^L of compress -> recover -> compare, and the oracle's."""
    x = np.zeros((rows, ld), np.uint16)
    x[:, :cols] = synth.activation_unit(np.random.default_rng(rows + cols + fmt), rows, cols)
    e, n2 = codec_rel_error_gpu(x, fmt, cols=cols)
    codes, scales, _ = G.compress(x, fmt, cols=cols)
    xh = G.recover(codes, scales, fmt)
    e2, n22 = rel_error_gpu(x, xh, cols=cols)
    assert e == pytest.approx(e2, rel=1e-12) and np.allclose(n2, n22, rtol=1e-12, atol=0)
    oc, osc = oracle.compress(np.ascontiguousarray(x[:, :cols]), fmt)[:2]
    oxh = oracle.recover(oc, osc, fmt)
    assert e == pytest.approx(oracle.relative_error(np.ascontiguousarray(x[:, :cols]), oxh), rel=1e-6)
    assert codec_rel_error_gpu(x, fmt, cols=cols)[0] == e     # fixed reduction order


def test_fused_relative_error_extreme_blocks_and_errors():
    # blocks with amax = 0, subnormal maxima (unit scale), large values whose squares still fit fp32; no NaN / Inf
    # (they make e^L NaN by definition)
    x = np.zeros((8, 256), np.uint16)
    x[1, :64] = 0x0001
    x[2, 64:128] = 0x5D00
    x[3, :] = np.random.default_rng(5).integers(0, 0x5D00, 256).astype(np.uint16)
    x[4, :] = x[3, :] | 0x8000
    for fmt in (api.FMT_E4M3FN_BLK, api.FMT_INT8_BLK):
        e, _ = codec_rel_error_gpu(x, fmt)
        codes, scales, _ = G.compress(x, fmt)
        assert e == pytest.approx(rel_error_gpu(x, G.recover(codes, scales, fmt))[0], rel=1e-12)
    x[5, 3] = 0x7FC0
    assert np.isnan(codec_rel_error_gpu(x, api.FMT_E4M3FN_BLK)[0])
    d = torch.zeros(64 * 4, dtype=torch.int16, device="cuda")
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    ws = torch.zeros(api.hilore_relative_error_workspace_bytes(), dtype=torch.uint8, device="cuda")
    call = lambda cols=64, fmt=1, block=64, nws=ws.numel(): api.hilore_codec_relative_error(
        d, 4, cols, 64, fmt, block, out, None, ws, nws, check=False)
    assert call() == api.OK and call(cols=48) == api.SHAPE and call(fmt=7) == api.INVALID_ARG
    assert call(block=32) == api.SHAPE and call(nws=16) == api.WORKSPACE
