"""Pins for the oracle's low-precision codec.

Unscaled format (the paper's, Eq. "fp8-roundtrip"): the paper names the routine -- torch's
float8_e4m3fn cast without scales -- so the oracle's hand-written rounding is compared with
that cast on every bf16 bit pattern and every code, with spot values worked from the format
definition, and with a brute-force nearest-grid-point search.
Block-scaled formats (not in the paper): worked block, reduction to the unscaled format for
power-of-two scales, error bounds, brute force.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import FMT_E4M3FN_BLK, FMT_E4M3FN_RAW, FMT_INT8_BLK

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x):
    return torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def bits_to_f32(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


ALL_BITS = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(1024, 64)


def torch_cast_bf16_to_e4m3(bits):
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    return t.to(torch.float8_e4m3fn).view(torch.uint8).numpy()


def test_raw_encode_matches_named_cast_exhaustively():
    codes, scales = oracle.compress(ALL_BITS, FMT_E4M3FN_RAW, 0)
    assert scales is None
    want = torch_cast_bf16_to_e4m3(ALL_BITS)
    nan_in = (ALL_BITS & 0x7FFF) > 0x7F80
    # NaN inputs: the cast yields a NaN code; compare as a class (magnitude bits 0x7F)
    assert np.all((codes[nan_in] & 0x7F) == 0x7F) and np.all((want[nan_in] & 0x7F) == 0x7F)
    assert np.array_equal(codes[~nan_in], want[~nan_in])


def test_raw_decode_matches_named_cast_exhaustively():
    codes = np.arange(256, dtype=np.uint32).astype(np.uint8).reshape(4, 64)
    got = oracle.recover(codes, None, FMT_E4M3FN_RAW, 0)
    want = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    is_nan = (codes & 0x7F) == 0x7F
    assert np.array_equal(got[~is_nan], want[~is_nan])
    for a in (got[is_nan], want[is_nan]):
        assert np.all((a & 0x7FFF) > 0x7F80)
    # decode is exact: re-encoding every non-NaN decoded value returns the code (-0 keeps its sign)
    back, _ = oracle.compress(got, FMT_E4M3FN_RAW, 0)
    assert np.array_equal(back[~is_nan], codes[~is_nan])


def test_raw_spot_values_from_format_definition():
    for line in open(os.path.join(GOLD, "e4m3fn_spot_values.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        v, code, dec = [f.strip() for f in line.split("|")]
        b = bf16_bits([[float(v)]])
        assert bits_to_f32(b)[0, 0] == float(v), "spot value must be exact in bf16"
        c, _ = oracle.compress(b, FMT_E4M3FN_RAW, 0)
        assert int(c[0, 0]) == int(code, 16), (v, hex(int(c[0, 0])))
        d = bits_to_f32(oracle.recover(c, None, FMT_E4M3FN_RAW, 0))[0, 0]
        if dec == "nan":
            assert np.isnan(d)
        else:
            assert d == float(dec) and np.signbit(d) == dec.startswith("-")


def _grid():
    """All finite E4M3FN magnitudes, written from the format definition (not via the oracle)."""
    vals = [m * 2.0 ** -9 for m in range(8)]
    for E in range(1, 16):
        for M in range(8):
            if E == 15 and M == 7:
                continue
            vals.append((8 + M) * 2.0 ** (E - 10))
    return np.array(vals)


def test_grid_has_the_documented_shape():
    g = _grid()
    assert len(g) == 127 and g.max() == 448.0 and np.all(np.diff(g) > 0)
    assert g[8] == 2.0 ** -6 and g[1] == 2.0 ** -9


def test_raw_encode_is_nearest_grid_point_brute_force():
    """Nearest value of the 127-point grid, ties to the even code, for every finite bf16 <= 464."""
    g = _grid()
    bits = np.arange(0x0000, 0x43E9, dtype=np.uint32).astype(np.uint16)      # +0 .. 464
    x = bits_to_f32(bits).astype(np.float64)
    d = np.abs(x[:, None] - g[None, :])
    best = d.min(axis=1)
    cand = d == best[:, None]
    idx = np.where(cand.sum(axis=1) == 1, cand.argmax(axis=1), -1)
    ties = np.where(idx < 0)[0]
    for i in ties:
        two = np.where(cand[i])[0]
        assert len(two) == 2
        idx[i] = two[0] if two[0] % 2 == 0 else two[1]       # code index = magnitude code; even mantissa
    pad = (-len(bits)) % 64
    bits_p = np.concatenate([bits, np.zeros(pad, np.uint16)]).reshape(-1, 64)
    codes, _ = oracle.compress(bits_p, FMT_E4M3FN_RAW, 0)
    codes = codes.reshape(-1)[: len(bits)]
    assert np.array_equal(codes.astype(np.int64), idx)
    # and the error bound of the format: relative 2^-4 in the normal range, absolute 2^-10 below it
    xh = g[codes]
    normal = x >= 2.0 ** -6
    assert np.all(np.abs(xh - x)[normal & (x <= 448)] <= x[normal & (x <= 448)] * 2.0 ** -4)
    assert np.all(np.abs(xh - x)[~normal] <= 2.0 ** -10)


def test_raw_codes_monotone_and_odd_symmetric():
    pos = np.arange(0, 0x7F80, dtype=np.uint32).astype(np.uint16)
    pad = (-len(pos)) % 64
    p = np.concatenate([pos, np.full(pad, pos[-1], np.uint16)]).reshape(-1, 64)
    c_pos, _ = oracle.compress(p, FMT_E4M3FN_RAW, 0)
    c_neg, _ = oracle.compress(p | 0x8000, FMT_E4M3FN_RAW, 0)
    assert np.array_equal(c_neg, c_pos | 0x80)
    flat = c_pos.reshape(-1).astype(np.int64)
    assert np.all(np.diff(flat) >= 0)
    assert flat[0x43E8] == 0x7E and flat[0x43E9] == 0x7F          # 464 -> 448, next bf16 (466) -> NaN


def _read_worked():
    d = {}
    for line in open(os.path.join(GOLD, "block64_worked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = [f.strip() for f in line.split("|")]
        d[k] = v.split()
    return d


def test_blk_worked_block():
    w = _read_worked()
    x = bf16_bits([[(i - 32) / 8 for i in range(64)]])
    codes, scales = oracle.compress(x, FMT_E4M3FN_BLK, 64)
    assert scales.view(np.uint32)[0, 0] == int(w["scale_bits"][0], 16)
    assert [f"{c:02X}" for c in codes[0]] == w["codes"]
    rec = oracle.recover(codes, scales, FMT_E4M3FN_BLK, 64)
    assert [f"{c:04X}" for c in rec[0]] == w["recovered"]


def _acts(seed, rows, cols, outliers=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    if outliers:
        x[:, rng.permutation(cols)[: max(1, cols // 100)]] *= 20
    return bf16_bits(x)


def test_blk_encode_step_matches_named_cast_on_scaled_values():
    """codes = cast_E4M3FN(fl32(x * fl32(448/amax))): scale arithmetic redone in NumPy fp32, the
    rounding step done by the cast the paper names (RNE for |q| <= 448)."""
    x = _acts(0, 64, 256)
    codes, scales = oracle.compress(x, FMT_E4M3FN_BLK, 64)
    xf = bits_to_f32(x).reshape(64, 4, 64)
    amax = np.abs(xf).max(axis=2)
    s = (amax / np.float32(448.0)).astype(np.float32)
    inv = (np.float32(448.0) / amax).astype(np.float32)
    assert np.array_equal(s.view(np.uint32), scales.view(np.uint32))
    q = (xf * inv[:, :, None]).astype(np.float32)
    assert np.abs(q).max() <= 448.0 * (1 + 2.0 ** -22)
    q = np.clip(q, -448.0, 448.0)
    want = torch.from_numpy(q.reshape(64, 256)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes, want)
    # the block's amax element always lands on +-448
    flat = np.abs(xf).argmax(axis=2)
    c3 = codes.reshape(64, 4, 64)
    top = np.take_along_axis(c3, flat[:, :, None], axis=2)[:, :, 0]
    assert np.all((top & 0x7F) == 0x7E)


@pytest.mark.parametrize("k", [-3, 0, 2, 7])
def test_blk_reduces_to_raw_for_power_of_two_scales(k):
    """amax = 448 * 2^-k  =>  inv = 2^k, s = 2^-k exactly and BLK(x) == RAW(x * 2^k)."""
    rng = np.random.default_rng(7)
    y = (rng.standard_normal((8, 64)) * 60).astype(np.float32)
    y = np.clip(y, -440, 440)
    y[:, 5] = 448.0 * np.where(rng.random(8) < 0.5, -1, 1)
    yb = bf16_bits(y)                                   # |y| <= 448, amax = 448
    xb = bf16_bits(bits_to_f32(yb) * np.float32(2.0 ** -k))
    assert np.array_equal(bits_to_f32(xb) * np.float32(2.0 ** k), bits_to_f32(yb))   # exact scaling
    c_blk, s_blk = oracle.compress(xb, FMT_E4M3FN_BLK, 64)
    c_raw, _ = oracle.compress(yb, FMT_E4M3FN_RAW, 0)
    assert np.array_equal(c_blk, c_raw)
    assert np.all(s_blk == np.float32(2.0 ** -k))
    r_blk = bits_to_f32(oracle.recover(c_blk, s_blk, FMT_E4M3FN_BLK, 64))
    r_raw = bits_to_f32(oracle.recover(c_raw, None, FMT_E4M3FN_RAW, 0))
    assert np.array_equal(r_blk, r_raw * np.float32(2.0 ** -k))


def test_blk_scale_invariance_and_error_bound():
    x = _acts(1, 32, 512)
    xf = bits_to_f32(x)
    c1, s1 = oracle.compress(x, FMT_E4M3FN_BLK, 64)
    c2, s2 = oracle.compress(bf16_bits(xf * np.float32(0.125)), FMT_E4M3FN_BLK, 64)
    assert np.array_equal(c1, c2) and np.array_equal(s1 * np.float32(0.125), s2)
    # pre-rounding reconstruction error: half a grid step of q, times s
    deq = oracle.dequant_f32(c1, s1, FMT_E4M3FN_BLK, 64).astype(np.float64)
    s = np.repeat(s1.astype(np.float64), 64, axis=1)
    q = np.abs(xf.astype(np.float64)) / s
    step_half = 2.0 ** (np.maximum(np.floor(np.log2(np.maximum(q, 1e-300))), -6) - 4)
    assert np.all(np.abs(deq - xf) <= s * step_half * (1 + 1e-5) + 1e-30)


def test_int8_error_bound_half_scale():
    """The literal bound of a uniform grid: |fl32(code*s) - x| <= s/2 before the bf16 rounding."""
    x = _acts(2, 32, 512)
    xf = bits_to_f32(x).astype(np.float64)
    c, s = oracle.compress(x, FMT_INT8_BLK, 64)
    ci = c.view(np.int8)
    assert ci.min() >= -127 and ci.max() <= 127
    deq = oracle.dequant_f32(c, s, FMT_INT8_BLK, 64).astype(np.float64)
    srep = np.repeat(s.astype(np.float64), 64, axis=1)
    assert np.all(np.abs(deq - xf) <= 0.5 * srep * (1 + 1e-5))
    # brute force: the code is the nearest integer multiple of s (in the fp32 arithmetic of the definition)
    inv = (np.float32(127.0) / np.abs(bits_to_f32(x)).reshape(32, 8, 64).max(axis=2)).astype(np.float32)
    q = (bits_to_f32(x).reshape(32, 8, 64) * inv[:, :, None]).astype(np.float32)
    assert np.array_equal(ci.reshape(32, 8, 64), np.clip(np.rint(q), -127, 127).astype(np.int8))
    rec = bits_to_f32(oracle.recover(c, s, FMT_INT8_BLK, 64))
    assert np.array_equal(rec, bits_to_f32(bf16_bits(deq.astype(np.float32))))


@pytest.mark.parametrize("fmt", [FMT_E4M3FN_BLK, FMT_INT8_BLK])
def test_blk_degenerate_blocks(fmt):
    x = np.zeros((1, 256), np.uint16)
    x[0, 1] = 0x8000                                        # -0 in an all-zero block
    x[0, 64:128] = bf16_bits([np.linspace(-1, 1, 64)])[0]
    x[0, 70] = 0x7FC0                                       # NaN inside a finite block
    x[0, 71] = 0x7F80                                       # +Inf
    x[0, 72] = 0xFF80                                       # -Inf
    x[0, 128:192] = 0x0001                                  # tiny subnormals: 448/amax overflows fp32
    x[0, 192:256] = 0x7FC0                                  # no finite element at all
    c, s = oracle.compress(x, fmt, 64)
    assert s[0, 0] == 1.0 and np.all(c[0, 0:64] == np.where(np.arange(64) == 1, 0x80 if fmt == FMT_E4M3FN_BLK else 0, 0))
    Q = 448.0 if fmt == FMT_E4M3FN_BLK else 127.0
    assert s[0, 1] == np.float32(1.0) / np.float32(Q)       # amax ignores the non-finite entries
    nan_code = 0x7F if fmt == FMT_E4M3FN_BLK else 0x80
    top = 0x7E if fmt == FMT_E4M3FN_BLK else 127
    assert (c[0, 70] & (0x7F if fmt == FMT_E4M3FN_BLK else 0xFF)) == nan_code
    assert c[0, 71] == top and c[0, 72] == ((0xFE) if fmt == FMT_E4M3FN_BLK else np.uint8(np.int8(-127).view(np.uint8)))
    assert s[0, 2] == 1.0 and np.all(c[0, 128:192] == 0)
    assert s[0, 3] == 1.0
    rec = bits_to_f32(oracle.recover(c, s, fmt, 64))
    assert np.isnan(rec[0, 70]) and np.all(np.isnan(rec[0, 192:256]))
    assert abs(rec[0, 71] - 1.0) < 1e-2 and abs(rec[0, 72] + 1.0) < 1e-2


def test_relative_error_statistic_on_gaussian_data():
    """e^L of the unscaled round trip on N(0,1): a 3-bit mantissa gives a relative RMS error of
    about 2^-4/sqrt(3) * c with c in (0.7, 1): between 0.02 and 0.035."""
    x = _acts(3, 64, 1024, outliers=False)
    c, _ = oracle.compress(x, FMT_E4M3FN_RAW, 0)
    e = oracle.relative_error(x, oracle.recover(c, None, FMT_E4M3FN_RAW, 0))
    assert 0.02 < e < 0.035
    xf = bits_to_f32(x).astype(np.float64)
    rf = bits_to_f32(oracle.recover(c, None, FMT_E4M3FN_RAW, 0)).astype(np.float64)
    assert e == pytest.approx(np.linalg.norm(rf - xf) / (np.linalg.norm(xf) + 1e-8), rel=1e-12)


def test_leading_dimension_and_shape_errors():
    x = _acts(4, 4, 192)
    wide = np.zeros((4, 256), np.uint16)
    wide[:, :192] = x
    wide[:, 192:] = 0x7FC0                                   # padding must never be read
    for fmt, blk in ((FMT_E4M3FN_RAW, 0), (FMT_E4M3FN_BLK, 64), (FMT_INT8_BLK, 64)):
        c1, s1 = oracle.compress(x, fmt, blk)
        c2, s2 = oracle.compress(wide, fmt, blk, cols=192)
        assert np.array_equal(c1, c2) and (s1 is None or np.array_equal(s1, s2))
        out = oracle.recover(c1, s1, fmt, blk, ld_out=200)
        assert np.array_equal(out[:, :192], oracle.recover(c1, s1, fmt, blk)) and np.all(out[:, 192:] == 0)
    with pytest.raises(oracle.OracleError):
        oracle.compress(_acts(5, 2, 96), FMT_E4M3FN_BLK, 64)


@pytest.mark.parametrize("fmt,Q,last_unit", [(FMT_E4M3FN_BLK, 448.0, 0x03E0), (FMT_INT8_BLK, 127.0, 0x02FE)])
def test_blk_unit_scale_threshold(fmt, Q, last_unit):
    """s = inv = 1 exactly when fl32(Q / amax) overflows: amax <= 1.75 * 2^-120 (Q = 448) resp.
    1.984375 * 2^-122 (Q = 127); the next bf16 value already gets a finite reciprocal."""
    for bits, unit in ((last_unit, True), (last_unit + 1, False), (1, True), (last_unit - 1, True)):
        x = np.full((1, 64), 0x0001, np.uint16)
        x[0, 7] = bits
        amax = float(bits_to_f32(np.array([bits], np.uint16))[0])
        with np.errstate(over="ignore"):
            overflow = np.isinf(np.float32(Q) / np.float32(amax))
        assert overflow == unit
        c, s = oracle.compress(x, fmt, 64)
        if unit:
            assert s[0, 0] == 1.0 and np.all(c == 0)
        else:
            assert s[0, 0] == np.float32(amax) / np.float32(Q) and (c[0, 7] & 0x7F) == (0x7E if fmt == FMT_E4M3FN_BLK else 127)


def test_unscaled_tables_match_the_recorded_digests():
    """The exhaustive encode / decode tables of the oracle hash to the digests recorded from the cast the paper
    names (a fixed pin that does not depend on the torch installed next to the tests)."""
    import hashlib
    want = {}
    for line in open(os.path.join(GOLD, "e4m3fn_table_digests.txt")):
        if not line.startswith("#") and "|" in line:
            k, v = (p.strip() for p in line.split("|"))
            want[k] = v
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(1024, 64)
    codes, _ = oracle.compress(bits, 0, 0)
    assert hashlib.sha256(codes.tobytes()).hexdigest() == want["encode"]
    every = np.arange(256, dtype=np.uint32).astype(np.uint8).reshape(4, 64)
    rec = oracle.recover(every, None, 0, 0)
    assert hashlib.sha256(rec.astype("<u2").tobytes()).hexdigest() == want["decode"]
