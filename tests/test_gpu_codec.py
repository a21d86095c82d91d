"""Parity of hilore_compress / hilore_recover with the CPU oracle: codes, scales and recovered bf16
bit-exact; token RMS within 1e-5 relative.  All calls go through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2609_33570_b200 import api, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu
FMTS = [api.FMT_E4M3FN_RAW, api.FMT_E4M3FN_BLK, api.FMT_INT8_BLK]
RMS_RTOL = 1e-5


def block_of(fmt):
    return 0 if fmt == api.FMT_E4M3FN_RAW else 64


def check_roundtrip(x, fmt, cols=None, ld_out=None):
    blk = block_of(fmt)
    codes, scales, rms = G.compress(x, fmt, cols=cols)
    o_codes, o_scales = oracle.compress(x, fmt, blk, cols=cols)
    assert np.array_equal(codes, o_codes), f"codes differ at {np.argwhere(codes != o_codes)[:5]}"
    if blk:
        assert np.array_equal(scales.view(np.uint32), o_scales.view(np.uint32))
    o_rms = oracle.row_rms(x, cols=cols)
    # the kernel squares and accumulates in fp32 (as the paper does): rows whose squares leave the fp32
    # range (|x| beyond 1e18 overflows, below 1e-19 underflows) differ from the fp64 oracle -- not compared
    in_range = np.isfinite(o_rms) & (o_rms < 1e15) & ((o_rms > 1e-15) | (o_rms == 0))
    assert np.all(np.isfinite(rms[in_range])) and not np.any(np.isfinite(rms[~np.isfinite(o_rms)]))
    assert G.rel_err(rms[in_range], o_rms[in_range]).max(initial=0) <= RMS_RTOL
    rec = G.recover(o_codes, o_scales, fmt, ld_out=ld_out)
    o_rec = oracle.recover(o_codes, o_scales, fmt, blk, ld_out=ld_out)
    c = o_codes.shape[1]
    nan = (o_rec[:, :c] & 0x7FFF) > 0x7F80
    assert np.array_equal(((rec[:, :c] & 0x7FFF) > 0x7F80), nan)
    assert np.array_equal(rec[:, :c][~nan], o_rec[:, :c][~nan])
    if ld_out is not None and ld_out > c:
        assert np.all(rec[:, c:] == (G.CANARY | (G.CANARY << 8))), "padding columns of the output were written"
    return codes, scales, rms


@pytest.mark.parametrize("fmt", FMTS)
def test_every_bf16_pattern(fmt):
    """All 65 536 bf16 bit patterns (overflow, subnormals, signed zeros, Inf, NaN payloads)."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(1024, 64)
    check_roundtrip(bits, fmt)
    # patterns shuffled so that blocks mix magnitudes, signs and non-finite values
    rng = np.random.default_rng(0)
    check_roundtrip(rng.permutation(bits.reshape(-1)).reshape(64, 1024), fmt)


@pytest.mark.parametrize("fmt", [api.FMT_E4M3FN_BLK, api.FMT_INT8_BLK])
def test_every_block_absmax(fmt):
    """One block per finite bf16 magnitude as its absmax (all 32 640 of them, either sign), the other elements
    spread below it: the scale, its reciprocal and every code must match the oracle's IEEE divisions bit for bit
    over the whole exponent range (unit-scale blocks, the subnormal-scale band and the table range)."""
    rng = np.random.default_rng(11)
    amax = np.arange(0, 0x7F80, dtype=np.uint32)
    nblk = len(amax)
    frac = rng.integers(0, 0x0400, size=(nblk, 64), dtype=np.uint32)          # up to 8 binades below the absmax
    mag = np.maximum(amax[:, None].astype(np.int64) - frac, 0).astype(np.uint32)
    pos = rng.integers(0, 64, nblk)
    mag[np.arange(nblk), pos] = amax
    sign = rng.integers(0, 2, size=(nblk, 64), dtype=np.uint32) << 15
    x = (mag | sign).astype(np.uint16).reshape(nblk // 16, 1024)                  # 2040 rows of 16 blocks
    check_roundtrip(x, fmt)


def test_every_code_decodes():
    codes = np.arange(256, dtype=np.uint32).astype(np.uint8).reshape(4, 64)
    for fmt in FMTS:
        scales = None if fmt == api.FMT_E4M3FN_RAW else np.array([[1.0], [0.37], [3e-5], [1e20]], np.float32)
        rec = G.recover(codes, scales, fmt)
        o = oracle.recover(codes, scales, fmt, block_of(fmt))
        nan = (o & 0x7FFF) > 0x7F80
        assert np.array_equal((rec & 0x7FFF) > 0x7F80, nan)
        assert np.array_equal(rec[~nan], o[~nan])


@pytest.mark.parametrize("fmt", FMTS)
def test_config1_tiny_units(fmt):
    """Tiny GRPO step: two units [8192, 896], N(0,1) with 1% x20 outlier channels, seed 0."""
    rng = np.random.default_rng(0)
    for _ in range(2):
        x = synth.activation_unit(rng, 8192, 896)
        check_roundtrip(x, fmt)


@pytest.mark.parametrize("rows,cols", [(1, 64), (3, 192), (37, 4096), (5, 18944), (300, 64), (129, 1536),
                                       (2, 8960), (1, 262144)])
@pytest.mark.parametrize("fmt", FMTS)
def test_ragged_shapes(rows, cols, fmt):
    x = synth.activation_unit(np.random.default_rng(rows * 131 + cols), rows, cols)
    check_roundtrip(x, fmt)


@pytest.mark.parametrize("fmt", FMTS)
def test_leading_dimensions(fmt):
    rng = np.random.default_rng(5)
    x = synth.activation_unit(rng, 50, 640)
    wide = np.full((50, 704), 0x7FC0, np.uint16)      # NaN padding: must never be read
    wide[:, :640] = x
    c1, s1, r1 = G.compress(x, fmt)
    c2, s2, r2 = check_roundtrip(wide, fmt, cols=640, ld_out=672)
    assert np.array_equal(c1, c2) and np.array_equal(r1, r2)


@pytest.mark.parametrize("fmt", FMTS)
def test_special_values_inside_gaussian_data(fmt):
    rng = np.random.default_rng(6)
    x = synth.activation_unit(rng, 64, 1024)
    x[0, 0:64] = 0                                     # all-zero block
    x[1, 64:128] = 0x8000                              # all minus-zero block
    x[2, 5] = 0x7FC0
    x[3, 70] = 0x7F80
    x[4, 130] = 0xFF80
    x[5, 192:256] = 0x0001                             # smallest subnormals
    x[6, 256:320] = 0x7FC1                             # block without a finite element
    x[7, 320:384] = 0x7F7F                             # largest finite value
    x[8, 0] = 0x43E8                                   # 464: last value that still rounds to 448 unscaled
    x[9, 0] = 0x43E9                                   # 466: overflows to NaN unscaled
    x[10, 3] = 0xC3E9
    # blocks whose absmax sits at / just above the point where Q / amax stops fitting fp32
    for row, bits in ((11, 0x03E0), (12, 0x03E1), (13, 0x02FE), (14, 0x02FF), (15, 0x0380), (16, 0x0400)):
        x[row, 384:448] = 0x0001
        x[row, 400] = bits
        x[row, 401] = bits | 0x8000
    check_roundtrip(x, fmt)


def test_stats_only_and_no_stats():
    rng = np.random.default_rng(7)
    x = synth.activation_unit(rng, 77, 1536)
    _, _, rms = G.compress(x, api.FMT_E4M3FN_RAW, want_codes=False)
    assert G.rel_err(rms, oracle.row_rms(x)).max() <= RMS_RTOL
    codes, scales, none = G.compress(x, api.FMT_E4M3FN_BLK, want_rms=False)
    o_codes, o_scales = oracle.compress(x, api.FMT_E4M3FN_BLK, 64)
    assert none is None and np.array_equal(codes, o_codes) and np.array_equal(scales, o_scales)


@pytest.mark.parametrize("fmt", FMTS)
def test_codes_only_pass_on_16KB_pieces_with_special_values_and_a_ragged_tail(fmt):
    """Without the token RMS a contiguous unit is shared as 16 KB pieces (rows do not matter) plus one short tail:
    77 x 1536 elements = 14 pieces and 144 chunks.  Special values sit in whole pieces and in the tail."""
    rng = np.random.default_rng(17)
    x = synth.activation_unit(rng, 77, 1536)
    x[0, 5] = 0x7FC0                                   # NaN in the first piece
    x[3, 70] = 0x7F80                                  # +Inf
    x[40, 640:704] = 0                                 # an all-zero block
    x[41, 0] = 0x43E9                                  # 466: overflows to NaN in the unscaled cast
    x[76, 1500] = 0xFF80                               # -Inf in the tail
    x[76, 1535] = 0xFFC0                               # NaN in the last element
    codes, scales, none = G.compress(x, fmt, want_rms=False)
    o_codes, o_scales = oracle.compress(x, fmt, 0 if fmt == api.FMT_E4M3FN_RAW else 64)
    assert none is None and np.array_equal(codes, o_codes)
    if o_scales is not None:
        assert np.array_equal(scales.view(np.uint32), o_scales.view(np.uint32))
    got = G.recover(codes, scales, fmt)
    want = oracle.recover(o_codes, o_scales, fmt, 0 if fmt == api.FMT_E4M3FN_RAW else 64)
    nan = lambda b: (b & 0x7FFF) > 0x7F80
    assert np.array_equal(nan(got), nan(want)) and np.array_equal(got[~nan(want)], want[~nan(want)])


def test_run_to_run_determinism():
    x = synth.activation_unit(np.random.default_rng(8), 4096, 3584)
    a = G.compress(x, api.FMT_E4M3FN_BLK)
    b = G.compress(x, api.FMT_E4M3FN_BLK)
    for p, q in zip(a, b):
        assert p.tobytes() == q.tobytes()


def test_error_statistic_of_gpu_roundtrip_matches_oracle():
    """e^L of the paper's unscaled round trip on N(0,1) data, GPU recovery vs oracle recovery."""
    x = synth.activation_unit(np.random.default_rng(9), 256, 1536)
    codes, _, _ = G.compress(x, api.FMT_E4M3FN_RAW)
    rec = G.recover(codes, None, api.FMT_E4M3FN_RAW)
    o_codes, _ = oracle.compress(x, api.FMT_E4M3FN_RAW, 0)
    o_rec = oracle.recover(o_codes, None, 0, 0)
    assert np.array_equal(codes, o_codes) and np.array_equal(rec, o_rec)
    assert 0.02 < oracle.relative_error(x, o_rec) < 0.035


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_leading_dimensions_and_specials(seed):
    """Random rows / widths / leading dimensions / formats with special values sprinkled in (zeros, tiny and huge
    magnitudes, Inf, NaN, whole blocks of one value): everything bit-exact against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    for _ in range(5):
        rows = int(rng.integers(1, 700))
        cols = 64 * int(rng.integers(1, 80))
        pad = 16 * int(rng.integers(0, 4))
        fmt = FMTS[int(rng.integers(0, 3))]
        x = synth.activation_unit(rng, rows, cols)
        n_special = int(rng.integers(0, 40))
        specials = np.array([0x0000, 0x8000, 0x0001, 0x007F, 0x0080, 0x03E0, 0x03E1, 0x04DF, 0x04E0, 0x02FE, 0x03FE, 0x43E8, 0x43E9,
                             0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x7FC0, 0xFFC1, 0x3F80], np.uint16)
        r_idx, c_idx = rng.integers(0, rows, n_special), rng.integers(0, cols, n_special)
        x[r_idx, c_idx] = specials[rng.integers(0, len(specials), n_special)]
        for _ in range(int(rng.integers(0, 4))):                      # whole blocks of one special value
            r, b = int(rng.integers(0, rows)), int(rng.integers(0, cols // 64))
            x[r, 64 * b:64 * b + 64] = specials[int(rng.integers(0, len(specials)))]
        if pad:
            wide = np.full((rows, cols + pad), 0x7FC0, np.uint16)      # NaN padding: must never be read
            wide[:, :cols] = x
            check_roundtrip(wide, fmt, cols=cols, ld_out=cols + 16 * int(rng.integers(0, 3)))
        else:
            check_roundtrip(x, fmt)
