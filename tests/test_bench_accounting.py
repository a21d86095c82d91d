"""The byte accounting of bench.py (what the method itself must move), against the per-unit figures written out by hand."""
import bench


def test_codec_bytes_per_element():
    n = 8192 * 1536
    assert bench.codec_bytes(8192, 1536, fmt_scaled=True, with_rms=True) == 2 * n + n + 4 * n // 64 + 4 * 8192
    assert bench.codec_bytes(8192, 1536, fmt_scaled=True, with_rms=False) == 3 * n + n // 16
    assert bench.codec_bytes(8192, 1536, fmt_scaled=False, with_rms=False) == 3 * n          # the paper's unscaled codec
    assert bench.stats_bytes(16384, 18944) == 2 * 16384 * 18944 + 4 * 16384


def test_coefficient_and_exposure_bytes():
    assert bench.coeff_bytes(1 << 24) == 13 << 24                        # two fp32 reads, one mask byte, one fp32 write
    assert bench.coeff_bytes(1 << 24, with_ref=True) == 17 << 24         # + the reference log-probabilities
    assert bench.coeff_bytes(1024, extras=True) == 18 * 1024             # + ratio and clip indicator
    assert bench.exposure_bytes(16384, 84) == 16384 * (5 + 4 * 84)       # omega + mask once, one token RMS per unit


def test_configs_are_the_shapes_the_benchmark_names():
    c2, c3 = bench.CONFIGS[2], bench.CONFIGS[3]
    assert (c2["P"], c2["G"], c2["T"], c2["mb_resp"], c2["layers"], c2["model"], c2["plan"]) == (64, 8, 1024, 8, 28, "1.5B", "all_L")
    assert (c3["P"], c3["G"], c3["T"], c3["mb_resp"], c3["layers"], c3["model"], c3["plan"]) == (128, 16, 2048, 8, 28, "7B", "mixed")
    assert bench.DEFAULT_CONFIG == 3 and c3["workload"].startswith("7B-shaped")
