"""Small single-kernel cases for profiler captures (`python -m paper_2609_33570_b200.profile_case ...`).

Each case holds well under a few GB on the device, uses inputs larger than L2, and launches the kernel
of interest a handful of times, so that a multi-pass profiler capture ends by itself quickly.
"""
from __future__ import annotations

import argparse

import torch

from . import api, synth


def codec_case(rows: int, cols: int, fmt: int, reps: int, units: int, rms: bool = True, codes_on: bool = True,
               recover: bool = True):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(0)
    block = 0 if fmt == api.FMT_E4M3FN_RAW else 64
    xs = [synth.activation_unit_device(gen, rows, cols) for _ in range(units)]
    codes = [torch.empty((rows, cols), dtype=torch.uint8, device="cuda") for _ in range(units)]
    scales = [torch.empty((rows, max(cols // 64, 1)), dtype=torch.float32, device="cuda") for _ in range(units)]
    outs = [torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda") for _ in range(units)]
    rms_buf = torch.empty((units, rows), dtype=torch.float32, device="cuda")
    for _ in range(reps):
        for i in range(units):
            api.hilore_compress(xs[i], rows, cols, cols, fmt, block, codes[i] if codes_on else None,
                                scales[i] if (block and codes_on) else None, rms_buf[i] if (rms or not codes_on) else None)
        for i in range(units if recover else 0):
            api.hilore_recover(codes[i], scales[i] if block else None, rows, cols, fmt, block, outs[i], cols)
    torch.cuda.synchronize()


def coeffs_case(log2_slots: int, reps: int):
    n_resp = (1 << log2_slots) // 1024
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1)
    lp = torch.randn((n_resp, 1024), generator=gen, device="cuda") * 0.5 - 1.5
    lo = lp + torch.randn((n_resp, 1024), generator=gen, device="cuda") * 0.05
    mask = torch.ones((n_resp, 1024), dtype=torch.uint8, device="cuda")
    rewards = (torch.rand(n_resp, generator=gen, device="cuda") < 0.5).float()
    omega = torch.empty_like(lp)
    for _ in range(reps):
        api.hilore_grpo_coeffs(rewards, n_resp, 16, 0, n_resp, 1024, lp, lo, None, mask, n_resp * 1024, None, 0.2,
                               0.0, 1e-6, None, omega, None, None)
    torch.cuda.synchronize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", choices=["codec", "coeffs"], default="codec")
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--cols", type=int, default=8960)
    ap.add_argument("--fmt", type=int, default=api.FMT_E4M3FN_BLK)
    ap.add_argument("--units", type=int, default=2)
    ap.add_argument("--reps", type=int, default=2)
    ap.add_argument("--log2-slots", type=int, default=24)
    ap.add_argument("--no-rms", action="store_true", help="compress without the fused token RMS")
    ap.add_argument("--stats-only", action="store_true", help="token RMS only, no codes")
    ap.add_argument("--no-recover", action="store_true")
    a = ap.parse_args()
    if a.kernel == "codec":
        codec_case(a.rows, a.cols, a.fmt, a.reps, a.units, rms=not a.no_rms, codes_on=not a.stats_only,
                   recover=not a.no_recover)
    else:
        coeffs_case(a.log2_slots, a.reps)
    print("done")


if __name__ == "__main__":
    main()
