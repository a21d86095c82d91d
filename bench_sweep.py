"""Bandwidth sweep of the single-unit entry points and the auxiliary kernels (`python bench_sweep.py`).

Units [rows, cols] bf16 of 1 MiB ... 4 GiB (row width 4096 by default), compress then recover, and the
coefficient kernel over 2^16 ... 2^24 slots at G = 16.  Each point is timed with CUDA events over `reps`
calls that rotate through a pool of distinct buffers larger than L2, so the numbers are HBM numbers.
Prints one JSON line per point.  `bench.py` imports the point functions for the per-config legs of its line.

`--case codec|coeffs|coeffs-packed|exposure|scores|allocate|relerr|diagnostics` runs one small single-kernel case
a few times and exits: inputs larger than L2 where the kernel streams, well under a few GB on the device, a handful
of launches -- the cases the profiler captures under `profiles/` were taken on.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
from paper_2609_33570_b200 import api, synth  # noqa: E402

L2_BYTES = 126 << 20


def time_calls(fn_list, reps, warm=3):
    """Rotate through `fn_list` for `reps` calls.  loop_ms: CUDA events around the whole back-to-back loop, per call
    (the throughput figure).  device_us: median over calls of an event pair around each single call (what the GPU
    spends on one call, launch gaps of the stream included).  host_us: wall clock the host spends issuing one call
    (binding + launch), measured without synchronising -- a call is launch-bound when host_us exceeds device_us."""
    import time
    for f in fn_list[: min(len(fn_list), warm)]:
        f()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    t0 = time.perf_counter()
    for i in range(reps):
        fn_list[i % len(fn_list)]()
    host = (time.perf_counter() - t0) / reps
    e1.record()
    torch.cuda.synchronize()
    loop_ms = e0.elapsed_time(e1) / reps
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for i in range(reps):
        pairs[i][0].record()
        fn_list[i % len(fn_list)]()
        pairs[i][1].record()
    torch.cuda.synchronize()
    dev = sorted(a.elapsed_time(b) for a, b in pairs)[reps // 2]
    return {"loop_ms": loop_ms, "device_us": dev * 1e3, "host_us": host * 1e6}


def _time(fn_list, reps):
    return time_calls(fn_list, reps)["loop_ms"]


def codec_point(rows, cols, fmt, reps, with_rms=True, max_pool_bytes=6 << 30):
    block = 0 if fmt == api.FMT_E4M3FN_RAW else 64
    unit_bytes = rows * cols * 2
    pool = max(1, min(8, -(-3 * L2_BYTES // unit_bytes)))          # enough distinct units to defeat L2
    pool = max(1, min(pool, max_pool_bytes // (unit_bytes * 2 + rows * cols)))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(0)
    base = synth.activation_unit_device(gen, min(rows, 4096), cols)
    xs = [base.repeat(-(-rows // base.shape[0]), 1)[:rows].contiguous() for _ in range(pool)]
    codes = [torch.empty((rows, cols), dtype=torch.uint8, device="cuda") for _ in range(pool)]
    scales = [torch.empty((rows, max(cols // 64, 1)), dtype=torch.float32, device="cuda") for _ in range(pool)]
    outs = [torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda") for _ in range(pool)]
    rms = torch.empty(rows, dtype=torch.float32, device="cuda")
    comp = [lambda i=i: api.hilore_compress(xs[i], rows, cols, cols, fmt, block, codes[i], scales[i] if block else None,
                                            rms if with_rms else None) for i in range(pool)]
    rec = [lambda i=i: api.hilore_recover(codes[i], scales[i] if block else None, rows, cols, fmt, block, outs[i], cols)
           for i in range(pool)]
    n = rows * cols
    nbytes = 3 * n + (4 * n // 64 if block else 0)
    dc, dr = time_calls(comp, reps), time_calls(rec, reps)
    tc, tr = dc["loop_ms"], dr["loop_ms"]
    return {"kernel": "codec", "rows": rows, "cols": cols, "fmt": fmt, "unit_mib": unit_bytes / 2 ** 20, "pool": pool,
            "compress_us": tc * 1e3, "compress_gbs": (nbytes + (4 * rows if with_rms else 0)) / tc / 1e6,
            "compress_device_us": dc["device_us"], "compress_host_us": dc["host_us"],
            "recover_us": tr * 1e3, "recover_gbs": nbytes / tr / 1e6,
            "recover_device_us": dr["device_us"], "recover_host_us": dr["host_us"]}


def coeffs_point(log2_slots, reps, G=16, T=1024, beta=0.0):
    """hilore_grpo_coeffs over 2^log2_slots slots (13 B/slot; 17 with the K3 term, beta != 0)."""
    n_resp = max(G, (1 << log2_slots) // T)
    slots = n_resp * T
    bps = 17 if beta else 13
    pool = max(1, min(8, -(-3 * L2_BYTES // (slots * bps))))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1)
    lp = [torch.randn((n_resp, T), generator=gen, device="cuda") * 0.5 - 1.5 for _ in range(pool)]
    lo = [x + torch.randn((n_resp, T), generator=gen, device="cuda") * 0.05 for x in lp]
    lr = [x + torch.randn((n_resp, T), generator=gen, device="cuda") * 0.05 for x in lp] if beta else [None] * pool
    mask = torch.ones((n_resp, T), dtype=torch.uint8, device="cuda")
    rewards = (torch.rand(n_resp, generator=gen, device="cuda") < 0.5).float()
    omega = [torch.empty_like(x) for x in lp]
    fns = [lambda i=i: api.hilore_grpo_coeffs(rewards, n_resp, G, 0, n_resp, T, lp[i], lo[i], lr[i], mask, slots, None, 0.2,
                                              beta, 1e-6, None, omega[i], None, None) for i in range(pool)]
    d = time_calls(fns, reps)
    t = d["loop_ms"]
    return {"kernel": "grpo_coeffs", "slots": slots, "beta": beta, "pool": pool, "us": t * 1e3, "device_us": d["device_us"],
            "host_us": d["host_us"], "tokens_per_s": slots / t * 1e3, "gbs": bps * slots / t / 1e6}


def coeffs_rollout_point(ro, reps):
    """hilore_grpo_coeffs over a whole host-drawn rollout batch (masks and rewards as drawn), N on the device."""
    dev = lambda a: torch.from_numpy(a).cuda()
    R, ln, lo, mk = dev(ro.rewards), dev(ro.logp_new), dev(ro.logp_old), dev(ro.mask)
    omega = [torch.empty_like(ln) for _ in range(3)]
    n = torch.zeros(1, dtype=torch.int64, device="cuda")
    api.hilore_mask_count(mk, mk.numel(), n)
    fns = [lambda i=i: api.hilore_grpo_coeffs(R, ro.n_resp, ro.G, 0, ro.n_resp, ro.T, ln, lo, None, mk, 0, n, 0.2, 0.0, 1e-6,
                                              None, omega[i], None, None) for i in range(3)]
    d = time_calls(fns, reps)
    slots = ro.n_resp * ro.T
    t = d["loop_ms"]
    return {"kernel": "grpo_coeffs", "slots": slots, "valid": ro.n_valid, "us": t * 1e3, "device_us": d["device_us"],
            "tokens_per_s": slots / t * 1e3, "valid_tokens_per_s": ro.n_valid / t * 1e3, "gbs": 13 * slots / t / 1e6}


def relerr_point(rows, cols, fmt, reps):
    """e^L of one unit: fused (x read once, codec in registers) against compress + recover + compare."""
    block = 0 if fmt == api.FMT_E4M3FN_RAW else 64
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4)
    pool = max(1, min(8, -(-3 * L2_BYTES // (rows * cols * 2))))
    base = synth.activation_unit_device(gen, min(rows, 4096), cols)
    xs = [base.repeat(-(-rows // base.shape[0]), 1)[:rows].contiguous() for _ in range(pool)]
    nws = api.hilore_relative_error_workspace_bytes()
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    e = torch.zeros(1, dtype=torch.float64, device="cuda")
    fused = [lambda i=i: api.hilore_codec_relative_error(xs[i], rows, cols, cols, fmt, block, e, None, ws, nws)
             for i in range(pool)]
    t = _time(fused, reps)
    return {"kernel": "codec_relative_error", "rows": rows, "cols": cols, "fmt": fmt, "us": t * 1e3,
            "gbs": 2 * rows * cols / t / 1e6, "e": e.item()}


def exposure_point(log2_tok, U, reps, masked_fraction=0.8):
    """hilore_unit_exposure over n_tok tokens (a share `masked_fraction` of them valid) and U units:
    n_tok * (5 + 4 U) bytes."""
    n_tok = 1 << log2_tok
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    omega = torch.randn(n_tok, generator=gen, device="cuda") * 1e-5
    mask = (torch.rand(n_tok, generator=gen, device="cuda") < masked_fraction).to(torch.uint8)
    pool = max(1, min(4, -(-3 * L2_BYTES // (n_tok * 4 * U))))
    rms = [torch.rand((U, n_tok), generator=gen, device="cuda") + 0.5 for _ in range(pool)]
    out = torch.zeros(U, device="cuda")
    nws = api.hilore_workspace_bytes(U, n_tok)
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    fns = [lambda i=i: api.hilore_unit_exposure(omega, mask, 1, n_tok, rms[i], U, n_tok, 0, 1e-8, out, None, ws, nws)
           for i in range(pool)]
    d = time_calls(fns, reps)
    t = d["loop_ms"]
    return {"kernel": "unit_exposure", "n_tok": n_tok, "U": U, "pool": pool, "us": t * 1e3, "device_us": d["device_us"],
            "host_us": d["host_us"], "gbs": n_tok * (5 + 4 * U) / t / 1e6}


def coeffs_packed_point(log2_tokens, reps, G=8, mean_len=2048):
    """The coefficient kernel on the packed layout: sequences of U{mean_len/2 .. 3 mean_len/2} tokens back to back."""
    import numpy as np
    n_tok = 1 << log2_tokens
    rng = np.random.default_rng(log2_tokens)
    lens = rng.integers(mean_len // 2, 3 * mean_len // 2 + 1, size=2 * n_tok // mean_len + 8)
    ends = np.cumsum(lens)
    ends = ends[: int(np.searchsorted(ends, n_tok)) + 1]
    ends[-1] = n_tok
    ends = np.concatenate([ends, np.full((-len(ends)) % G, n_tok)])      # empty sequences fill the last group
    n_seq = len(ends)
    cu = torch.from_numpy(np.concatenate([[0], ends]).astype(np.int32)).cuda()
    pool = max(1, min(8, -(-3 * L2_BYTES // (n_tok * 13))))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(3)
    lp = [torch.randn(n_tok, generator=gen, device="cuda") * 0.5 - 1.5 for _ in range(pool)]
    lo = [x + torch.randn(n_tok, generator=gen, device="cuda") * 0.05 for x in lp]
    mask = (torch.rand(n_tok, generator=gen, device="cuda") < 0.75).to(torch.uint8)
    rewards = (torch.rand(n_seq, generator=gen, device="cuda") < 0.5).float()
    adv = torch.empty(n_seq, device="cuda")
    omega = [torch.empty_like(x) for x in lp]
    fns = [lambda i=i: api.hilore_grpo_coeffs_packed(rewards, n_seq, G, 0, n_seq, cu, n_tok, lp[i], lo[i], None, mask, n_tok,
                                                     None, 0.2, 0.0, 1e-6, adv, omega[i], None, None) for i in range(pool)]
    tc = time_calls(fns, reps)
    t = tc["loop_ms"]
    return {"kernel": "grpo_coeffs_packed", "tokens": n_tok, "n_seq": n_seq, "pool": pool, "us": t * 1e3,
            "device_us": tc["device_us"], "host_us": tc["host_us"], "tokens_per_s": n_tok / t * 1e3, "gbs": 13 * n_tok / t / 1e6}


def diagnostics_point(log2_slots, reps, G=16, T=1024):
    """The omega diagnostics (cause counts + exact top-decile share) over one record of coefficients."""
    n_resp = max(G, (1 << log2_slots) // T)
    slots = n_resp * T
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2)
    lp = torch.randn((n_resp, T), generator=gen, device="cuda") * 0.5 - 1.5
    lo = lp + torch.randn((n_resp, T), generator=gen, device="cuda") * 0.15
    mask = (torch.rand((n_resp, T), generator=gen, device="cuda") < 0.8).to(torch.uint8)
    rewards = (torch.rand(n_resp, generator=gen, device="cuda") < 0.5).float()
    adv = torch.empty(n_resp, device="cuda")
    omega, ratio = torch.empty_like(lp), torch.empty_like(lp)
    api.hilore_grpo_coeffs(rewards, n_resp, G, 0, n_resp, T, lp, lo, None, mask, slots, None, 0.2, 0.0, 1e-6, adv, omega,
                           ratio, None)
    nws = api.hilore_omega_diagnostics_workspace_bytes()
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    counts = torch.zeros(5, dtype=torch.int64, device="cuda")
    share, total = torch.zeros(1, dtype=torch.float64, device="cuda"), torch.zeros(1, dtype=torch.float64, device="cuda")
    fn = lambda: api.hilore_omega_diagnostics(adv, ratio, mask, omega, n_resp, T, 0.2, counts, share, total, ws, nws)
    t = _time([fn], reps)
    # bytes the four sweeps read: 9 (ratio, mask, omega) + 3 x 5 (mask, omega) per slot
    return {"kernel": "omega_diagnostics", "slots": slots, "us": t * 1e3, "slots_per_s": slots / t * 1e3,
            "gbs": 24 * slots / t / 1e6, "zero_omega_fraction": counts[3].item() / slots, "top_decile_share": share.item()}


def allocate_point(U, reps, N=1024):
    """The DP allocator on the paper's grid: U units, synthetic utilities / memory costs / risks."""
    import numpy as np
    rng = np.random.default_rng(U)
    psi = torch.from_numpy(rng.uniform(0, 0.004, U).astype(np.float32)).cuda()
    dmem = np.zeros((U, 3))
    dmem[:, 1] = rng.uniform(20, 600, U)
    dmem[:, 2] = dmem[:, 1] * 0.53
    dtau = np.zeros((U, 3))
    dtau[:, 1] = rng.uniform(-0.5, 4.0, U)
    dtau[:, 2] = dtau[:, 1] - rng.uniform(0.05, 0.8, U)
    M_res, delta_b = float(dmem[:, 1].sum() * 0.35), float(psi.sum().item() * 0.3)
    dt, dm = torch.from_numpy(dtau).cuda(), torch.from_numpy(dmem).cuda()
    avail = torch.full((U,), api.ACT_H, dtype=torch.uint8, device="cuda")
    action = torch.zeros(U, dtype=torch.uint8, device="cuda")
    nws = api.hilore_allocate_workspace_bytes(U, N)
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    fn = lambda: api.hilore_allocate(U, psi, dt, dm, avail, M_res, delta_b, N, action, None, None, ws, nws)
    t = _time([fn], reps)
    return {"kernel": "allocate", "U": U, "N": N, "us": t * 1e3, "state_updates_per_s": U * (N + 1) ** 2 / t * 1e3,
            "workspace_mib": nws / 2 ** 20}


def plan_points(model="7B", rows=16384, layers=28, reps=5):
    """hilore_plan_apply over a whole microbatch table (3 units per layer) under different candidate plans: token RMS
    only (all H), capture of all units (all L), a 50 % L / 30 % H / 20 % R mix, post-forward encode of half the units."""
    dev = torch.device("cuda", torch.cuda.current_device())
    shapes = synth.layer_unit_shapes(model, rows, layers)
    U = len(shapes)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    x = [synth.activation_unit_device(gen, r, c, dev) for r, c in shapes]
    codes = [torch.empty((r, c), dtype=torch.uint8, device=dev) for r, c in shapes]
    scales = [torch.empty((r, c // 64), dtype=torch.float32, device=dev) for r, c in shapes]
    rms = torch.empty((U, rows), dtype=torch.float32, device=dev)
    units = [dict(x=x[i], codes=codes[i], scales=scales[i], out=None, row_rms=rms[i], rows=r, cols=c, fmt=api.FMT_E4M3FN_BLK,
                  block=64) for i, (r, c) in enumerate(shapes)]
    udev, uhost = api.make_unit_table(units, dev)
    H, L, R = api.ACT_H, api.ACT_L, api.ACT_R
    cases = (("capture, all H (token RMS only)", [H] * U, None), ("capture, all L", [L] * U, None),
             ("capture, 50% L / 30% H / 20% R", [(L, H, L, R, L, H, L, R, H, L)[i % 10] for i in range(U)], None),
             ("encode, every second H candidate assigned L", [H] * U, [(L, H)[i % 2] for i in range(U)]))
    out = []
    for name, q, a in cases:
        avail = torch.tensor(q, dtype=torch.uint8, device=dev)
        action = torch.tensor(a if a else q, dtype=torch.uint8, device=dev)
        phase = api.PHASE_ENCODE if a else api.PHASE_CAPTURE
        fn = lambda: api.hilore_plan_apply(udev, uhost, U, phase, None, None, None, 0, 0, avail, action, None, None, None)
        t = _time([fn], reps)
        nbytes = 0
        for i, (r, c) in enumerate(shapes):
            if a:
                nbytes += (r * c * 3 + r * c // 16) if a[i] == L else 0
            elif q[i] == L:
                nbytes += r * c * 3 + r * c // 16 + 4 * r
            elif q[i] == H:
                nbytes += r * c * 2 + 4 * r
        out.append({"kernel": "plan_apply", "table": f"{model} x {layers} layers x {rows} rows", "case": name, "ms": t,
                    "gbs": nbytes / t / 1e6})
    return out

# ---------------------------------------------------------------- small single-kernel cases (profiler captures)
def codec_case(rows, cols, fmt, reps, units, rms=True, codes_on=True, recover=True):
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


def coeffs_case(log2_slots, reps, beta=0.0, G=16, T=1024):
    n_resp = (1 << log2_slots) // T
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1)
    lp = torch.randn((n_resp, T), generator=gen, device="cuda") * 0.5 - 1.5
    lo = lp + torch.randn((n_resp, T), generator=gen, device="cuda") * 0.05
    lr = lp + torch.randn((n_resp, T), generator=gen, device="cuda") * 0.05 if beta else None
    mask = torch.ones((n_resp, T), dtype=torch.uint8, device="cuda")
    rewards = (torch.rand(n_resp, generator=gen, device="cuda") < 0.5).float()
    omega = torch.empty_like(lp)
    for _ in range(reps):
        api.hilore_grpo_coeffs(rewards, n_resp, G, 0, n_resp, T, lp, lo, lr, mask, n_resp * T, None, 0.2,
                               beta, 1e-6, None, omega, None, None)
    torch.cuda.synchronize()


def exposure_case(log2_tok, U, reps):
    n_tok = 1 << log2_tok
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    omega = torch.randn(n_tok, generator=gen, device="cuda") * 1e-5
    mask = (torch.rand(n_tok, generator=gen, device="cuda") < 0.8).to(torch.uint8)
    rms = torch.rand((U, n_tok), generator=gen, device="cuda") + 0.5
    out = torch.zeros(U, device="cuda")
    nws = api.hilore_workspace_bytes(U, n_tok)
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    for _ in range(reps):
        api.hilore_unit_exposure(omega, mask, 1, n_tok, rms, U, n_tok, 0, 1e-8, out, None, ws, nws)
    torch.cuda.synchronize()


class ScoreRefresh:
    """Inputs of one microbatch's score refresh (coefficients, exposure of U units, plan) at the 7B-shaped size: 16
    responses of 1024 tokens, 84 units; only the token RMS of the units is needed, not the units themselves."""

    def __init__(self, n_resp=16, T=1024, U=84, G=16):
        gen = torch.Generator(device="cuda")
        gen.manual_seed(9)
        self.n_resp, self.T, self.U, self.G = n_resp, T, U, G
        n_tok = n_resp * T
        self.lp = torch.randn((n_resp, T), generator=gen, device="cuda") * 0.5 - 1.5
        self.lo = self.lp + torch.randn((n_resp, T), generator=gen, device="cuda") * 0.05
        self.mask = (torch.rand((n_resp, T), generator=gen, device="cuda") < 0.9).to(torch.uint8)
        self.rewards = (torch.rand(n_resp, generator=gen, device="cuda") < 0.5).float()
        self.rms = torch.rand((U, n_tok), generator=gen, device="cuda") + 0.5
        self.omega = torch.empty((n_resp, T), device="cuda")
        self.exposure, self.psi = torch.zeros(U, device="cuda"), torch.zeros(U, device="cuda")
        self.kappa, self.ebar = torch.ones(U, device="cuda"), torch.full((U,), 0.03, device="cuda")
        self.avail = torch.full((U,), api.ACT_H, dtype=torch.uint8, device="cuda")
        self.action, self.recompute = torch.zeros(U, dtype=torch.uint8, device="cuda"), torch.zeros(U, dtype=torch.uint8, device="cuda")
        self.retained = torch.zeros(U, dtype=torch.int64, device="cuda")
        self.units_dev, self.units_host = api.make_unit_table(
            [dict(rows=n_tok, cols=3584 if i % 3 else 18944, fmt=api.FMT_E4M3FN_BLK, block=64) for i in range(U)], "cuda")
        self.ws_bytes = max(api.hilore_workspace_bytes(U, n_tok), api.hilore_scores_plan_workspace_bytes(U, n_tok))
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device="cuda")

    def one_launch(self):
        api.hilore_scores_plan(self.rewards, self.n_resp, self.G, 0, self.n_resp, self.T, self.lp, self.lo, None, self.mask,
                               self.n_resp * self.T, None, 0.2, 0.0, 1e-6, self.rms, self.U, self.n_resp * self.T, 0, 1e-8,
                               self.omega, self.exposure, None, self.units_dev, self.kappa, self.ebar, 1e-9, 1e-8, self.avail,
                               self.action, self.psi, self.recompute, self.retained, self.ws, self.ws_bytes)

    def separate_calls(self):
        api.hilore_coeffs_exposure(self.rewards, self.n_resp, self.G, 0, self.n_resp, self.T, self.lp, self.lo, None, self.mask,
                                   self.n_resp * self.T, None, 0.2, 0.0, 1e-6, self.rms, self.U, self.n_resp * self.T, 0, 1e-8,
                                   self.omega, self.exposure, None, self.ws, self.ws_bytes)
        api.hilore_plan_apply(self.units_dev, self.units_host, self.U, api.PHASE_DECIDE, self.exposure, self.kappa, self.ebar,
                              1e-9, 1e-8, self.avail, self.action, self.psi, self.recompute, self.retained)


def score_refresh_point(reps):
    """The score refresh of a 7B-shaped microbatch (16384 tokens, 84 units): one launch against the separate calls."""
    sr = ScoreRefresh()
    a, b = time_calls([sr.one_launch], reps), time_calls([sr.separate_calls], reps)
    return {"case": "score_refresh", "tokens": sr.n_resp * sr.T, "U": sr.U,
            "one_launch_us": a["loop_ms"] * 1e3, "one_launch_device_us": a["device_us"], "one_launch_host_us": a["host_us"],
            "separate_calls_us": b["loop_ms"] * 1e3, "separate_calls_device_us": b["device_us"],
            "separate_calls_host_us": b["host_us"]}


def score_refresh_case(reps):
    sr = ScoreRefresh()
    for _ in range(reps):
        sr.one_launch()
    torch.cuda.synchronize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--cols", type=int, default=4096)
    ap.add_argument("--min-log2-rows", type=int, default=7)
    ap.add_argument("--max-log2-rows", type=int, default=19)
    ap.add_argument("--fmts", type=int, nargs="*", default=[api.FMT_E4M3FN_RAW, api.FMT_E4M3FN_BLK])
    ap.add_argument("--shapes", type=str, default="", help="extra unit shapes, e.g. 8192x1536,8192x8960")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--no-coeffs", action="store_true")
    ap.add_argument("--no-rms", action="store_true", help="compress without the fused token RMS")
    ap.add_argument("--plan-table", action="store_true", help="only the 7B-shaped table under several candidate plans")
    ap.add_argument("--case", choices=["codec", "coeffs", "coeffs-packed", "exposure", "scores", "allocate", "relerr", "diagnostics"], help="run one small single-kernel case and exit")
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--fmt", type=int, default=api.FMT_E4M3FN_BLK)
    ap.add_argument("--units", type=int, default=2)
    ap.add_argument("--log2-slots", type=int, default=24)
    ap.add_argument("--beta", type=float, default=0.0)
    ap.add_argument("--U", type=int, default=12)
    ap.add_argument("--stats-only", action="store_true", help="--case codec: token RMS only, no codes")
    ap.add_argument("--no-recover", action="store_true")
    a = ap.parse_args()
    if a.case == "codec":
        codec_case(a.rows, a.cols, a.fmt, a.reps, a.units, rms=not a.no_rms, codes_on=not a.stats_only, recover=not a.no_recover)
    elif a.case == "coeffs":
        coeffs_case(a.log2_slots, a.reps, a.beta)
    elif a.case == "exposure":
        exposure_case(a.log2_slots, a.U, a.reps)
    elif a.case == "scores":
        score_refresh_case(a.reps)
    elif a.case == "coeffs-packed":
        print(json.dumps(coeffs_packed_point(a.log2_slots, a.reps)))
    elif a.case == "allocate":
        print(json.dumps(allocate_point(a.U, a.reps)))
    elif a.case == "relerr":
        print(json.dumps(relerr_point(a.rows, a.cols, a.fmt, a.reps)))
    elif a.case == "diagnostics":
        print(json.dumps(diagnostics_point(a.log2_slots, a.reps)))
    if a.case:
        print("done")
        return
    if a.plan_table:
        for p in plan_points():
            print(json.dumps(p), flush=True)
        return
    for fmt in a.fmts:
        for lr in range(a.min_log2_rows, a.max_log2_rows + 1):
            rows = 1 << lr
            reps = a.reps if rows * a.cols * 2 < (1 << 30) else max(3, a.reps // 4)
            print(json.dumps(codec_point(rows, a.cols, fmt, reps, with_rms=not a.no_rms)), flush=True)
            torch.cuda.empty_cache()
    for shp in [s for s in a.shapes.split(",") if s]:
        r, c = (int(v) for v in shp.split("x"))
        for fmt in a.fmts:
            print(json.dumps(codec_point(r, c, fmt, a.reps, with_rms=not a.no_rms)), flush=True)
            torch.cuda.empty_cache()
    if not a.no_coeffs:
        for ls in range(16, 25):
            for beta in (0.0, 1e-3):
                print(json.dumps(coeffs_point(ls, a.reps, beta=beta)), flush=True)
        for fmt in a.fmts:
            print(json.dumps(relerr_point(65536, 8960, fmt, a.reps)), flush=True)
        for ls, U in ((13, 84), (17, 84), (20, 84), (24, 12)):
            print(json.dumps(exposure_point(ls, U, a.reps)), flush=True)
        for ls in (15, 20, 24, 27):
            print(json.dumps(coeffs_packed_point(ls, a.reps)), flush=True)
        for ls in (20, 24, 27):
            print(json.dumps(diagnostics_point(ls, max(3, a.reps // 4))), flush=True)
        for U in (36, 84):
            print(json.dumps(allocate_point(U, max(3, a.reps // 4))), flush=True)
        print(json.dumps(score_refresh_point(a.reps)), flush=True)


if __name__ == "__main__":
    main()
