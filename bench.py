#!/usr/bin/env python
"""Benchmark of the HiLoRe hot path on B200: one step = the starred steps of Algorithm 1 for one
microbatch, through the C ABI.  The default workload is the largest single-GPU configuration, the
7B-shaped microbatch (84 saved units [16384, 3584|3584|18944] bf16, 24 GB): capture with the candidate
plan "all H" (token RMS of every unit), coefficients + exposure, risk scores and the threshold plan
(42 L / 25 H / 17 R), post-forward encoding of the L units, and their recovery.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2|3]

Prints ONE JSON line (rank 0).  `value` is the algorithmic HBM traffic of the timed steps divided by
their device-timed duration (inputs resident in HBM); `e2e` is the same with host buffers, the
host<->device copies inside the timed region; `roofline` is the compress kernel against the measured
HBM copy bandwidth; `sustained` repeats the step for at least two seconds with a clock record;
`kernels` carries the per-configuration legs (1.5B-shaped all-L step, 7B-shaped all-L capture, the
variable-length coefficient / exposure calls, the single-unit and coefficient end points of the
bandwidth sweep); `cpu_baseline` is the CPU oracle on a bounded sample of the same workload, on one
core and on all host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "compress+recover HBM GB/s (coeff tokens/s alongside); fraction of HBM roofline"
CONFIGS = {
    2: dict(model="1.5B", P=64, G=8, T=1024, mb_resp=8, layers=28, plan="all_L",
            workload="1.5B-shaped: 64 prompts x G=8 x 1024 tokens; microbatch of 8 responses (8192 token rows); "
                     "28 layers x (1536, 1536, 8960) bf16 units, all L, E4M3FN + fp32 scale per 64"),
    3: dict(model="7B", P=128, G=16, T=2048, mb_resp=8, layers=28, plan="mixed",
            workload="7B-shaped: 128 prompts x G=16 x 2048 tokens; microbatch of 8 responses (16384 token rows); "
                     "28 layers x (3584, 3584, 18944) bf16 units; candidate plan all H, threshold plan 42 L / 25 H / 17 R "
                     "per microbatch; capture (token RMS) -> coefficients + exposure -> decide -> encode L -> recover L; "
                     "E4M3FN + fp32 scale per 64"),
}
DEFAULT_CONFIG = 3
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) per algorithmic byte of the codec kernels, from profiler captures of one 7B-shaped
# unit [16384, 18944] (five times the L2; summarised under profiles/; traffic grows in proportion to the
# elements processed, every element being read once and written once).  Reads match the algorithmic reads; a
# few percent of the written bytes are still dirty in L2 when such a single-unit kernel ends.
DRAM_PER_ALGORITHMIC = {"compress": (620.847616 + 296.770048) / 950.6,   # codes + scales + token RMS
                        "encode": (620.838400 + 288.768000) / 950.5,     # codes + scales
                        "stats": (620.841728 + 3.612672) / 620.8,        # token RMS only
                        "recover": (329.943552 + 562.304512) / 950.5}


# ---------------------------------------------------------------- accounting (bytes the method must move)
def codec_bytes(rows, cols, fmt_scaled=True, with_rms=False):
    n = rows * cols
    return 3 * n + (4 * n // 64 if fmt_scaled else 0) + (4 * rows if with_rms else 0)


def stats_bytes(rows, cols):
    return 2 * rows * cols + 4 * rows


def coeff_bytes(slots, with_ref=False, extras=False):
    return slots * (13 + (4 if with_ref else 0) + (5 if extras else 0))


def exposure_bytes(n_tok, U):
    return n_tok * (5 + 4 * U)


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def fractions(gbs, peak):
    return {"gbs": gbs, "frac_measured": gbs / peak, "frac_nominal": gbs / NOMINAL_HBM_GBS}


# ---------------------------------------------------------------- clocks during the timed region (read only)
class ClockSampler:
    """Samples SM clock, power and the throttle reasons of one GPU while a region runs: through NVML from a
    thread (a few milliseconds per sample), else through an `nvidia-smi` child.  Nothing is ever set."""
    SMI_FIELDS = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown," \
                 "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown," \
                 "clocks_event_reasons.sw_power_cap"

    def __init__(self, cuda_index: int, period_s: float = 0.01):
        self.cuda_index, self.period = cuda_index, period_s
        self.rows, self.proc, self.thread, self.stop_flag, self.how = [], None, None, False, None
        self.nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(cuda_index)
            try:
                bus = "%08x:%02x:%02x.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
                self.handle = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
        except Exception:
            self.nvml = None

    def _nvml_loop(self):
        nv = self.nvml
        bits = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))
        while not self.stop_flag:
            try:
                sm = float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                try:
                    power = nv.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
                except Exception:
                    power = None
                self.rows.append((sm, self.max_sm, power, [n for n, b in bits if reasons & b]))
            except Exception:
                pass
            time.sleep(self.period)

    def _smi_read(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.proc.stdout:
            r = [f.strip() for f in line.split(",")]
            if len(r) < 7:
                continue
            try:
                self.rows.append((float(r[0]), float(r[1]), float(r[2]) if r[2].replace(".", "").isdigit() else None,
                                  [n for n, v in zip(names, r[3:7]) if v.lower().startswith("active")]))
            except ValueError:
                continue

    def start(self):
        self.rows, self.stop_flag = [], False
        if self.nvml is not None:
            self.how = "nvml"
            self.thread = threading.Thread(target=self._nvml_loop, daemon=True)
            self.thread.start()
            return
        try:
            self.how = "nvidia-smi"
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.cuda_index), f"--query-gpu={self.SMI_FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._smi_read, daemon=True).start()
        except Exception:
            self.proc = None

    def stop(self):
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            self.thread = None
        elif self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.proc = None
        else:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["no clock source"]}
        sm = [r[0] for r in self.rows]
        power = [r[2] for r in self.rows if r[2] is not None]
        reasons = sorted({n for r in self.rows for n in r[3]})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(r[1] for r in self.rows) if self.rows else None, "samples": len(sm),
                "power_w_max": max(power) if power else None, "reasons": reasons, "source": self.how}


# ---------------------------------------------------------------- the workload on one GPU
class Workload:
    """Device-resident state of one data-parallel rank: the rollout batch's log-probabilities and one
    microbatch pool of activation units (reused across microbatches; far larger than L2)."""

    def __init__(self, api, synth, cfg, seed: int, device, with_out=True):
        self.api, self.device, self.cfg = api, device, cfg
        P, G_, T = cfg["P"], cfg["G"], cfg["T"]
        self.G, self.T, self.mb_resp = G_, T, cfg["mb_resp"]
        ro = synth.rollout(seed, P, G_, T)
        self.ro = ro
        self.n_resp = ro.n_resp
        self.rewards = torch.from_numpy(ro.rewards).to(device)
        self.logp_new = torch.from_numpy(ro.logp_new).to(device)
        self.logp_old = torch.from_numpy(ro.logp_old).to(device)
        self.mask = torch.from_numpy(ro.mask).to(device)
        self.n_microbatches = self.n_resp // self.mb_resp
        self.rows = self.mb_resp * T
        self.shapes = synth.layer_unit_shapes(cfg["model"], self.rows, cfg["layers"])
        self.U = U = len(self.shapes)
        gen = torch.Generator(device=device)
        gen.manual_seed(seed)
        self.x = [synth.activation_unit_device(gen, r, c, device) for r, c in self.shapes]
        self.codes = [torch.empty((r, c), dtype=torch.uint8, device=device) for r, c in self.shapes]
        self.scales = [torch.empty((r, c // 64), dtype=torch.float32, device=device) for r, c in self.shapes]
        self.out = [torch.empty((r, c), dtype=torch.bfloat16, device=device) for r, c in self.shapes] if with_out else [None] * U
        self.rms = torch.empty((U, self.rows), dtype=torch.float32, device=device)
        units = [dict(x=self.x[i], codes=self.codes[i], scales=self.scales[i], out=self.out[i], row_rms=self.rms[i],
                      rows=r, cols=c, fmt=api.FMT_E4M3FN_BLK, block=64) for i, (r, c) in enumerate(self.shapes)]
        self.units_dev, self.units_host = api.make_unit_table(units, device)
        self.mixed = cfg["plan"] == "mixed"
        q = api.ACT_H if self.mixed else api.ACT_L     # candidate plan
        self.avail = torch.full((U,), q, dtype=torch.uint8, device=device)
        self.action = torch.zeros(U, dtype=torch.uint8, device=device)
        self.recompute = torch.zeros(U, dtype=torch.uint8, device=device)
        self.retained = torch.zeros(U, dtype=torch.int64, device=device)
        self.psi = torch.zeros(U, dtype=torch.float32, device=device)
        self.exposure = torch.zeros(U, dtype=torch.float32, device=device)
        kgen = np.random.default_rng(seed + 1)
        self.kappa = torch.from_numpy(kgen.uniform(0.5, 2.0, U).astype(np.float32)).to(device)
        self.ebar = torch.full((U,), 0.025, dtype=torch.float32, device=device)
        self.omega = torch.empty((self.mb_resp, T), dtype=torch.float32, device=device)
        self.ws_bytes = api.hilore_scores_plan_workspace_bytes(U, self.rows)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=device)
        self.n_valid = ro.n_valid
        self.elements = sum(r * c for r, c in self.shapes)
        self.bytes_coeffs = coeff_bytes(self.rows)
        self.bytes_exposure = exposure_bytes(self.rows, U)
        self.bytes_decide = 13 * U
        inf = float("inf")
        if self.mixed:
            self.bytes_capture = sum(stats_bytes(r, c) for r, c in self.shapes)
            self.n_plan = min(self.n_microbatches, 64)          # microbatches the steps rotate through
            self.tau = [(inf, inf)] * self.n_plan                  # filled by prepare_plan()
            self.bytes_encode = [0] * self.n_plan
            self.bytes_recover = [0] * self.n_plan
            self.expected_action = [None] * self.n_plan
            self.launches_per_step = 4   # capture, scores + plan, encode, recover
        else:
            self.bytes_capture = sum(codec_bytes(r, c, True, True) for r, c in self.shapes)
            self.n_plan = self.n_microbatches
            self.tau = [(inf, inf)] * self.n_plan
            self.bytes_encode = [0] * self.n_plan
            self.bytes_recover = [sum(codec_bytes(r, c, True, False) for r, c in self.shapes)] * self.n_plan
            self.launches_per_step = 3   # capture, scores + plan, recover

    def bytes_step(self, mb):
        mb %= self.n_plan
        return (self.bytes_capture + self.bytes_coeffs + self.bytes_exposure + self.bytes_decide
                + self.bytes_encode[mb] + self.bytes_recover[mb])

    # ---- the calls of a step
    def capture(self):
        a = self.api
        a.hilore_plan_apply(self.units_dev, self.units_host, self.U, a.PHASE_CAPTURE, None, None, None, 0.0, 0.0,
                            self.avail, self.action, None, None, None)

    def scores(self, mb):
        a = self.api
        sl = slice(mb * self.mb_resp, (mb + 1) * self.mb_resp)
        a.hilore_coeffs_exposure(self.rewards, self.n_resp, self.G, mb * self.mb_resp, self.mb_resp, self.T, self.logp_new[sl],
                                 self.logp_old[sl], None, self.mask[sl], self.n_valid, None, 0.2, 0.0, 1e-6, self.rms,
                                 self.U, self.rows, 0, 1e-8, self.omega, self.exposure, None, self.ws, self.ws_bytes)

    def scores_plan(self, mb, tau_lo, tau_hi):
        a = self.api
        sl = slice(mb * self.mb_resp, (mb + 1) * self.mb_resp)
        a.hilore_scores_plan(self.rewards, self.n_resp, self.G, mb * self.mb_resp, self.mb_resp, self.T, self.logp_new[sl],
                             self.logp_old[sl], None, self.mask[sl], self.n_valid, None, 0.2, 0.0, 1e-6, self.rms, self.U,
                             self.rows, 0, 1e-8, self.omega, self.exposure, None, self.units_dev, self.kappa, self.ebar, tau_lo,
                             tau_hi, self.avail, self.action, self.psi, self.recompute, self.retained, self.ws, self.ws_bytes)

    def decide(self, tau_lo, tau_hi):
        a = self.api
        a.hilore_plan_apply(self.units_dev, self.units_host, self.U, a.PHASE_DECIDE, self.exposure, self.kappa,
                            self.ebar, tau_lo, tau_hi, self.avail, self.action, self.psi, self.recompute, self.retained)

    def encode(self):
        a = self.api
        a.hilore_plan_apply(self.units_dev, self.units_host, self.U, a.PHASE_ENCODE, None, None, None, 0.0, 0.0,
                            self.avail, self.action, None, None, None)

    def recover(self):
        a = self.api
        a.hilore_plan_apply(self.units_dev, self.units_host, self.U, a.PHASE_RECOVER, None, None, None, 0.0, 0.0,
                            self.avail, self.action, None, None, None)

    def prepare_plan(self):
        """Thresholds of the mixed plan, once per microbatch the steps rotate through (outside every timed
        region): psi of the microbatch from the library's own calls, tau_lo / tau_hi at the midpoints between the
        order statistics that split the units 50 % L (lowest risk) / 30 % H (highest) / 20 % R."""
        if not self.mixed:
            return
        api, U = self.api, self.U
        self.capture()
        psi_all = torch.empty((self.n_plan, U), dtype=torch.float32, device=self.device)
        for mb in range(self.n_plan):
            self.scores(mb)
            self.decide(float("inf"), float("inf"))
            psi_all[mb].copy_(self.psi)
        psi_h = psi_all.cpu().numpy()
        n_L, n_H = U // 2, (3 * U) // 10
        for mb in range(self.n_plan):
            p = psi_h[mb]
            srt = np.sort(p)
            lo = float((np.float64(srt[n_L - 1]) + np.float64(srt[n_L])) / 2)
            hi = float((np.float64(srt[U - n_H - 1]) + np.float64(srt[U - n_H])) / 2)
            lo32, hi32 = float(np.float32(lo)), float(np.float32(hi))
            act = np.where(p < np.float32(lo32), api.ACT_L, np.where(p >= np.float32(hi32), api.ACT_H, api.ACT_R)).astype(np.uint8)
            self.tau[mb] = (lo32, hi32)
            self.expected_action[mb] = act
            sel = [i for i in range(U) if act[i] == api.ACT_L]
            self.bytes_encode[mb] = sum(codec_bytes(*self.shapes[i], True, False) for i in sel)
            self.bytes_recover[mb] = self.bytes_encode[mb]

    def step(self, mb: int, ev=None):
        """One microbatch.  all-L plan: capture (compress every unit + token RMS), coefficients + exposure, risk +
        gating, recover.  Mixed plan: capture (token RMS, bf16 kept), coefficients + exposure, risk + thresholds,
        post-forward encoding of the units assigned L, their recovery.  `ev`: optional event pairs per phase."""
        mb %= self.n_plan
        rec = (lambda k, i: ev[k][i].record()) if ev is not None else (lambda k, i: None)
        rec("capture", 0)
        self.capture()
        rec("capture", 1)
        rec("scores", 0)   # coefficients, their reduction to exposure scores and the plan: one launch
        self.scores_plan(mb, *self.tau[mb])
        rec("scores", 1)
        if self.mixed:
            rec("encode", 0)
            self.encode()
            rec("encode", 1)
        rec("recover", 0)
        self.recover()
        rec("recover", 1)

    @property
    def kinds(self):
        return ("capture", "scores", "encode", "recover") if self.mixed else ("capture", "scores", "recover")


def time_steps(wl, first_mb, steps, barrier, with_events=True):
    """`steps` steps bracketed by barrier + synchronize on both sides; returns (ms in total, ms per phase and step)."""
    evs = [{k: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for k in wl.kinds}
           for _ in range(steps)] if with_events else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(steps):
        wl.step(first_mb + i, evs[i] if evs else None)
    e1.record()
    barrier()
    kern = {k: sum(e[k][0].elapsed_time(e[k][1]) for e in evs) / steps for k in wl.kinds} if evs else {}
    return e0.elapsed_time(e1), kern


# ---------------------------------------------------------------- per-configuration legs (kernels alone)
def config_legs(api, synth, device, peak, wl3=None):
    import bench_sweep as sw
    legs = {}

    def put(name, d, gbs_key="gbs"):
        d = dict(d)
        d.update({k: v for k, v in fractions(d[gbs_key], peak).items() if k != "gbs"})
        legs[name] = d

    # config 3: capture with every unit a candidate for L (codes + scales + token RMS of all 84 units)
    if wl3 is not None and wl3.mixed:
        wl3.avail.fill_(api.ACT_L)
        nb = sum(codec_bytes(r, c, True, True) for r, c in wl3.shapes)
        ms = sw.time_calls([wl3.capture], 3, warm=1)["loop_ms"]
        wl3.avail.fill_(api.ACT_H)
        put("cfg3_all_L_capture", {"ms": ms, "gbs": nb / ms / 1e6, "bytes": nb})
    # config 2: the 1.5B-shaped all-L step
    wl2 = Workload(api, synth, CONFIGS[2], seed=0, device=device)
    for i in range(3):
        wl2.step(i)
    ms, kern = time_steps(wl2, 3, 10, torch.cuda.synchronize)
    put("cfg2_compress", {"ms": kern["capture"], "gbs": wl2.bytes_capture / kern["capture"] / 1e6})
    put("cfg2_recover", {"ms": kern["recover"], "gbs": wl2.bytes_recover[0] / kern["recover"] / 1e6})
    put("cfg2_step", {"ms": ms / 10, "gbs": wl2.bytes_step(0) / (ms / 10) / 1e6, "scores_decide_us": kern["scores"] * 1e3})
    del wl2
    torch.cuda.empty_cache()
    # config 4: variable-length rollout batch, masked coefficients over all 8.39 M slots; exposure of one microbatch
    ro = synth.rollout(0, 256, 8, 4096, rewards="uniform", lengths="uniform", equal_group_fraction=0.05)
    d = sw.coeffs_rollout_point(ro, 10)
    d["gbs_padding_skipped_bound"] = (5 * d["slots"] + 8 * ro.n_valid) / d["us"] / 1e3
    put("cfg4_masked_coeffs", d)
    legs["cfg4_masked_exposure_16384tok_84units"] = sw.exposure_point(14, 84, 20, masked_fraction=0.52)
    del ro
    # config 5: end points of the bandwidth sweep
    for name, lr in (("64MiB", 13), ("512MiB", 16), ("4GiB", 19)):
        for fname, fmt in (("RAW", api.FMT_E4M3FN_RAW), ("BLK", api.FMT_E4M3FN_BLK)):
            p = sw.codec_point(1 << lr, 4096, fmt, 20 if lr < 19 else 5)
            put(f"cfg5_unit_{name}_{fname}_compress", {"us": p["compress_us"], "gbs": p["compress_gbs"],
                                                        "device_us": p["compress_device_us"], "host_us": p["compress_host_us"]})
            put(f"cfg5_unit_{name}_{fname}_recover", {"us": p["recover_us"], "gbs": p["recover_gbs"],
                                                       "device_us": p["recover_device_us"], "host_us": p["recover_host_us"]})
            torch.cuda.empty_cache()
    for ls in (16, 20, 24):
        for bname, beta in (("beta0", 0.0), ("beta1e-3", 1e-3)):
            put(f"cfg5_coeffs_2p{ls}_{bname}", sw.coeffs_point(ls, 20, beta=beta))
    alloc = sw.allocate_point(84, 5)      # the paper's DP allocator on its 1025 x 1025 grid (not part of the step)
    legs["allocate_dp_u84_n1024"] = {"ms": alloc["us"] / 1e3, "state_updates_per_s": alloc["state_updates_per_s"]}
    return legs


# ---------------------------------------------------------------- CPU oracle legs
REFERENCE_BUDGET_S = 120.0     # the whole `--impl reference` run is sized to end within about this time


def oracle_sample_step(synth_mod, cfg, seed=0, rows=None, threads=1, inputs=None):
    """The oracle on a bounded sample of the workload: the first `rows` token rows of layer 0's three units of one
    microbatch, through the steps of the workload's plan (mixed: token RMS of the three units, coefficients of
    those slots, exposure, plan, compress + recover of the two units assigned L; all-L: compress with token RMS and
    recover of all three), `threads` > 1: the same calls over row ranges on a thread pool (the oracle's C
    functions are called as they stand; ctypes releases the interpreter lock during a call).
    Returns (seconds, algorithmic bytes of the sample, inputs)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    T, G_ = cfg["T"], cfg["G"]
    rows = cfg["mb_resp"] * T if rows is None else rows
    shapes = synth_mod.layer_unit_shapes(cfg["model"], rows, 1)
    if inputs is None:
        rng = np.random.default_rng(seed)
        xs = [synth_mod.activation_unit(rng, r, c) for r, c in shapes]
        n_rows = max(1, rows // T)                      # responses the sampled token rows belong to
        t_len = min(T, rows)
        ro = synth_mod.rollout(seed, max(1, -(-n_rows // G_)), G_, t_len)
        inputs = (xs, ro, n_rows, t_len)
    xs, ro, n_rows, t_len = inputs
    mixed = cfg["plan"] == "mixed"
    L_units = [0, 2] if mixed else [0, 1, 2]
    oracle.lib()
    pool = ThreadPoolExecutor(threads) if threads > 1 else None

    def over_rows(fn, n, *arrays):
        """fn over row ranges of the arrays (rows are independent), results concatenated in order."""
        if pool is None:
            return fn(*arrays)
        cuts = [n * i // threads for i in range(threads + 1)]
        parts = list(pool.map(lambda ab: fn(*[a[ab[0]:ab[1]] for a in arrays]), zip(cuts[:-1], cuts[1:])))
        if isinstance(parts[0], tuple):
            return tuple(np.concatenate([p[i] for p in parts]) if parts[0][i] is not None else None for i in range(len(parts[0])))
        return np.concatenate(parts)

    t0 = time.perf_counter()
    rms = [over_rows(oracle.row_rms, rows, x) for x in xs]
    adv = oracle.group_advantages(ro.rewards, G_)
    omega = over_rows(lambda a, ln, lo, mk: oracle.grpo_coeffs(a, ln, lo, None, mk, N_norm=cfg["P"] * G_ * T)[0], n_rows,
                      adv[:n_rows], ro.logp_new[:n_rows], ro.logp_old[:n_rows], ro.mask[:n_rows])
    E, _ = oracle.unit_exposure(np.ascontiguousarray(omega), np.ascontiguousarray(ro.mask[:n_rows]),
                                np.ascontiguousarray(np.stack(rms)[:, :n_rows * t_len]))
    for i in L_units:
        codes, scales = over_rows(lambda x: oracle.compress(x, oracle.FMT_E4M3FN_BLK, 64), rows, xs[i])
        over_rows(lambda c, s: oracle.recover(c, s, oracle.FMT_E4M3FN_BLK, 64), rows, codes, scales)
    dt = time.perf_counter() - t0
    if pool is not None:
        pool.shutdown()
    if mixed:
        nbytes = sum(stats_bytes(r, c) for r, c in shapes) + 2 * sum(codec_bytes(*shapes[i], True, False) for i in L_units)
    else:
        nbytes = sum(codec_bytes(r, c, True, True) + codec_bytes(r, c, True, False) for r, c in shapes)
    nbytes += coeff_bytes(n_rows * t_len) + exposure_bytes(n_rows * t_len, len(shapes))
    return dt, nbytes, inputs


def sample_text(cfg, rows):
    w = {"1.5B": "[.,1536]x2 + [.,8960]", "7B": "[.,3584]x2 + [.,18944]"}[cfg["model"]]
    what = ("token RMS of the three units, compress + recover of the two assigned L" if cfg["plan"] == "mixed"
            else "compress with token RMS + recover of the three units")
    return (f"first {rows} of {cfg['mb_resp'] * cfg['T']} token rows of layer 0's units ({w}) of one microbatch: {what}, the "
            f"coefficients of those {rows} slots, exposure U=3")


def run_reference(args):
    """The tier's reference arm: the CPU oracle, as it stands, on the host cores.  Each step is a bounded
    sample of the workload, sized from a short calibration so that warm-up + timed steps end within about two
    minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_33570_b200 import synth
    cfg = CONFIGS[args.config]
    cal_rows = 256
    oracle_sample_step(synth, cfg, seed=12344, rows=64)          # loads the library, touches the allocator
    w0 = time.perf_counter()
    oracle_sample_step(synth, cfg, seed=12345, rows=cal_rows)
    rows_per_s = cal_rows / max(time.perf_counter() - w0, 1e-6)        # wall clock: input generation included
    budget = REFERENCE_BUDGET_S / max(1, args.steps + args.warmup)
    rows = int(min(cfg["mb_resp"] * cfg["T"], max(64, rows_per_s * budget * 0.8)))
    rows -= rows % 64
    times = []
    nbytes = 0
    for i in range(args.warmup + args.steps):
        dt, nbytes, _ = oracle_sample_step(synth, cfg, seed=i, rows=rows)
        if i >= args.warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    val = nbytes / sec / 1e9
    sample = sample_text(cfg, rows)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16->e4m3fn (fp32 scales, fp64 oracle arithmetic)", "data": "synthetic",
        "config": {"workload": cfg["workload"], "sample_per_step": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
                         "nproc": os.cpu_count()},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(synth, cfg):
    """The oracle on one core and on all host cores, same sample (about 10-30 s of CPU work on one core)."""
    rows = cfg["mb_resp"] * cfg["T"]
    oracle_sample_step(synth, cfg, seed=1, rows=64)
    dt1, nb, inputs = oracle_sample_step(synth, cfg, seed=0, rows=rows)
    nproc = os.cpu_count() or 1
    out = {"value": nb / dt1 / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "seconds": dt1, "nproc": nproc,
           "sample": sample_text(cfg, rows)}
    if nproc > 1:
        dtn, _, _ = oracle_sample_step(synth, cfg, rows=rows, threads=nproc, inputs=inputs)
        out["all_cores"] = {"value": nb / dtn / 1e9, "unit": "GB/s", "cores": nproc, "seconds": dtn,
                            "how": "the same oracle calls over row / response ranges on a thread pool"}
    return out


# ---------------------------------------------------------------- main (our arm)
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG, choices=sorted(CONFIGS))
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the per-configuration kernel legs")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustain-s", type=float, default=2.0, help="length of the sustained leg (0 = skip)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        args.warmup = 3

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    from paper_2609_33570_b200 import api, dist as hdist, synth

    cfg = CONFIGS[args.config]
    wl = Workload(api, synth, cfg, seed=rank, device=device)
    # batch-wide normaliser N: the one exchange of the path (once per update, outside the microbatch step)
    local_count = torch.zeros(1, dtype=torch.int64, device=device)
    api.hilore_mask_count(wl.mask, wl.mask.numel(), local_count)
    n_global = hdist.global_token_count(local_count) if world > 1 else int(local_count.item())
    wl.n_valid = n_global
    wl.prepare_plan()
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        wl.step(i)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_total, kern_ms = time_steps(wl, args.warmup, args.steps, barrier)
    clocks = sampler.stop() if rank == 0 else None
    t = torch.tensor([ms_total], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_step = float(t.item()) / args.steps
    bytes_timed = sum(wl.bytes_step(args.warmup + i) for i in range(args.steps))
    plan_ok = True
    if wl.mixed:   # the last step's decisions are the ones the thresholds were derived for
        last = (args.warmup + args.steps - 1) % wl.n_plan
        plan_ok = bool(np.array_equal(wl.action.cpu().numpy(), wl.expected_action[last]))

    # sustained: the same step for at least `sustain_s` seconds, with its own clock record
    sustained = None
    if args.sustain_s > 0:
        n_sus = max(args.steps, int(math.ceil(1.1 * args.sustain_s * 1e3 / ms_step)))
        if rank == 0:
            sampler.start()
        ms_sus, _ = time_steps(wl, 0, n_sus, barrier, with_events=False)
        sus_clocks = sampler.stop() if rank == 0 else None
        ts = torch.tensor([ms_sus], dtype=torch.float64, device=device)
        if world > 1:
            dist.all_reduce(ts, op=dist.ReduceOp.MAX)
        b_sus = sum(wl.bytes_step(i) for i in range(n_sus))
        sustained = {"steps": n_sus, "seconds": float(ts.item()) / 1e3, "value": world * b_sus / float(ts.item()) / 1e6,
                     "unit": "GB/s", "ms_per_step": float(ts.item()) / n_sus, "clocks": sus_clocks}
        if sus_clocks and sus_clocks.get("sm_mhz"):
            sustained["ms_per_step_x_sm_mhz"] = sustained["ms_per_step"] * sus_clocks["sm_mhz"]

    # end to end: host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        # pinned host copies of one layer's units (the 28 layers' device units are refilled from them: the same
        # bytes cross PCIe as from 28 distinct host buffers, without pinning 24 GB of host memory)
        per_layer = len(wl.shapes) // cfg["layers"]
        hx = [torch.empty(wl.x[j].shape, dtype=wl.x[j].dtype, pin_memory=True).copy_(wl.x[j]) for j in range(per_layer)]
        h_ln, h_lo, h_mk = (torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for v in
                            (wl.logp_new, wl.logp_old, wl.mask))
        outs = (("exposure", wl.exposure), ("psi", wl.psi), ("action", wl.action), ("retained", wl.retained))
        h_out = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in outs}
        h2d = sum(x.numel() * x.element_size() for x in wl.x) + wl.rows * 9
        d2h = sum(v.numel() * v.element_size() for v in h_out.values())

        def e2e_step(mb):
            sl = slice(mb * wl.mb_resp, (mb + 1) * wl.mb_resp)
            for j, x in enumerate(wl.x):
                x.copy_(hx[j % per_layer], non_blocking=True)
            wl.logp_new[sl].copy_(h_ln[sl], non_blocking=True)
            wl.logp_old[sl].copy_(h_lo[sl], non_blocking=True)
            wl.mask[sl].copy_(h_mk[sl], non_blocking=True)
            wl.step(mb)
            for k, v in outs:
                h_out[k].copy_(v, non_blocking=True)
            torch.cuda.current_stream().synchronize()

        e2e_step(0)
        barrier()
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            e2e_step(i % wl.n_plan)
        barrier()
        dt = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device=device)
        if world > 1:
            dist.all_reduce(dt, op=dist.ReduceOp.MAX)
        e2e_s = float(dt.item()) / args.e2e_steps
        b_e2e = sum(wl.bytes_step(i % wl.n_plan) for i in range(args.e2e_steps)) / args.e2e_steps
        e2e = {"value": world * b_e2e / e2e_s / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3, "steps": args.e2e_steps}
        del hx

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = peak_hbm()
    b_enc = sum(wl.bytes_encode[(args.warmup + i) % wl.n_plan] for i in range(args.steps)) / args.steps
    b_rec = sum(wl.bytes_recover[(args.warmup + i) % wl.n_plan] for i in range(args.steps)) / args.steps

    def roof(kernel, launches):
        """launches: [(algorithmic bytes, ms, DRAM-per-algorithmic ratio)] of one step's launches of this kernel."""
        nb = sum(l[0] for l in launches) / len(launches)
        ms = sum(l[1] for l in launches) / len(launches)
        achieved = nb / ms / 1e6
        return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}",
                "unit": "GB/s", "frac": achieved / peak, "frac_of_8000_nominal": achieved / NOMINAL_HBM_GBS,
                "launches_per_step": len(launches), "algorithmic_bytes_per_launch": nb, "ms_per_launch": ms,
                "traffic": sum(l[0] * l[2] for l in launches) / len(launches)}

    kernels = {}
    if wl.mixed:
        roofline = roof("compress_kernel<E4M3FN_BLK>: two launches per step, each over the 84-unit table (capture = token RMS of "
                        "all units, 2 B/element; encode = codes + scales of the units assigned L, 3.0625 B/element)",
                        [(wl.bytes_capture, kern_ms["capture"], DRAM_PER_ALGORITHMIC["stats"]),
                         (b_enc, kern_ms["encode"], DRAM_PER_ALGORITHMIC["encode"])])
        kernels["capture_token_rms"] = {"ms": kern_ms["capture"], **fractions(wl.bytes_capture / kern_ms["capture"] / 1e6, peak)}
        kernels["encode_L_units"] = {"ms": kern_ms["encode"], **fractions(b_enc / kern_ms["encode"] / 1e6, peak)}
    else:
        roofline = roof("compress_kernel<E4M3FN_BLK> (one launch covers the 84 units)",
                        [(wl.bytes_capture, kern_ms["capture"], DRAM_PER_ALGORITHMIC["compress"])])
        kernels["compress"] = {"ms": kern_ms["capture"], **fractions(wl.bytes_capture / kern_ms["capture"] / 1e6, peak)}
    roofline_recover = roof("recover_kernel<E4M3FN_BLK> (one launch over the 84-unit table, L units decoded)",
                            [(b_rec, kern_ms["recover"], DRAM_PER_ALGORITHMIC["recover"])])
    kernels["recover_L_units" if wl.mixed else "recover"] = {"ms": kern_ms["recover"], **fractions(b_rec / kern_ms["recover"] / 1e6, peak)}
    kernels["scores_decide_microbatch"] = {"us": kern_ms["scores"] * 1e3, "tokens_per_s": wl.rows / kern_ms["scores"] * 1e3,
                                           "launches": 1}
    out = {
        "metric": METRIC, "value": world * bytes_timed / (ms_step * args.steps) / 1e6, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16->e4m3fn codes (fp32 scales, fp32 coefficients)",
        "data": "synthetic",
        "config": {"workload": cfg["workload"], "config_index": args.config,
                   "l2": f"inputs larger than L2 ({wl.elements * 2 / 1e9:.1f} GB of units per step)",
                   "units": wl.U, "elements_per_step": wl.elements, "bytes_per_step": bytes_timed / args.steps,
                   "plan_matches_thresholds": plan_ok,
                   "parallelism": f"dp{world} (microbatches sharded, no data-path collective)"},
        "gpu_launches": wl.launches_per_step * args.steps,
        "clocks": clocks,
        "roofline": roofline,
        "roofline_recover": roofline_recover,
        "sustained": sustained,
        "kernels": kernels,
        "e2e": e2e,
    }
    if world == 1 and not args.no_legs:
        kernels.update(config_legs(api, synth, device, peak, wl))
        if "cfg5_coeffs_2p24_beta0" in kernels:
            out["coeff_tokens_per_s"] = kernels["cfg5_coeffs_2p24_beta0"]["tokens_per_s"]
    del wl
    torch.cuda.empty_cache()
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(synth, cfg)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
