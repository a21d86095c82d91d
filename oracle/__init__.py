"""ctypes front end of the CPU oracle (oracle/hilore_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the product path never does.  It compiles the C file with gcc on first use
(``-O2 -ffp-contract=off``: no fused multiply-add, so every fp32 product is rounded once)
and marshals NumPy arrays in and out.  bf16 tensors are ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hilore_oracle.c")
_LIB = os.path.join(_HERE, "libhilore_oracle.so")

FMT_E4M3FN_RAW, FMT_E4M3FN_BLK, FMT_INT8_BLK = 0, 1, 2
ACT_R, ACT_H, ACT_L = 0, 1, 2
OK, INVALID, SHAPE, ZERO_NORM = 0, 1, 2, 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_grpo_objective.restype = C.c_double
        _lib.orc_relative_error.restype = C.c_double
        _lib.orc_risk_budget.restype = C.c_double
        _lib.orc_fit_kappa.restype = C.c_double
    return _lib


def _p(a, dtype):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(C.c_void_p)


class OracleError(RuntimeError):
    def __init__(self, status):
        super().__init__(f"oracle status {status}")
        self.status = status


def _check(st):
    if st != OK:
        raise OracleError(st)


def group_advantages(rewards: np.ndarray, G: int, adv_eps: float = 1e-6) -> np.ndarray:
    rewards = np.ascontiguousarray(rewards, dtype=np.float32)
    adv = np.empty_like(rewards)
    _check(lib().orc_group_advantages(_p(rewards, np.float32), C.c_int64(rewards.size), C.c_int32(G),
                                      C.c_float(adv_eps), _p(adv, np.float32)))
    return adv


def grpo_coeffs(adv_rows, logp_new, logp_old, logp_ref, mask, N_norm=0, clip_eps=0.2, beta=0.0):
    """-> (omega, ratio, clip_mask) for rows whose advantages are adv_rows."""
    n_rows, T = logp_new.shape
    adv_rows = np.ascontiguousarray(adv_rows, dtype=np.float32)
    assert adv_rows.size == n_rows
    omega = np.empty((n_rows, T), np.float32)
    ratio = np.empty((n_rows, T), np.float32)
    chi = np.empty((n_rows, T), np.uint8)
    _check(lib().orc_grpo_coeffs(_p(adv_rows, np.float32), _p(logp_new, np.float32), _p(logp_old, np.float32),
                                 _p(logp_ref, np.float32), _p(mask, np.uint8), C.c_int64(n_rows), C.c_int64(T),
                                 C.c_int64(N_norm), C.c_float(clip_eps), C.c_float(beta), _p(omega, np.float32),
                                 _p(ratio, np.float32), _p(chi, np.uint8)))
    return omega, ratio, chi


def grpo_objective(adv_rows, s_f64, logp_old, logp_ref, mask, N, clip_eps=0.2, beta=0.0) -> float:
    n_rows, T = s_f64.shape
    adv_rows = np.ascontiguousarray(adv_rows, dtype=np.float32)
    return float(lib().orc_grpo_objective(_p(adv_rows, np.float32), _p(s_f64, np.float64), _p(logp_old, np.float32),
                                          _p(logp_ref, np.float32), _p(mask, np.uint8), C.c_int64(n_rows),
                                          C.c_int64(T), C.c_int64(N), C.c_float(clip_eps), C.c_float(beta)))


def row_rms(x_bits: np.ndarray, cols: int | None = None) -> np.ndarray:
    rows, ld = x_bits.shape
    cols = ld if cols is None else cols
    out = np.empty(rows, np.float32)
    _check(lib().orc_row_rms(_p(x_bits, np.uint16), C.c_int64(rows), C.c_int64(cols), C.c_int64(ld),
                             _p(out, np.float32)))
    return out


def unit_exposure(omega, mask, rms, row_shift=0, eps_alpha=1e-8):
    """omega, mask: [n_rows, T]; rms: [U, rms_ld] -> (exposure[U], sum_abs_omega)."""
    n_rows, T = omega.shape
    U, rms_ld = rms.shape
    out = np.empty(U, np.float32)
    sw = np.zeros(1, np.float32)
    _check(lib().orc_unit_exposure(_p(omega, np.float32), _p(mask, np.uint8), C.c_int64(n_rows), C.c_int64(T),
                                   _p(rms, np.float32), C.c_int32(U), C.c_int64(rms_ld), C.c_int32(row_shift),
                                   C.c_float(eps_alpha), _p(out, np.float32), _p(sw, np.float32)))
    return out, float(sw[0])


def compress(x_bits: np.ndarray, fmt: int, block: int = 64, cols: int | None = None):
    """x_bits: [rows, ld] uint16 -> (codes[rows, cols] uint8, scales[rows, cols/block] fp32 or None)."""
    rows, ld = x_bits.shape
    cols = ld if cols is None else cols
    codes = np.empty((rows, cols), np.uint8)
    scales = None
    if fmt != FMT_E4M3FN_RAW:
        if block <= 0 or cols % block:
            raise OracleError(SHAPE)
        scales = np.empty((rows, cols // block), np.float32)
    _check(lib().orc_compress(_p(x_bits, np.uint16), C.c_int64(rows), C.c_int64(cols), C.c_int64(ld), C.c_int32(fmt),
                              C.c_int32(block), _p(codes, np.uint8), _p(scales, np.float32)))
    return codes, scales


def recover(codes: np.ndarray, scales, fmt: int, block: int = 64, ld_out: int | None = None) -> np.ndarray:
    rows, cols = codes.shape
    ld_out = cols if ld_out is None else ld_out
    out = np.zeros((rows, ld_out), np.uint16)
    _check(lib().orc_recover(_p(codes, np.uint8), _p(scales, np.float32), C.c_int64(rows), C.c_int64(cols),
                             C.c_int32(fmt), C.c_int32(block), _p(out, np.uint16), C.c_int64(ld_out)))
    return out


def dequant_f32(codes, scales, fmt, block=64) -> np.ndarray:
    rows, cols = codes.shape
    out = np.empty((rows, cols), np.float32)
    _check(lib().orc_dequant_f32(_p(codes, np.uint8), _p(scales, np.float32), C.c_int64(rows), C.c_int64(cols),
                                 C.c_int32(fmt), C.c_int32(block), _p(out, np.float32)))
    return out


def relative_error(x_bits, xhat_bits) -> float:
    rows, ld = x_bits.shape
    return float(lib().orc_relative_error(_p(x_bits, np.uint16), _p(xhat_bits, np.uint16), C.c_int64(rows),
                                          C.c_int64(ld), C.c_int64(ld), C.c_int64(xhat_bits.shape[1])))


def plan(exposure, kappa, ebar, tau_lo, tau_hi, avail, rows, cols, fmt, block, action_in=None):
    """-> (action, psi, recompute, retained_bytes).  exposure None => gate action_in only."""
    U = len(avail)
    avail = np.ascontiguousarray(avail, np.uint8)
    action = np.zeros(U, np.uint8) if action_in is None else np.ascontiguousarray(action_in, np.uint8).copy()
    psi = np.zeros(U, np.float32)
    rec = np.zeros(U, np.uint8)
    ret = np.zeros(U, np.uint64)
    rows = np.ascontiguousarray(rows, np.int64)
    cols = np.ascontiguousarray(cols, np.int64)
    fmt = np.ascontiguousarray(fmt, np.int32)
    block = np.ascontiguousarray(block, np.int32)
    if exposure is not None:
        exposure = np.ascontiguousarray(exposure, np.float32)
        kappa = np.ascontiguousarray(kappa, np.float32)
        ebar = np.ascontiguousarray(ebar, np.float32)
    _check(lib().orc_plan(_p(exposure, np.float32), _p(kappa, np.float32), _p(ebar, np.float32), C.c_int32(U),
                          C.c_float(tau_lo), C.c_float(tau_hi), _p(avail, np.uint8), _p(rows, np.int64),
                          _p(cols, np.int64), _p(fmt, np.int32), _p(block, np.int32), _p(action, np.uint8),
                          _p(psi, np.float32), _p(rec, np.uint8), _p(ret, np.uint64)))
    return action, psi, rec, ret


def allocate(psi, dtau, dmem, avail, M_res, delta_b, N=1024):
    """The paper's DP allocator.  dtau, dmem: [U, 3] by action code (R, H, L).  -> (action[U], totals[3])
    with totals = (utility of the selection, its memory cost, its risk)."""
    psi = np.ascontiguousarray(psi, np.float32)
    U = psi.size
    dtau = np.ascontiguousarray(dtau, np.float64).reshape(U, 3)
    dmem = np.ascontiguousarray(dmem, np.float64).reshape(U, 3)
    avail = np.ascontiguousarray(avail, np.uint8)
    action = np.zeros(U, np.uint8)
    totals = np.zeros(3, np.float64)
    _check(lib().orc_allocate(C.c_int32(U), _p(psi, np.float32), _p(dtau, np.float64), _p(dmem, np.float64),
                              _p(avail, np.uint8), C.c_double(M_res), C.c_double(delta_b), C.c_int32(N),
                              _p(action, np.uint8), _p(totals, np.float64)))
    return action, totals


def risk_budget(delta, N_b, N_total) -> float:
    return float(lib().orc_risk_budget(C.c_double(delta), C.c_int64(N_b), C.c_int64(N_total)))


def fit_kappa(x, y) -> float:
    x = np.ascontiguousarray(x, np.float64)
    y = np.ascontiguousarray(y, np.float64)
    return float(lib().orc_fit_kappa(_p(x, np.float64), _p(y, np.float64), C.c_int64(x.size)))


def grpo_coeffs_variant(adv_rows, logp_new, logp_old, logp_ref, mask, N_norm=0, clip_eps=0.2, beta=0.0, variant=0):
    n_rows, T = logp_new.shape
    adv_rows = np.ascontiguousarray(adv_rows, dtype=np.float32)
    omega = np.empty((n_rows, T), np.float32)
    ratio = np.empty((n_rows, T), np.float32)
    chi = np.empty((n_rows, T), np.uint8)
    _check(lib().orc_grpo_coeffs_variant(_p(adv_rows, np.float32), _p(logp_new, np.float32), _p(logp_old, np.float32),
                                         _p(logp_ref, np.float32), _p(mask, np.uint8), C.c_int64(n_rows), C.c_int64(T),
                                         C.c_int64(N_norm), C.c_float(clip_eps), C.c_float(beta), C.c_int32(variant),
                                         _p(omega, np.float32), _p(ratio, np.float32), _p(chi, np.uint8)))
    return omega, ratio, chi


def omega_diagnostics(adv_rows, ratio, mask, omega, clip_eps=0.2):
    """-> (counts[5] = padding, zero-advantage, clipped, zero-omega, slots; top-decile share; sum |omega|)."""
    n_rows, T = omega.shape
    adv_rows = np.ascontiguousarray(adv_rows, dtype=np.float32)
    counts = np.zeros(5, np.int64)
    share = C.c_double(0.0)
    total = C.c_double(0.0)
    _check(lib().orc_omega_diagnostics(_p(adv_rows, np.float32), _p(ratio, np.float32), _p(mask, np.uint8),
                                       _p(omega, np.float32), C.c_int64(n_rows), C.c_int64(T), C.c_float(clip_eps),
                                       _p(counts, np.int64), C.byref(share), C.byref(total)))
    return counts, float(share.value), float(total.value)


def grpo_coeffs_packed(adv_seq, cu_seqlens, logp_new, logp_old, logp_ref, mask, N_norm=0, clip_eps=0.2, beta=0.0):
    """Packed layout: adv_seq [n_seq], cu_seqlens int32 [n_seq + 1], per-token arrays [n_tok]."""
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    n_seq, n_tok = len(cu) - 1, int(cu[-1])
    adv_seq = np.ascontiguousarray(adv_seq, dtype=np.float32)
    omega, ratio, chi = np.empty(n_tok, np.float32), np.empty(n_tok, np.float32), np.empty(n_tok, np.uint8)
    _check(lib().orc_grpo_coeffs_packed(_p(adv_seq, np.float32), _p(cu, np.int32), C.c_int64(n_seq),
                                        _p(logp_new, np.float32), _p(logp_old, np.float32), _p(logp_ref, np.float32),
                                        _p(mask, np.uint8), C.c_int64(N_norm), C.c_float(clip_eps), C.c_float(beta),
                                        _p(omega, np.float32), _p(ratio, np.float32), _p(chi, np.uint8)))
    return omega, ratio, chi


def unit_exposure_packed(omega, mask, cu_seqlens, rms, row_shift=0, eps_alpha=1e-8):
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    U, rms_ld = rms.shape
    out = np.empty(U, np.float32)
    sw = np.zeros(1, np.float32)
    _check(lib().orc_unit_exposure_packed(_p(omega, np.float32), _p(mask, np.uint8), _p(cu, np.int32),
                                          C.c_int64(len(cu) - 1), _p(rms, np.float32), C.c_int32(U), C.c_int64(rms_ld),
                                          C.c_int32(row_shift), C.c_float(eps_alpha), _p(out, np.float32),
                                          _p(sw, np.float32)))
    return out, float(sw[0])
