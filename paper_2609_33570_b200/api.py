"""Thin ctypes binding of the C ABI declared in include/hilore.h (argument marshalling only).

Every function has the name and the argument order of its C entry point; tensors are torch
CUDA tensors of which only ``data_ptr()`` is passed on, and the current torch CUDA stream is
used unless ``stream`` is given.  Nothing here computes: every step of the path runs in the
library's CUDA kernels.  If the shared library is missing the import fails loudly; there is
no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

OK, INVALID_ARG, SHAPE, ALIGN, ZERO_NORM, CUDA, WORKSPACE = range(7)
FMT_E4M3FN_RAW, FMT_E4M3FN_BLK, FMT_INT8_BLK = 0, 1, 2
ACT_R, ACT_H, ACT_L = 0, 1, 2
PHASE_DECIDE, PHASE_CAPTURE, PHASE_ENCODE, PHASE_RECOVER = 0, 1, 2, 3
BLOCK = 64

EXPORTS = ("hilore_status_string", "hilore_abi_version", "hilore_mask_count", "hilore_grpo_coeffs",
           "hilore_unit_exposure", "hilore_workspace_bytes", "hilore_compress", "hilore_recover",
           "hilore_plan_apply", "hilore_unit_exposure_static", "hilore_static_scratch_bytes",
           "hilore_allocate", "hilore_allocate_workspace_bytes", "hilore_risk_budget",
           "hilore_relative_error", "hilore_relative_error_workspace_bytes", "hilore_fit_kappa",
           "hilore_grpo_coeffs_variant", "hilore_omega_diagnostics", "hilore_omega_diagnostics_workspace_bytes",
           "hilore_grpo_coeffs_packed", "hilore_unit_exposure_packed", "hilore_codec_relative_error",
           "hilore_coeffs_exposure", "hilore_scores_plan", "hilore_scores_plan_workspace_bytes")


class HiloreUnit(C.Structure):
    """Mirror of ``struct hilore_unit``."""
    _fields_ = [("x", C.c_void_p), ("codes", C.c_void_p), ("scales", C.c_void_p), ("out", C.c_void_p),
                ("row_rms", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("fmt", C.c_int32), ("block", C.c_int32)]


class HiloreError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> C.CDLL:
    """Load libhilore_b200.so (built in-tree by paper_2609_33570_b200.build)."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: run `python -m paper_2609_33570_b200.build` "
                              "(there is no fallback path)")
        _lib = C.CDLL(path)
        _lib.hilore_status_string.restype = C.c_char_p
        _lib.hilore_status_string.argtypes = [C.c_int]
        _lib.hilore_abi_version.restype = C.c_int
        _lib.hilore_workspace_bytes.restype = C.c_size_t
        _lib.hilore_workspace_bytes.argtypes = [C.c_int32, C.c_int64]
        vp, i64, i32, f32 = C.c_void_p, C.c_int64, C.c_int32, C.c_float
        _lib.hilore_mask_count.argtypes = [vp, i64, vp, vp]
        _lib.hilore_grpo_coeffs.argtypes = [vp, i64, i32, i64, i64, i64, vp, vp, vp, vp, i64, vp, f32, f32, f32,
                                            vp, vp, vp, vp, vp]
        _lib.hilore_unit_exposure.argtypes = [vp, vp, i64, i64, vp, i32, i64, i32, f32, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_unit_exposure_static.argtypes = [vp, vp, i64, i64, vp, i32, i64, i32, f32, vp, vp, vp]
        _lib.hilore_static_scratch_bytes.restype = C.c_size_t
        _lib.hilore_static_scratch_bytes.argtypes = []
        _lib.hilore_allocate.argtypes = [i32, vp, vp, vp, vp, C.c_double, C.c_double, i32, vp, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_allocate_workspace_bytes.restype = C.c_size_t
        _lib.hilore_allocate_workspace_bytes.argtypes = [i32, i32]
        _lib.hilore_risk_budget.restype = C.c_double
        _lib.hilore_risk_budget.argtypes = [C.c_double, i64, i64]
        _lib.hilore_relative_error.argtypes = [vp, vp, i64, i64, i64, i64, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_relative_error_workspace_bytes.restype = C.c_size_t
        _lib.hilore_relative_error_workspace_bytes.argtypes = []
        _lib.hilore_fit_kappa.restype = C.c_double
        _lib.hilore_fit_kappa.argtypes = [vp, vp, i64]
        _lib.hilore_grpo_coeffs_variant.argtypes = [vp, i64, i32, i64, i64, i64, vp, vp, vp, vp, i64, vp, f32, f32, f32, i32,
                                                    vp, vp, vp, vp, vp]
        _lib.hilore_grpo_coeffs_packed.argtypes = [vp, i64, i32, i64, i64, vp, i64, vp, vp, vp, vp, i64, vp, f32, f32, f32,
                                                   vp, vp, vp, vp, vp]
        _lib.hilore_unit_exposure_packed.argtypes = [vp, vp, i64, vp, i64, vp, i32, i64, i32, f32, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_coeffs_exposure.argtypes = [vp, i64, i32, i64, i64, i64, vp, vp, vp, vp, i64, vp, f32, f32, f32, vp, i32, i64,
                                                i32, f32, vp, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_scores_plan.argtypes = [vp, i64, i32, i64, i64, i64, vp, vp, vp, vp, i64, vp, f32, f32, f32, vp, i32, i64, i32,
                                            f32, vp, vp, vp, vp, vp, vp, f32, f32, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_scores_plan_workspace_bytes.restype = C.c_size_t
        _lib.hilore_scores_plan_workspace_bytes.argtypes = [i32, i64]
        _lib.hilore_codec_relative_error.argtypes = [vp, i64, i64, i64, i32, i32, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_omega_diagnostics.argtypes = [vp, vp, vp, vp, i64, i64, f32, vp, vp, vp, vp, C.c_size_t, vp]
        _lib.hilore_omega_diagnostics_workspace_bytes.restype = C.c_size_t
        _lib.hilore_omega_diagnostics_workspace_bytes.argtypes = []
        _lib.hilore_compress.argtypes = [vp, i64, i64, i64, i32, i32, vp, vp, vp, vp]
        _lib.hilore_recover.argtypes = [vp, vp, i64, i64, i32, i32, vp, i64, vp]
        _lib.hilore_plan_apply.argtypes = [vp, vp, i32, i32, vp, vp, vp, f32, f32, vp, vp, vp, vp, vp, vp]
        for name in EXPORTS:
            if name not in ("hilore_status_string", "hilore_workspace_bytes", "hilore_static_scratch_bytes",
                            "hilore_allocate_workspace_bytes", "hilore_risk_budget",
                            "hilore_relative_error_workspace_bytes", "hilore_fit_kappa",
                            "hilore_omega_diagnostics_workspace_bytes", "hilore_scores_plan_workspace_bytes"):
                getattr(_lib, name).restype = C.c_int
    return _lib


def status_string(status: int) -> str:
    return lib().hilore_status_string(int(status)).decode()


def _ptr(t):
    """Device (or host) address of a tensor; None -> NULL; ints pass through as raw addresses."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


# the current stream's handle without building a Stream object (3.2 us -> 1.2 us per call where torch has these)
_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)
_raw_device = getattr(torch._C, "_cuda_getDevice", None)


def _stream(stream):
    if stream is None:
        if _raw_stream is not None and _raw_device is not None:
            return _raw_stream(_raw_device())
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(st, where, check):
    if check and st != OK:
        raise HiloreError(st, where)
    return st


def hilore_mask_count(mask, n, count, stream=None, check=True):
    return _check(lib().hilore_mask_count(_ptr(mask), n, _ptr(count), _stream(stream)), "hilore_mask_count", check)


def hilore_grpo_coeffs(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask,
                       N_norm, N_norm_dev, clip_eps, beta, adv_eps, adv_out, omega, ratio, clip_mask,
                       stream=None, check=True):
    st = lib().hilore_grpo_coeffs(_ptr(rewards), n_resp_total, G, resp_offset, n_rows, T, _ptr(logp_new),
                                  _ptr(logp_old), _ptr(logp_ref), _ptr(mask), N_norm, _ptr(N_norm_dev),
                                  clip_eps, beta, adv_eps, _ptr(adv_out), _ptr(omega), _ptr(ratio),
                                  _ptr(clip_mask), _stream(stream))
    return _check(st, "hilore_grpo_coeffs", check)


def hilore_grpo_coeffs_variant(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask,
                               N_norm, N_norm_dev, clip_eps, beta, adv_eps, variant, adv_out, omega, ratio, clip_mask,
                               stream=None, check=True):
    st = lib().hilore_grpo_coeffs_variant(_ptr(rewards), n_resp_total, G, resp_offset, n_rows, T, _ptr(logp_new),
                                          _ptr(logp_old), _ptr(logp_ref), _ptr(mask), N_norm, _ptr(N_norm_dev),
                                          clip_eps, beta, adv_eps, variant, _ptr(adv_out), _ptr(omega), _ptr(ratio),
                                          _ptr(clip_mask), _stream(stream))
    return _check(st, "hilore_grpo_coeffs_variant", check)


def hilore_grpo_coeffs_packed(rewards, n_resp_total, G, resp_offset, n_seq, cu_seqlens, n_tok, logp_new, logp_old,
                              logp_ref, mask, N_norm, N_norm_dev, clip_eps, beta, adv_eps, adv_out, omega, ratio,
                              clip_mask, stream=None, check=True):
    st = lib().hilore_grpo_coeffs_packed(_ptr(rewards), n_resp_total, G, resp_offset, n_seq, _ptr(cu_seqlens), n_tok,
                                         _ptr(logp_new), _ptr(logp_old), _ptr(logp_ref), _ptr(mask), N_norm,
                                         _ptr(N_norm_dev), clip_eps, beta, adv_eps, _ptr(adv_out), _ptr(omega),
                                         _ptr(ratio), _ptr(clip_mask), _stream(stream))
    return _check(st, "hilore_grpo_coeffs_packed", check)


def hilore_unit_exposure_packed(omega, mask, n_tok, cu_seqlens, n_seq, row_rms, U, rms_ld, row_shift, eps_alpha,
                                exposure, sum_abs_omega, workspace, workspace_bytes, stream=None, check=True):
    st = lib().hilore_unit_exposure_packed(_ptr(omega), _ptr(mask), n_tok, _ptr(cu_seqlens), n_seq, _ptr(row_rms), U,
                                           rms_ld, row_shift, eps_alpha, _ptr(exposure), _ptr(sum_abs_omega),
                                           _ptr(workspace), workspace_bytes, _stream(stream))
    return _check(st, "hilore_unit_exposure_packed", check)


def hilore_coeffs_exposure(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask, N_norm,
                           N_norm_dev, clip_eps, beta, adv_eps, row_rms, U, rms_ld, row_shift, eps_alpha, omega, exposure,
                           sum_abs_omega, workspace, workspace_bytes, stream=None, check=True):
    st = lib().hilore_coeffs_exposure(_ptr(rewards), n_resp_total, G, resp_offset, n_rows, T, _ptr(logp_new), _ptr(logp_old),
                                      _ptr(logp_ref), _ptr(mask), N_norm, _ptr(N_norm_dev), clip_eps, beta, adv_eps,
                                      _ptr(row_rms), U, rms_ld, row_shift, eps_alpha, _ptr(omega), _ptr(exposure),
                                      _ptr(sum_abs_omega), _ptr(workspace), workspace_bytes, _stream(stream))
    return _check(st, "hilore_coeffs_exposure", check)


def hilore_scores_plan_workspace_bytes(U, n_tok):
    return int(lib().hilore_scores_plan_workspace_bytes(U, n_tok))


def hilore_scores_plan(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask, N_norm, N_norm_dev,
                       clip_eps, beta, adv_eps, row_rms, U, rms_ld, row_shift, eps_alpha, omega, exposure, sum_abs_omega,
                       units_dev, kappa, ebar, tau_lo, tau_hi, avail, action_io, psi, recompute, retained_bytes, workspace,
                       workspace_bytes, stream=None, check=True):
    st = lib().hilore_scores_plan(_ptr(rewards), n_resp_total, G, resp_offset, n_rows, T, _ptr(logp_new), _ptr(logp_old),
                                  _ptr(logp_ref), _ptr(mask), N_norm, _ptr(N_norm_dev), clip_eps, beta, adv_eps, _ptr(row_rms), U,
                                  rms_ld, row_shift, eps_alpha, _ptr(omega), _ptr(exposure), _ptr(sum_abs_omega), _ptr(units_dev),
                                  _ptr(kappa), _ptr(ebar), tau_lo, tau_hi, _ptr(avail), _ptr(action_io), _ptr(psi),
                                  _ptr(recompute), _ptr(retained_bytes), _ptr(workspace), workspace_bytes, _stream(stream))
    return _check(st, "hilore_scores_plan", check)


def hilore_codec_relative_error(x, rows, cols, ld, fmt, block, e_out, norms2, workspace, workspace_bytes, stream=None,
                                check=True):
    st = lib().hilore_codec_relative_error(_ptr(x), rows, cols, ld, fmt, block, _ptr(e_out), _ptr(norms2), _ptr(workspace),
                                           workspace_bytes, _stream(stream))
    return _check(st, "hilore_codec_relative_error", check)


def hilore_omega_diagnostics_workspace_bytes():
    return int(lib().hilore_omega_diagnostics_workspace_bytes())


def hilore_omega_diagnostics(adv, ratio, mask, omega, n_rows, T, clip_eps, counts, top_share, sum_abs, workspace,
                             workspace_bytes, stream=None, check=True):
    st = lib().hilore_omega_diagnostics(_ptr(adv), _ptr(ratio), _ptr(mask), _ptr(omega), n_rows, T, clip_eps,
                                        _ptr(counts), _ptr(top_share), _ptr(sum_abs), _ptr(workspace), workspace_bytes,
                                        _stream(stream))
    return _check(st, "hilore_omega_diagnostics", check)


def hilore_workspace_bytes(U, n_tok):
    return int(lib().hilore_workspace_bytes(U, n_tok))


def hilore_unit_exposure(omega, mask, n_rows, T, row_rms, U, rms_ld, row_shift, eps_alpha, exposure,
                         sum_abs_omega, workspace, workspace_bytes, stream=None, check=True):
    st = lib().hilore_unit_exposure(_ptr(omega), _ptr(mask), n_rows, T, _ptr(row_rms), U, rms_ld, row_shift,
                                    eps_alpha, _ptr(exposure), _ptr(sum_abs_omega), _ptr(workspace),
                                    workspace_bytes, _stream(stream))
    return _check(st, "hilore_unit_exposure", check)


def hilore_allocate_workspace_bytes(U, n_intervals=1024):
    return int(lib().hilore_allocate_workspace_bytes(U, n_intervals))


def hilore_risk_budget(delta, N_b, N_total):
    return float(lib().hilore_risk_budget(delta, N_b, N_total))


def hilore_allocate(U, psi, dtau, dmem, avail, M_res, delta_b, n_intervals, action, recompute, totals, workspace,
                    workspace_bytes, stream=None, check=True):
    st = lib().hilore_allocate(U, _ptr(psi), _ptr(dtau), _ptr(dmem), _ptr(avail), M_res, delta_b, n_intervals,
                               _ptr(action), _ptr(recompute), _ptr(totals), _ptr(workspace), workspace_bytes,
                               _stream(stream))
    return _check(st, "hilore_allocate", check)


def hilore_relative_error_workspace_bytes():
    return int(lib().hilore_relative_error_workspace_bytes())


def hilore_relative_error(x, xhat, rows, cols, ld, ld_hat, e_out, norms2, workspace, workspace_bytes, stream=None,
                          check=True):
    st = lib().hilore_relative_error(_ptr(x), _ptr(xhat), rows, cols, ld, ld_hat, _ptr(e_out), _ptr(norms2),
                                     _ptr(workspace), workspace_bytes, _stream(stream))
    return _check(st, "hilore_relative_error", check)


def hilore_fit_kappa(x, y):
    """x, y: sequences of host floats (calibration pairs)."""
    n = len(x)
    ax = (C.c_double * n)(*[float(v) for v in x])
    ay = (C.c_double * n)(*[float(v) for v in y])
    return float(lib().hilore_fit_kappa(C.cast(ax, C.c_void_p), C.cast(ay, C.c_void_p), n))


def hilore_static_scratch_bytes():
    return int(lib().hilore_static_scratch_bytes())


def hilore_unit_exposure_static(omega, mask, n_rows, T, row_rms, U, rms_ld, row_shift, eps_alpha, exposure,
                                sum_abs_omega, stream=None, check=True):
    """hilore_unit_exposure without a workspace argument: the partial sums use the library's built-in
    1 MiB scratch array, so the call allocates nothing (see include/hilore.h for the limits)."""
    st = lib().hilore_unit_exposure_static(_ptr(omega), _ptr(mask), n_rows, T, _ptr(row_rms), U, rms_ld, row_shift,
                                           eps_alpha, _ptr(exposure), _ptr(sum_abs_omega), _stream(stream))
    return _check(st, "hilore_unit_exposure_static", check)


def hilore_compress(x, rows, cols, ld, fmt, block, codes, scales, row_rms, stream=None, check=True):
    st = lib().hilore_compress(_ptr(x), rows, cols, ld, fmt, block, _ptr(codes), _ptr(scales), _ptr(row_rms),
                               _stream(stream))
    return _check(st, "hilore_compress", check)


def hilore_recover(codes, scales, rows, cols, fmt, block, out, ld_out, stream=None, check=True):
    st = lib().hilore_recover(_ptr(codes), _ptr(scales), rows, cols, fmt, block, _ptr(out), ld_out,
                              _stream(stream))
    return _check(st, "hilore_recover", check)


def hilore_plan_apply(units_dev, units_host, U, phase, exposure, kappa, ebar, tau_lo, tau_hi, avail, action_io,
                      psi, recompute, retained_bytes, stream=None, check=True):
    """units_dev: device address (tensor or int) of the hilore_unit table; units_host: a ctypes array
    ``(HiloreUnit * U)`` holding the same table on the host."""
    host = C.cast(units_host, C.c_void_p) if units_host is not None else None
    st = lib().hilore_plan_apply(_ptr(units_dev), host, U, phase, _ptr(exposure), _ptr(kappa), _ptr(ebar),
                                 tau_lo, tau_hi, _ptr(avail), _ptr(action_io), _ptr(psi), _ptr(recompute),
                                 _ptr(retained_bytes), _stream(stream))
    return _check(st, "hilore_plan_apply", check)


def make_unit_table(units, device="cuda"):
    """Marshal a list of dicts (x, codes, scales, out, row_rms tensors or None; rows, cols, ld, fmt, block)
    into the host ctypes array and a device copy of it.  Returns (units_dev tensor, units_host array)."""
    arr = (HiloreUnit * len(units))()
    for i, u in enumerate(units):
        arr[i] = HiloreUnit(_ptr(u.get("x")), _ptr(u.get("codes")), _ptr(u.get("scales")), _ptr(u.get("out")),
                            _ptr(u.get("row_rms")), u["rows"], u["cols"], u.get("ld", u["cols"]), u["fmt"],
                            u["block"])
    raw = bytes(arr)
    host = torch.frombuffer(bytearray(raw), dtype=torch.uint8)
    dev = host.to(device)
    return dev, arr
