"""Helpers of the GPU parity tests: guarded device buffers and NumPy-in / NumPy-out calls of the C ABI."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_33570_b200 import api

GUARD = 256          # bytes of canary before and after every output buffer
CANARY = 0xA5

_NP2T = {np.dtype(np.uint8): torch.uint8, np.dtype(np.uint16): torch.int16, np.dtype(np.float32): torch.float32,
         np.dtype(np.int64): torch.int64, np.dtype(np.uint64): torch.int64}


class Guarded:
    """A device buffer of `nbytes` with canary bands on both sides; payload starts 256-byte aligned."""

    def __init__(self, nbytes: int, fill: int = CANARY):
        self.nbytes = int(nbytes)
        pad = (-self.nbytes) % 256
        self.raw = torch.full((GUARD + self.nbytes + pad + GUARD,), fill if fill is not None else 0,
                              dtype=torch.uint8, device="cuda")
        self.raw[:GUARD] = CANARY
        self.raw[GUARD + self.nbytes:] = CANARY
        self.view = self.raw[GUARD:GUARD + self.nbytes]
        assert self.view.data_ptr() % 256 == 0 or self.nbytes == 0

    def ptr(self) -> int:
        return self.view.data_ptr()

    def numpy(self, dtype, shape):
        torch.cuda.synchronize()
        assert bool((self.raw[:GUARD] == CANARY).all()), "write before the start of an output buffer"
        assert bool((self.raw[GUARD + self.nbytes:] == CANARY).all()), "write past the end of an output buffer"
        return self.view.cpu().numpy().view(dtype).reshape(shape).copy()


def dev(a: np.ndarray) -> torch.Tensor:
    """Host array -> device tensor with the same bits."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    if a.dtype == np.uint64:
        return torch.from_numpy(a.view(np.int64)).cuda()
    return torch.from_numpy(a).cuda()


def compress(x_bits: np.ndarray, fmt: int, cols=None, want_codes=True, want_rms=True):
    rows, ld = x_bits.shape
    cols = ld if cols is None else cols
    block = 0 if fmt == api.FMT_E4M3FN_RAW else 64
    x = dev(x_bits)
    codes = Guarded(rows * cols) if want_codes else None
    scales = Guarded(rows * (cols // 64) * 4) if (want_codes and block) else None
    rms = Guarded(rows * 4) if want_rms else None
    api.hilore_compress(x, rows, cols, ld, fmt, block, codes.ptr() if codes else None,
                        scales.ptr() if scales else None, rms.ptr() if rms else None)
    return (codes.numpy(np.uint8, (rows, cols)) if codes else None,
            scales.numpy(np.float32, (rows, cols // 64)) if scales else None,
            rms.numpy(np.float32, (rows,)) if rms else None)


def recover(codes: np.ndarray, scales, fmt: int, ld_out=None):
    rows, cols = codes.shape
    ld_out = cols if ld_out is None else ld_out
    block = 0 if fmt == api.FMT_E4M3FN_RAW else 64
    c = dev(codes)
    s = dev(scales) if scales is not None else None
    out = Guarded(rows * ld_out * 2)
    api.hilore_recover(c, s, rows, cols, fmt, block, out.ptr(), ld_out)
    return out.numpy(np.uint16, (rows, ld_out))


def grpo_coeffs(ro, *, resp_offset=0, n_rows=None, N_norm=0, N_on_device=False, clip_eps=0.2, beta=0.0,
                extras=True):
    """Run hilore_grpo_coeffs on rows [resp_offset, resp_offset + n_rows) of a synth.Rollout."""
    n_rows = ro.n_resp - resp_offset if n_rows is None else n_rows
    sl = slice(resp_offset, resp_offset + n_rows)
    T = ro.T
    R = dev(ro.rewards)
    ln, lo, lr, mk = dev(ro.logp_new[sl]), dev(ro.logp_old[sl]), dev(ro.logp_ref[sl]), dev(ro.mask[sl])
    adv, omega = Guarded(n_rows * 4), Guarded(n_rows * T * 4)
    ratio = Guarded(n_rows * T * 4) if extras else None
    chi = Guarded(n_rows * T) if extras else None
    ndev = None
    if N_on_device:
        ndev = torch.zeros(1, dtype=torch.int64, device="cuda")
        full = dev(ro.mask)
        api.hilore_mask_count(full, full.numel(), ndev)
    api.hilore_grpo_coeffs(R, ro.n_resp, ro.G, resp_offset, n_rows, T, ln, lo, lr if beta != 0 else None, mk,
                           N_norm, ndev, clip_eps, beta, 1e-6, adv.ptr(), omega.ptr(),
                           ratio.ptr() if ratio else None, chi.ptr() if chi else None)
    out = dict(adv=adv.numpy(np.float32, (n_rows,)), omega=omega.numpy(np.float32, (n_rows, T)))
    if extras:
        out["ratio"] = ratio.numpy(np.float32, (n_rows, T))
        out["chi"] = chi.numpy(np.uint8, (n_rows, T))
    if ndev is not None:
        out["N"] = int(ndev.item())
    return out


def unit_exposure(omega: np.ndarray, mask: np.ndarray, rms: np.ndarray, row_shift=0, eps_alpha=1e-8):
    n_rows, T = omega.shape
    U, rms_ld = rms.shape
    nbytes = api.hilore_workspace_bytes(U, n_rows * T)
    ws = Guarded(nbytes)
    E, sw = Guarded(U * 4), Guarded(4)
    api.hilore_unit_exposure(dev(omega), dev(mask), n_rows, T, dev(rms), U, rms_ld, row_shift, eps_alpha, E.ptr(),
                             sw.ptr(), ws.ptr(), nbytes)
    ws.numpy(np.uint8, (nbytes,))       # checks the workspace canaries
    return E.numpy(np.float32, (U,)), float(sw.numpy(np.float32, (1,))[0])


def rel_err(got, want):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    den = np.maximum(np.abs(want), 1e-300)
    return np.where(want == got, 0.0, np.abs(got - want) / den)
