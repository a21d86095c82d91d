"""Seeded synthetic inputs shaped like the paper's GRPO actor-update workloads.

This module only DRAWS inputs (rewards, log-probabilities, masks, bf16
activation units).  It holds none of the method's arithmetic, so both the CUDA
path and the CPU oracle may be fed from it.  The recipe follows the paper's
setup section (binary rewards, dense padded layout, 8 or 16 responses per
prompt, response-validity masks) with shapes of Qwen2.5-style decoders.

Host generators use NumPy's PCG64 (``default_rng``) and return NumPy arrays;
bf16 tensors are returned as ``uint16`` bit patterns.  The device generators
draw the same distributions with a seeded ``torch.Generator`` on the GPU, for
units too large to draw on the host in reasonable time.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

OUTLIER_FRACTION = 0.01
OUTLIER_GAIN = 20.0


def _to_bf16_bits(x_f32: np.ndarray) -> np.ndarray:
    """fp32 array -> bf16 bit patterns (uint16), round-to-nearest-even (torch CPU cast)."""
    t = torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def outlier_channels(rng: np.random.Generator, d: int) -> np.ndarray:
    """Indices of the ceil(1% * d) feature channels that carry x20 outliers."""
    n = int(math.ceil(OUTLIER_FRACTION * d))
    return np.sort(rng.permutation(d)[:n])


def activation_unit(rng: np.random.Generator, rows: int, d: int) -> np.ndarray:
    """One saved activation unit [rows, d] as bf16 bits: N(0,1) with 1% of channels x20."""
    x = rng.standard_normal((rows, d), dtype=np.float32)
    ch = outlier_channels(rng, d)
    x[:, ch] *= np.float32(OUTLIER_GAIN)
    return _to_bf16_bits(x)


def activation_unit_device(gen: torch.Generator, rows: int, d: int, device="cuda") -> torch.Tensor:
    """Device-side draw of the same recipe (N(0,1), 1% channels x20), bf16 [rows, d]."""
    x = torch.randn((rows, d), generator=gen, device=device, dtype=torch.float32)
    n = int(math.ceil(OUTLIER_FRACTION * d))
    ch = torch.randperm(d, generator=gen, device=device)[:n]
    x[:, ch] *= OUTLIER_GAIN
    return x.to(torch.bfloat16)


@dataclass
class Rollout:
    """One rollout batch in the dense padded layout: responses of a prompt are contiguous."""
    P: int
    G: int
    T: int
    rewards: np.ndarray    # [P*G] fp32
    logp_new: np.ndarray   # [P*G, T] fp32
    logp_old: np.ndarray   # [P*G, T] fp32
    logp_ref: np.ndarray   # [P*G, T] fp32 (only used when beta > 0)
    mask: np.ndarray       # [P*G, T] uint8, 1 = valid generated response token
    lengths: np.ndarray    # [P*G] int64

    @property
    def n_resp(self) -> int:
        return self.P * self.G

    @property
    def n_valid(self) -> int:
        return int(self.mask.sum(dtype=np.int64))


def rollout(seed: int, P: int, G: int, T: int, *, rewards: str = "bernoulli",
            lengths: str = "full", min_len: int = 128, equal_group_fraction: float = 0.0,
            mask_first_column: bool = False) -> Rollout:
    """Draw rewards, log-probabilities and masks for P prompts x G responses x T slots.

    rewards: "bernoulli" (0/1 with p = 0.5) or "uniform" (U[0,1) fp32).
    lengths: "full" (every slot valid) or "uniform" (integer lengths U{min_len..T}).
    equal_group_fraction: that share of the prompt groups gets one reward repeated G times.
    """
    ss = np.random.SeedSequence(seed)
    s_rew, s_lp, s_old, s_ref, s_len, s_eq = (np.random.default_rng(s) for s in ss.spawn(6))
    n_resp = P * G
    if rewards == "bernoulli":
        R = (s_rew.random(n_resp) < 0.5).astype(np.float32)
    elif rewards == "uniform":
        R = s_rew.random(n_resp, dtype=np.float32)
    else:
        raise ValueError(rewards)
    n_eq = int(round(equal_group_fraction * P))
    if n_eq:
        groups = s_eq.permutation(P)[:n_eq]
        Rg = R.reshape(P, G)
        Rg[groups, :] = Rg[groups, :1]
    logp_new = (s_lp.standard_normal((n_resp, T), dtype=np.float32) * np.float32(0.5)
                - np.float32(1.5)).astype(np.float32)
    logp_old = (logp_new + s_old.standard_normal((n_resp, T), dtype=np.float32) * np.float32(0.05)).astype(np.float32)
    logp_ref = (logp_new + s_ref.standard_normal((n_resp, T), dtype=np.float32) * np.float32(0.05)).astype(np.float32)
    if lengths == "full":
        L = np.full(n_resp, T, dtype=np.int64)
    elif lengths == "uniform":
        L = s_len.integers(min(min_len, T), T + 1, size=n_resp, dtype=np.int64)
    else:
        raise ValueError(lengths)
    mask = (np.arange(T, dtype=np.int64)[None, :] < L[:, None]).astype(np.uint8)
    if mask_first_column:
        mask[:, 0] = 0
    return Rollout(P, G, T, R, logp_new, logp_old, logp_ref, mask, L)


@dataclass
class PackedRollout:
    """A microbatch in the padding-removed layout: sequence i = prompt tokens then the valid response tokens of
    row `rows[i]` of a dense Rollout; tokens of all sequences back to back."""
    cu_seqlens: np.ndarray  # [n_seq + 1] int32
    rows: np.ndarray        # [n_seq] int64, response index in the dense rollout
    logp_new: np.ndarray    # [n_tok] fp32
    logp_old: np.ndarray
    logp_ref: np.ndarray
    mask: np.ndarray        # [n_tok] uint8, 1 = generated response token
    dense_t: np.ndarray     # [n_tok] int64: response slot t of the token in the dense layout, -1 for prompt tokens

    @property
    def n_tok(self) -> int:
        return int(self.cu_seqlens[-1])


def pack_rollout(ro: Rollout, seed: int, rows=None, max_prompt: int = 64, min_prompt: int = 1) -> PackedRollout:
    """Re-lay rows `rows` (default: all) of a dense rollout without padding, each behind a prompt of random length
    U{min_prompt..max_prompt} whose log-probabilities are drawn like the response's (they are masked out)."""
    rng = np.random.default_rng(np.random.SeedSequence([seed, 77]))
    rows = np.arange(ro.n_resp, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    plen = rng.integers(min_prompt, max_prompt + 1, size=len(rows), dtype=np.int64)
    lens = plen + ro.lengths[rows]
    cu = np.zeros(len(rows) + 1, dtype=np.int64)
    np.cumsum(lens, out=cu[1:])
    n_tok = int(cu[-1])
    out = {k: np.empty(n_tok, np.float32) for k in ("logp_new", "logp_old", "logp_ref")}
    mask = np.zeros(n_tok, np.uint8)
    dense_t = np.full(n_tok, -1, np.int64)
    for j, i in enumerate(rows):
        a, b, L = int(cu[j]), int(cu[j] + plen[j]), int(ro.lengths[i])
        for k in out:
            out[k][a:b] = (rng.standard_normal(b - a, dtype=np.float32) * np.float32(0.5) - np.float32(1.5))
            out[k][b:b + L] = getattr(ro, k)[i, :L]
        mask[b:b + L] = ro.mask[i, :L]
        dense_t[b:b + L] = np.arange(L)
    return PackedRollout(cu.astype(np.int32), rows, out["logp_new"], out["logp_old"], out["logp_ref"], mask, dense_t)


# Unit widths (attention input, MLP input, MLP intermediate) of the decoder shapes the configs name.
UNIT_WIDTHS = {
    "0.5B": (896, 896, 4864),
    "1.5B": (1536, 1536, 8960),
    "7B": (3584, 3584, 18944),
}


def layer_unit_shapes(model: str, rows: int, layers: int):
    """[(rows, d)] for `layers` decoder layers, three saved units per layer."""
    w = UNIT_WIDTHS[model]
    return [(rows, d) for _ in range(layers) for d in w]
