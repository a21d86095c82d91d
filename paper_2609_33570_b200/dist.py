"""Host-side plumbing of the data-parallel path (one process per GPU, torch.distributed).

The hot path shards by microbatch: every rank compresses, scores and recovers its own microbatches
with no data-path collective.  The one batch-wide quantity is the normaliser N of the GRPO objective
(all valid response tokens of the complete rollout batch): one integer all-reduce per update.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_microbatches(n_microbatches: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of microbatch indices for `rank` (sizes differ by at most one)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    lo = (n_microbatches * rank) // world
    hi = (n_microbatches * (rank + 1)) // world
    return range(lo, hi)


def global_token_count(local_count: torch.Tensor) -> int:
    """Sum of the ranks' valid-token counts (int64 tensor of one element, on the backend's device)."""
    total = local_count.clone()
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(total, op=dist.ReduceOp.SUM)
    return int(total.item())


def gather_rewards(local_rewards: torch.Tensor) -> torch.Tensor:
    """All ranks' rewards in rank order, for prompt groups whose responses are split across ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local_rewards.clone()
    parts = [torch.empty_like(local_rewards) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, local_rewards.contiguous())
    return torch.cat(parts)
