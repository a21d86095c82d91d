"""The multi-rank host logic on CPU: two gloo ranks shard the microbatches and agree on the normaliser N."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_33570_b200 import dist as hdist
from paper_2609_33570_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ro = synth.rollout(0, 8, 4, 64, lengths="uniform", min_len=8)
        mine = hdist.shard_microbatches(8, rank, world)            # one microbatch per prompt here
        rows = [r for mb in mine for r in range(mb * 4, mb * 4 + 4)]
        local = torch.tensor([int(ro.mask[rows].sum())], dtype=torch.int64)
        total = hdist.global_token_count(local)
        rewards = hdist.gather_rewards(torch.from_numpy(ro.rewards[rows]))
        q.put((rank, list(mine), total, rewards.numpy().tolist()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_and_agree_on_N():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ro = synth.rollout(0, 8, 4, 64, lengths="uniform", min_len=8)
    assert res[0][1] + res[1][1] == list(range(8))
    assert res[0][2] == res[1][2] == ro.n_valid
    assert np.allclose(res[0][3], ro.rewards) and res[0][3] == res[1][3]


def test_shard_is_a_balanced_partition():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            parts = [hdist.shard_microbatches(n, r, world) for r in range(world)]
            assert [i for p in parts for i in p] == list(range(n))
            sizes = [len(p) for p in parts]
            assert max(sizes) - min(sizes) <= 1
