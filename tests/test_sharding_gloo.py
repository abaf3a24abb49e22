"""The N > 1 host logic, run as two `gloo` ranks on CPU: per-rank workloads differ, the job time
is the max over ranks, throughput aggregates all ranks, head shards partition the kv heads."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_15105_b200 import sharding
from paper_2607_15105_b200.workloads import CONFIGS, make_inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert sharding.env_rank() == (rank, world, rank)
        cfg = sharding.rank_config(CONFIGS[1], rank)
        x = make_inputs(cfg, with_dO=False)
        digest = int(x["K"].astype(np.uint64).sum())
        my_ms = 10.0 + 5.0 * rank                    # rank 1 is the slow one
        total = sharding.max_over_ranks(my_ms)
        digests = [None] * world
        dist.all_gather_object(digests, digest)
        out[rank] = (total, digests, sharding.job_throughput(cfg.tokens_per_step, 4, world, total))
    finally:
        dist.destroy_process_group()


def test_two_ranks_weak_scaling_logic():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        total, digests, tps = res[rank]
        assert total == 15.0                                   # max over ranks, seen by every rank
        assert digests[0] != digests[1]                        # each rank drew its own sequence
        assert abs(tps - CONFIGS[1].tokens_per_step * 2 * 4 / 15.0e-3) < 1e-6
    assert res[0][1] == res[1][1]


def test_single_process_fallbacks():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.rank_config(CONFIGS[3], 0) is CONFIGS[3]
    assert sharding.rank_config(CONFIGS[3], 2).seed == CONFIGS[3].seed + 2000


def test_head_shards_partition_the_heads():
    for heads in (8, 6, 1):
        for world in (1, 2, 4, 8):
            covered = []
            for r in range(world):
                lo, hi = sharding.shard_heads(heads, r, world)
                assert 0 <= lo <= hi <= heads
                covered += list(range(lo, hi))
            assert covered == list(range(heads))
