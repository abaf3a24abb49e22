"""Host-side logic for running the HGA path on several GPUs of one node.

The path shards with no exchange step: items (batch, kv head, query block) are independent in
the forward pass and dK/dV reduce only across the query blocks of one (batch, kv head).  So
every rank processes its own sequences (weak scaling); the only collectives are the timing
barrier and the max over ranks of the measured time.  Nothing here touches the data path.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    """(rank, world_size, local_rank) from the launcher's environment (torchrun), else 0, 1, 0."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_config(cfg, rank: int):
    """The workload of `rank`: same shapes, its own sequence (seed shifted per rank)."""
    return cfg if rank == 0 else cfg.scaled(seed=cfg.seed + 1000 * rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_rank_step: int, steps: int, world: int, total_ms: float) -> float:
    """Whole-job tokens/s: every rank processed `steps` steps in the (max over ranks) time."""
    return tokens_per_rank_step * world * steps / (total_ms * 1e-3)


def shard_heads(n_kv_heads: int, rank: int, world: int):
    """Strong-scaling alternative: the kv heads [lo, hi) owned by `rank` (tensor-parallel head
    split; each rank then holds K/V, summaries and gradients of its own heads only)."""
    base, extra = divmod(n_kv_heads, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)
