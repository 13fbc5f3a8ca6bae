"""Host-side plumbing for running N independent replicas of the decode path, one process per GPU.

The path shards without any data-path exchange: every (layer, batch element, KV head) stream is independent in
selection, quantization and attention, so N GPUs run N replicas of the workload (weak scaling).  The only
communication is the reduction of the measured times: a job is as slow as its slowest rank.
"""
from __future__ import annotations

import os

import torch


def dist_env():
    """(rank, world size, local rank) from the launcher's environment; a single process when unset."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_tokens_per_s(batch_per_replica: int, world: int, us_per_step: float) -> float:
    """Whole-job decode throughput: every replica emits one token per sequence per step."""
    return world * batch_per_replica / (us_per_step * 1e-6)
