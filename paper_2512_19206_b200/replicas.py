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


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_local_ranks(n: int, argv, env=None, timeout=None) -> int:
    """Starts `argv` n times on this node, rank i with RANK = LOCAL_RANK = i, WORLD_SIZE = n and a rendezvous on
    127.0.0.1, waits for all of them and returns 0 if all ended with 0, else the exit code of the first rank seen failing.  The children inherit stdout and stderr, so
    the one line rank 0 prints is the job's line.  If a rank fails, the others are stopped."""
    import subprocess
    import time
    port = free_port()
    procs = []
    for rank in range(n):
        e = dict(os.environ if env is None else env)
        e.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=e))
    t0, rc = time.monotonic(), 0
    live = list(procs)
    stopped = set()
    while live:
        for p in list(live):
            code = p.poll()
            if code is not None:
                live.remove(p)
                if code != 0 and rc == 0 and p.pid not in stopped:
                    rc = abs(code)
                    for other in live:
                        stopped.add(other.pid)
                        other.terminate()
        if timeout is not None and time.monotonic() - t0 > timeout:
            for other in live:
                other.kill()
            return rc or 124
        time.sleep(0.05)
    return rc
