"""The N > 1 path of the benchmark on CPU: two gloo ranks, each a replica; the job time is the slowest rank's."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2512_19206_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.dist_env() == (rank, world, rank)
    mine = [100.0 + 50.0 * rank, 7.0 - rank]                 # this rank's step time and kernel time
    dist.barrier()
    got = replicas.max_over_ranks(mine)
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [150.0, 7.0]
    assert replicas.job_tokens_per_s(8, 2, 150.0) == 2 * 8 / 150e-6


def test_single_process_is_the_identity():
    assert replicas.dist_env()[1] >= 1
    assert replicas.max_over_ranks([3.0, 4.5]) == [3.0, 4.5]
