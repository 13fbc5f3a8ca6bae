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


def test_the_benchmark_launcher_starts_one_rank_per_gpu(tmp_path):
    """`bench.py --gpus N` without launcher variables starts its N ranks with replicas.spawn_local_ranks; here the same
    function starts two gloo ranks of a stub step on CPU: one line comes back, from rank 0, with the slowest rank's time."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    stub = os.path.join(root, "tests", "replica_stub.py")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["PYTHONPATH"] = root + os.pathsep + env.get("PYTHONPATH", "")
    code = ("import sys; from paper_2512_19206_b200 import replicas; "
            f"sys.exit(replicas.spawn_local_ranks(2, [sys.executable, {stub!r}] + sys.argv[1:], timeout=120))")
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=180)
    assert res.returncode == 0, res.stderr
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["us_per_step"] == 150.0 and line["kernel_us"] == 7.0
    assert line["tokens_per_s"] == 2 * 8 / 150e-6
    # a failing rank makes the job fail
    res = subprocess.run([sys.executable, "-c", code, "3"], env=env, capture_output=True, text=True, timeout=180)
    assert res.returncode == 3
