"""A stand-in for one rank of the benchmark: joins the job with gloo, reduces its own 'step time' with MAX and lets
rank 0 print the job's line.  Started by tests/test_replicas_gloo.py through replicas.spawn_local_ranks."""
import json
import sys

import torch.distributed as dist

from paper_2512_19206_b200 import replicas

rank, world, local = replicas.dist_env()
dist.init_process_group("gloo", rank=rank, world_size=world)
mine = [100.0 + 50.0 * rank, 7.0 - rank]
dist.barrier()
got = replicas.max_over_ranks(mine)
if rank == 0:
    print(json.dumps({"n_gpus": world, "us_per_step": got[0], "kernel_us": got[1],
                      "tokens_per_s": replicas.job_tokens_per_s(8, world, got[0])}), flush=True)
dist.barrier()
dist.destroy_process_group()
sys.exit(int(sys.argv[1]) if len(sys.argv) > 1 and rank == 1 else 0)
