"""Worker of the multi-process CPU tests (launched by torch.distributed.run with the gloo backend):
exercises the rank plumbing bench.py uses at N > 1 - replica plan, barrier, max-over-ranks timing."""
import json
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import spd_inputs as si  # noqa: E402


def main():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    w = si.WORKLOADS["c1"]
    plan = bench.replica_plan(w, rank, world)
    # every rank draws its own stack: different seeds give different weights
    mine = si.make_layer(w, 0, "cpu", plan["seed"])["wq"].double().sum().item()
    gathered = [None] * world
    dist.all_gather_object(gathered, (plan, mine))
    dist.barrier()
    # a rank-dependent "time": the job's time is the slowest rank's
    t_max, t_same = bench.max_over_ranks([1.0 + rank, 5.0])
    out = {"rank": rank, "world": world, "t_max": t_max, "t_same": t_same,
           "seeds": [g[0]["seed"] for g in gathered], "job_tokens": plan["tokens_per_step_job"],
           "distinct_weights": len({round(g[1], 9) for g in gathered})}
    if rank == 0:
        print("WORKER " + json.dumps(out), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
