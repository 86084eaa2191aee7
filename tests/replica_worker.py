"""Worker of test_bench_replicas.py: one rank of a 2-process gloo job exercising the multi-process
host logic of bench.py (rendezvous from the torchrun environment, barrier, max over ranks)."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch

import bench


def main():
    rank, world, local = bench.dist_setup(world_hint := int(os.environ.get("WORLD_SIZE", "1")))
    assert world == world_hint == 2 and rank == int(os.environ["RANK"])
    bench.barrier(world)
    # every replica reports its own time; the job's time is the slowest replica's
    mine = 10.0 + 5.0 * rank
    worst = bench.max_over_ranks(mine, world, torch.device("cpu"))
    # whole-job value = units of all replicas / that time
    flops_per_replica = 3.0e12
    value = world * flops_per_replica / (worst * 1e-3) / 1e12
    bench.barrier(world)
    if rank == 0:
        print(json.dumps({"worst_ms": worst, "value": value, "world": world}))
    import torch.distributed as dist
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
