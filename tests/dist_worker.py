"""Worker of test_multiprocess.py: one of two gloo ranks on CPU exercising bench.py's rank plumbing."""
import os
import sys

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    rank, world, local = bench.dist_env()
    dist.init_process_group("gloo")
    assert dist.get_world_size() == world == 2 and dist.get_rank() == rank
    # the job's step time is the slowest rank's; every rank must agree on it
    mine = 10.0 + 5.0 * rank
    worst = bench.max_over_ranks(mine, torch.device("cpu"), world)
    assert worst == 15.0, worst
    # replicas: each rank processes its own copy of the workload, no data-path exchange
    value = bench.whole_job_value(8192, world, worst)
    assert abs(value - 2 * 8192 / 0.015) < 1e-6
    dist.barrier()
    if rank == 0:
        print("DIST_OK %d %.1f %.3f" % (world, worst, value))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
