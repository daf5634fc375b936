"""Child process of test_bench_multirank.py: one gloo rank that exercises bench.py's cross-rank reduction."""
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    mine = 10.0 + 5.0 * rank  # rank 1 is the slow replica
    slowest = bench.max_over_ranks(mine, world, "cpu")
    assert slowest == 10.0 + 5.0 * (world - 1), slowest
    gbs = bench.whole_job_gbs(1e9, world, slowest)
    assert abs(gbs - world / slowest) < 1e-12, gbs
    dist.barrier()
    if rank == 0:
        print("GLOO_OK world=%d slowest=%.1f" % (world, slowest), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
