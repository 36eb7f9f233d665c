"""Worker of the 2-rank gloo test: the multi-rank plumbing of bench.py (replicas, max-over-ranks timing)."""
import os
import sys

import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    assert world == 2
    # ranks time different durations: everybody must end up with the slowest one
    mine = 10.0 + 5.0 * rank
    dist.barrier()
    slowest = bench.max_over_ranks(mine, "cpu")
    assert slowest == 15.0, slowest
    # replicas search on distinct random streams
    seeds = [None, None]
    dist.all_gather_object(seeds, bench.rank_seed(0, rank))
    assert seeds == [0, 1]
    # whole-job value: both ranks' units over the slowest rank's time
    assert bench.whole_job_rate(world, 1000, 4, slowest) == 2 * 1000 * 4 / 15e-3
    # the reference arm runs on rank 0 only
    if rank == 1:
        class A:
            steps, warmup, gpus = 1, 0, 2
        assert bench.run_reference(A, None) is None  # returns before touching the workload
    dist.barrier()
    dist.destroy_process_group()
    print(f"rank {rank} ok")


if __name__ == "__main__":
    main()
