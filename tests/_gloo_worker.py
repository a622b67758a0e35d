"""Worker of the world_size-2 gloo test: checks bench.py's cross-rank aggregation on CPU."""
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    # rank r took (10 + 5 r) ms for 1000 (r + 1) queries
    ms, units = bench.aggregate_ranks(dist, 10.0 + 5.0 * rank, 1000.0 * (rank + 1), device="cpu")
    assert ms == 10.0 + 5.0 * (world - 1), ms
    assert units == 1000.0 * world * (world + 1) / 2, units
    dist.barrier()
    if rank == 0:
        print("AGGREGATE_OK", ms, units)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
