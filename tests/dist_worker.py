"""Worker of test_bench_dist.py: exercises bench.py's multi-rank plumbing on CPU (gloo)."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import bench  # noqa: E402


def main():
    args = bench.parse_args()
    world, rank, local = bench.dist_setup(args)
    bench.barrier(world)
    # each rank "measures" a different step time; the job time is the slowest rank's
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    bench.barrier(world)
    if rank == 0:
        cfg, _ = bench.workload(args)
        print(json.dumps({"world": world, "ms": ms, "value": cfg.batch * world / (ms * 1e-3 / cfg.layers)}))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
