"""Worker for the world_size-2 gloo test of the benchmark's multi-process plumbing.
Launched by tests/test_multiprocess.py through torch.distributed.run."""
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def main():
    world, rank, local = bench.dist_setup(2)
    dev = torch.device("cpu")
    bench.barrier(world)
    slowest = bench.max_over_ranks(10.0 * (rank + 1), world, dev)
    # replicas: every rank derives its own gradient stream from (seed + rank)
    from paper_2306_06098_b200 import gradgen
    g = gradgen.GradStream(1000, 4, seed=rank).next()
    print(json.dumps({"rank": rank, "world": world, "local": local, "slowest": slowest,
                      "g0": float(g[0])}), flush=True)
    bench.barrier(world)
    import torch.distributed as dist
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
