"""Worker for tests/test_multi_rank_cpu.py: one rank of a world-size-2 gloo group on CPU."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch.distributed as dist  # noqa: E402

import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    # rank r "measured" (10 + 5 r) ms: the job time is the slowest rank's
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
    value = bench.whole_job_tflops(world, 3.0e12, slowest)
    dist.barrier()
    out = {"rank": rank, "world": world, "slowest_ms": slowest, "value": value}
    with open(os.path.join(sys.argv[1], f"rank{rank}.json"), "w") as f:
        json.dump(out, f)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
