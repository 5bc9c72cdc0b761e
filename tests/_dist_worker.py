"""Worker for the two-rank CPU test of bench.py's multi-rank bookkeeping (gloo backend)."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch.distributed as dist  # noqa: E402

import bench  # noqa: E402
from paper_2503_06671_b200 import synth  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    wl = synth.WORKLOADS_BY_NAME["cfg1_64x64_f32"]
    # each rank pretends to have measured a different step time; the job reports the slowest
    ms = 2.0 + rank
    worst = bench.max_over_ranks(ms, world)
    d = synth.make_inputs(wl.B, wl.C, wl.C_a, 8, 8, wl.K, wl.dtype, bench.rank_seed(wl, rank))
    out = {"rank": rank, "world": world, "worst_ms": worst, "value": bench.whole_job_value(wl.pixels, world, worst),
           "x0": float(d["x"].ravel()[0])}
    with open(os.path.join(os.environ["ESC_TEST_OUT"], f"rank{rank}.json"), "w") as f:
        json.dump(out, f)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
