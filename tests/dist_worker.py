"""Worker of tests/test_bench_dist.py: one rank of a gloo process group exercising bench.py's multi-rank logic."""
import json
import os
import sys
from pathlib import Path

import numpy as np
import torch
import torch.distributed as dist

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402


def main():
    out_dir = Path(sys.argv[1])
    rank, world, local = bench.dist_setup(int(os.environ["WORLD_SIZE"]))
    dist.init_process_group("gloo")
    # every rank reports its own timings; all must agree on the element-wise maximum
    mine = [10.0 + rank, 5.0 - rank]
    got = bench.max_over_ranks(mine, torch.device("cpu"), True)
    # per-rank batches differ, weights are replicated
    c = bench.rank_workload(rank)
    digest = {"rank": rank, "world": world, "local": local, "max": got,
              "a_sum": float(np.float64(c.a[:64].sum())), "w_sum": float(np.float64(c.w[:64].sum())),
              "value": bench.whole_job_value(2.0, world)}
    (out_dir / f"rank{rank}.json").write_text(json.dumps(digest))
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
