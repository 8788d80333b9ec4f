"""Child program of tests/test_dist_gloo.py: one rank of a job started by
paper_2510_11370_b200.dist.launch_command.  Joins the group over gloo, takes the slowest rank's
time and the total of the sharded units, and rank 0 prints one JSON line (as bench.py does)."""
import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_11370_b200 import dist as r3dist  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--units", type=int, default=1001)
    args = ap.parse_args()
    rank, world = r3dist.init("gloo")
    lo, hi = r3dist.shard_range(args.units, rank, world)
    r3dist.barrier()
    slowest = r3dist.max_over_ranks(10.0 + rank)
    units = r3dist.sum_over_ranks(hi - lo)
    if rank == 0:
        print(json.dumps({"n_gpus": world, "asked": args.gpus, "slowest": slowest, "units": units,
                          "local_rank": int(os.environ.get("LOCAL_RANK", "-1"))}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
