"""Worker of tests/test_multi_rank_cpu.py: one rank of a gloo job, launched by torch.distributed.run."""
import json
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
import workloads as wl  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    cfg = wl.config("r11")
    x, labels, theta = bench.replica_inputs(cfg, rank)
    # per-rank step times: rank 1 is the slow one for the first value, rank 0 for the second
    ms = bench.max_over_ranks(dist, [10.0 + 5.0 * rank, 30.0 - 7.0 * rank], torch.device("cpu"))
    gathered = [None] * world
    dist.all_gather_object(gathered, {"x_sum": float(x.sum()), "labels": labels.tolist(), "theta_sum": float(theta.astype(np.float64).sum())})
    if rank == 0:
        print(json.dumps({"ms": ms, "ranks": gathered, "value": bench.aggregate_throughput(world, cfg["B"], ms[0])}), flush=True)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
