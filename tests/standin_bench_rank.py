"""One rank of a CPU run of bench.py's multi-rank plumbing (started by tests/test_bench_launcher.py through
bench.launch_ranks; not a test itself).  The engine of the rank's shard is the fp64 oracle, the process group
is gloo, the timer is the wall clock; everything else is bench.py's own: the rank environment, the partition
of the workers, the warm-up / barrier / timed-periods loop, the maximum over ranks and the JSON line."""
import argparse
import json
import os
import sys
import time

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, HERE)
sys.path.insert(0, os.path.dirname(HERE))

import numpy as np
import torch.distributed as dist

import bench
from helpers import OracleEngine
from paper_1807_06629_b200 import sharded, synth


class WallTimer:
    def __init__(self):
        self.t, self.total = 0.0, 0.0

    def start(self, k):
        self.t = time.perf_counter()

    def stop(self, k):
        self.total += time.perf_counter() - self.t

    def total_ms(self):
        return 1e3 * self.total


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--scaling", default="strong")
    ap.add_argument("--steps", type=int, default=2)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()
    rank, _, world = bench.rank_env()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.Workload("standin", 5, (6, 5, 4), 4, 0.05, 3, 8, 0, 16, mean_shift=0.5, gumbel=True, seed=9)
    first, count, n_global = sharded.partition(w.N, world, rank, args.scaling)
    X, Y = synth.make_pools(w.with_(N=n_global))          # tiny: every rank holds the whole job's pools
    x0 = synth.init_params(w.dims, w.seed)
    eng = OracleEngine(w, X, Y, x0, first, count)
    job = sharded.ShardedPRSGD(eng, n_global, w.I, chunks=3)
    ms = bench.time_periods(lambda: job.local_steps(w.I), args.steps, args.warmup, WallTimer(), dist.barrier)
    ms = bench.max_over_ranks(ms, world)
    line = bench.result_line(bench.workload_config(w.with_(N=n_global)), n_global * w.I * args.steps / (ms * 1e-3), ms,
                             args.steps, args.warmup, world, args.scaling, "f64")
    line["node_average"] = [float(v) for v in eng.x.mean(0)] if rank == 0 else None
    line["rows_identical"] = bool(np.all(eng.x == eng.x[0:1]))
    line["local_workers"] = count
    if rank == 0:
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
