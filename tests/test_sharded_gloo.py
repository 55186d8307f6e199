"""World-size-2 test (gloo, CPU) of the multi-GPU orchestration: shard bounds, chunked all-reduce
averaging and the schedule.  The local engine here is the fp64 oracle, so the test exercises
`sharded.py` and the collective only; the GPU halves (partial_sum / assign_rows) are checked
against prsgd_average in the GPU tests."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import prsgd_oracle as orc
from paper_1807_06629_b200 import sharded, synth
from helpers import OracleEngine


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.Workload("t", 5, (6, 5, 4), 4, 0.05, 3, 8, 0, 16, mean_shift=0.5, gumbel=True, seed=9)
        X, Y = synth.make_pools(w)
        x0 = synth.init_params(w.dims, w.seed)
        first, count = sharded.shard_bounds(w.N, world, rank)
        eng = OracleEngine(w, X, Y, x0, first, count)
        job = sharded.ShardedPRSGD(eng, w.N, w.I, chunks=3)
        job.local_steps(2)
        job.local_steps(5)            # crosses the averages after t = 3 and t = 6
        # Algorithm 2 over the ranks: K^s and gamma^s come from the job's N (5), not from the shard's 3 or 2
        eng2 = OracleEngine(w, X, Y, x0, first, count)
        sharded.ShardedPRSGD(eng2, w.N, 0, chunks=2).run_time_varying(1, 130, 0.02)
        q.put((rank, first, count, eng.x.copy(), eng.t, eng2.x.copy(), eng2.t))
    finally:
        dist.destroy_process_group()


def test_shard_bounds_and_chunks():
    assert [sharded.shard_bounds(5, 2, r) for r in range(2)] == [(0, 3), (3, 2)]
    assert [sharded.shard_bounds(64, 8, r) for r in range(8)] == [(8 * r, 8) for r in range(8)]
    got = sharded.column_chunks(2784, 4)
    assert got[0][0] == 0 and sum(n for _, n in got) == 2784 and all(c % 4 == 0 and n % 4 == 0 for c, n in got)
    assert sharded.column_chunks(8, 16) == [(0, 4), (4, 4)]


def test_two_ranks_reproduce_the_single_process_run():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=150) for _ in procs)
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    w = synth.Workload("t", 5, (6, 5, 4), 4, 0.05, 3, 8, 0, 16, mean_shift=0.5, gumbel=True, seed=9)
    X, Y = synth.make_pools(w)
    x0 = synth.init_params(w.dims, w.seed).astype(np.float64)
    want = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, w.I, 7, orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed))
    got = np.concatenate([r[3] for r in res])
    assert [r[4] for r in res] == [7, 7]
    assert got.shape == want.shape and np.allclose(got, want, atol=1e-13)
    assert np.abs(got[0] - got[4]).max() > 1e-6        # t = 7 is one step past the average: workers differ again
    sched = [(K, g * 0.02) for (K, g) in orc.alg2_schedule(w.N, 130)]
    assert max(K for K, _ in sched) == 2               # (K^s changes inside the run: ceil(s^(1/3) / 5) = 2 from s = 126)
    want2 = orc.pr_sgd_time_varying(np.tile(x0, (w.N, 1)), sched, orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed))
    got2 = np.concatenate([r[5] for r in res])
    assert [r[6] for r in res] == [sum(K for K, _ in sched)] * 2
    assert np.allclose(got2, want2, atol=1e-9)              # (the library returns gamma^s as a float)
