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


class OracleEngine:
    """Stand-in shard: rows first..first+count of the oracle's state, padded to a multiple of 4 columns."""

    def __init__(self, w, X, Y, x0, first, count):
        self.w, self.first, self.count, self.t = w, first, count, 0
        self.m = x0.size
        self.m_pad = (self.m + 3) // 4 * 4
        self.x = np.tile(x0.astype(np.float64), (count, 1))
        g = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
        self.fn = lambda i, t, xi: g(self.first + i, t, xi)      # local row i is global worker first + i

    def new_row(self):
        return torch.zeros(self.m_pad, dtype=torch.float64)

    def get_step(self):
        return self.t

    def local_steps(self, k):
        self.x = orc.pr_sgd(self.x, self.w.gamma, 0, k, self.fn, t0=self.t)
        self.t += k

    def partial_sum(self, row, c0, n):
        s = np.zeros(self.m_pad)
        s[:self.m] = self.x.sum(0)
        row[c0:c0 + n] = torch.from_numpy(s[c0:c0 + n])

    def assign_rows(self, row, divisor, c0, n):
        hi = min(c0 + n, self.m)
        if hi > c0:
            self.x[:, c0:hi] = (row[c0:hi].numpy() / divisor)[None, :]


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
        q.put((rank, first, count, eng.x.copy(), eng.t))
    finally:
        dist.destroy_process_group()


def test_shard_bounds_and_chunks():
    assert [sharded.shard_bounds(5, 2, r) for r in range(2)] == [(0, 3), (3, 2)]
    assert [sharded.shard_bounds(64, 8, r) for r in range(8)] == [(8 * r, 8) for r in range(8)]
    got = sharded.column_chunks(2784, 4)
    assert got[0][0] == 0 and sum(n for _, n in got) == 2784 and all(c % 4 == 0 and n % 4 == 0 for c, n in got)
    assert sharded.column_chunks(8, 16) == [(0, 4), (4, 4)]


@pytest.mark.timeout(180)
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
