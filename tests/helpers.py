"""Shared helpers for the parity tests: build a context from a synth.Workload and
run the fp64 oracle on the same inputs."""
import numpy as np

from oracle import prsgd_oracle as orc
from paper_1807_06629_b200 import synth


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def make_inputs(w):
    """(X fp32 as the GPU sees it, Y, x0).  For bf16-operand workloads X is rounded to bf16 once."""
    X, Y = synth.make_pools(w)
    if w.precision == 1:
        X = synth.bf16_round(X)
    x0 = synth.init_params(w.dims, w.seed)
    return X, Y, x0


def make_ctx(w, X, Y, x0=None, I=None, gamma=None):
    import torch
    from paper_1807_06629_b200 import binding
    p = binding.PRSGD(w.N, w.dims, w.B, w.gamma if gamma is None else gamma, w.I if I is None else I,
                      w.precision, w.pool_samples, w.seed)
    dX = torch.from_numpy(X).to("cuda:0")
    if w.precision == 1:
        dX = dX.to(torch.bfloat16)
    p.bind_data(dX.contiguous(), torch.from_numpy(Y).to("cuda:0"))
    if x0 is not None:
        p.set_params(x0)
    return p


def oracle_run(w, X, Y, x_stacked, t0, T, I=None, gamma=None, losses=None, draws=None):
    fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed, losses=losses, draws=draws)
    return orc.pr_sgd(np.asarray(x_stacked, dtype=np.float64), w.gamma if gamma is None else gamma,
                      w.I if I is None else I, T, fn, t0=t0)


def _torch():
    import torch
    return torch


class OracleEngine:
    """Stand-in shard: rows first..first+count of the oracle's state, padded to a multiple of 4 columns."""

    def __init__(self, w, X, Y, x0, first, count):
        self.w, self.first, self.count, self.t, self.gamma = w, first, count, 0, w.gamma
        self.m = x0.size
        self.m_pad = (self.m + 3) // 4 * 4
        self.x = np.tile(x0.astype(np.float64), (count, 1))
        g = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
        self.fn = lambda i, t, xi: g(self.first + i, t, xi)      # local row i is global worker first + i

    def new_row(self):
        return _torch().zeros(self.m_pad, dtype=_torch().float64)

    def get_step(self):
        return self.t

    def set_lr(self, gamma):
        self.gamma = gamma

    def local_steps(self, k):
        self.x = orc.pr_sgd(self.x, self.gamma, 0, k, self.fn, t0=self.t)
        self.t += k

    def partial_sum(self, row, c0, n):
        s = np.zeros(self.m_pad)
        s[:self.m] = self.x.sum(0)
        row[c0:c0 + n] = _torch().from_numpy(s[c0:c0 + n])

    def assign_rows(self, row, divisor, c0, n):
        hi = min(c0 + n, self.m)
        if hi > c0:
            self.x[:, c0:hi] = (row[c0:hi].numpy() / divisor)[None, :]
