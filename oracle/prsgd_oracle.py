"""fp64 CPU oracle for Parallel Restarted SGD (PR-SGD).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
path is checked against.  It shares no code with the CUDA library and the
library never calls it; only the tests, the smoke check and the CPU-baseline
leg of the benchmark import it.

What is implemented (all arithmetic in float64):

* Algorithm 1 (PR-SGD): every worker i takes x_i <- x_i - gamma * G_i, and when
  t mod I == 0 the node average y = (1/N) sum_i x_i replaces every x_i.  The
  "restart" reading is the default: on an averaging iteration the local step
  is taken first and the models are averaged afterwards, so that each epoch of
  I iterations starts with all workers at the same point (the paragraph after
  Algorithm 1; Algorithm 2 and 3 are written in exactly this form).  The
  literal reading of Algorithm 1's printed update (gradient sampled at the
  un-averaged x_i^{t-1}, then x_i^t = y - gamma G_i^t) is available with
  ``literal=True``; it obeys the same mean dynamics (Eq. overline-x-update)
  but is not the target of the CUDA path.  PARITY UNPINNED for literal mode
  beyond the mean-dynamics and telescoping invariants.
* Algorithm 2 (time-varying rates, epochs of length K^s) and Algorithm 3
  (per-worker epoch lengths I_i) as schedules over the same step.
* The local step with momentum used in the paper's experiment (heavy-ball form, momentum buffers
  local by default; what happens to them at a restart is not stated in the paper).
* The stochastic gradient of the workload: an MLP with ReLU hidden layers and
  softmax cross-entropy averaged over the minibatch.  The paper leaves F_i
  generic; this is the F_i of the workloads.
* The minibatch draw zeta_i^t: an integer function of (seed, i, t) built from
  the SplitMix64 output function (Steele, Lea, Flood, OOPSLA 2014).

Convergence statements (Theorems 1-3, Corollaries 1-2) are expectations with
unknown constants: PARITY UNPINNED, nothing here evaluates them.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------
# minibatch draw (integer only)
# --------------------------------------------------------------------------
_MASK64 = (1 << 64) - 1
_GAMMA64 = 0x9E3779B97F4A7C15  # SplitMix64 increment (odd, 2^64 / golden ratio)


def splitmix64_mix(z: int) -> int:
    """Output function of SplitMix64: the 64-bit finaliser applied to a state word."""
    z &= _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def splitmix64_stream(seed: int, count: int) -> List[int]:
    """First ``count`` outputs of a SplitMix64 generator seeded with ``seed``."""
    out, s = [], seed & _MASK64
    for _ in range(count):
        s = (s + _GAMMA64) & _MASK64
        out.append(splitmix64_mix(s))
    return out


def draw_block(seed: int, i: int, t: int, n_blocks: int) -> int:
    """Index of the minibatch block worker i uses at iteration t (t >= 1).

    zeta_i^t must be independent across workers and iterations (Introduction,
    the paragraph defining G_i^t).  The t-th output of a SplitMix64 stream keyed
    by ``seed`` is mixed with the worker index through a second application of
    the same output function; the block is that word modulo the number of
    blocks (draw with replacement).
    """
    u = splitmix64_mix((seed + _GAMMA64 * t) & _MASK64)
    v = splitmix64_mix((u + _GAMMA64 * (i + 1)) & _MASK64)
    return v % n_blocks


# --------------------------------------------------------------------------
# the workload's F_i: MLP + softmax cross-entropy (mean over the minibatch)
# --------------------------------------------------------------------------
def param_count(dims: Sequence[int]) -> int:
    return sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))


def unpack(x: np.ndarray, dims: Sequence[int]) -> List[Tuple[np.ndarray, np.ndarray]]:
    """Views (W_l [d_l, d_{l-1}], b_l [d_l]) into a flat vector in canonical order."""
    out, off = [], 0
    for l in range(len(dims) - 1):
        fi, fo = dims[l], dims[l + 1]
        W = x[off:off + fo * fi].reshape(fo, fi)
        off += fo * fi
        b = x[off:off + fo]
        off += fo
        out.append((W, b))
    assert off == x.shape[0]
    return out


def mlp_loss_grad(x: np.ndarray, dims: Sequence[int], Xb: np.ndarray, yb: np.ndarray) -> Tuple[float, np.ndarray]:
    """Loss F(x; minibatch) and its gradient, flat in canonical order.

    a_0 = Xb;  z_l = a_{l-1} W_l^T + b_l;  a_l = max(z_l, 0) for l < L;
    F = (1/B) sum_b [ logsumexp(z_L[b,:]) - z_L[b, y_b] ].
    ReLU derivative at exactly 0 is 0.
    """
    x = np.asarray(x, dtype=np.float64)
    a = [np.asarray(Xb, dtype=np.float64)]
    layers = unpack(x, dims)
    L = len(layers)
    B = a[0].shape[0]
    zs = []
    for l, (W, b) in enumerate(layers):
        z = a[-1] @ W.T + b
        zs.append(z)
        if l < L - 1:
            a.append(np.maximum(z, 0.0))
    zL = zs[-1]
    mx = zL.max(axis=1, keepdims=True)
    lse = mx[:, 0] + np.log(np.exp(zL - mx).sum(axis=1))
    rows = np.arange(B)
    loss = float(np.mean(lse - zL[rows, yb]))
    delta = np.exp(zL - lse[:, None])
    delta[rows, yb] -= 1.0
    delta /= B
    g = np.empty_like(x)
    grads = unpack(g, dims)
    for l in range(L - 1, -1, -1):
        W, _ = layers[l]
        gW, gb = grads[l]
        gW[...] = delta.T @ a[l]
        gb[...] = delta.sum(axis=0)
        if l > 0:
            delta = (delta @ W) * (zs[l - 1] > 0.0)
    return loss, g


# --------------------------------------------------------------------------
# Algorithm 1
# --------------------------------------------------------------------------
GradFn = Callable[[int, int, np.ndarray], np.ndarray]  # (worker i, iteration t, x_i^{t-1}) -> G_i^t


def node_average(x: np.ndarray) -> np.ndarray:
    """y = (1/N) sum_i x_i, summed in worker-index order (Algorithm 1, the node average)."""
    y = np.zeros(x.shape[1], dtype=np.float64)
    for i in range(x.shape[0]):
        y += x[i]
    return y / x.shape[0]


def pr_sgd(x: np.ndarray, gamma: float, I: int, T: int, grad_fn: GradFn, t0: int = 0,
           literal: bool = False, on_step: Optional[Callable] = None) -> np.ndarray:
    """Run iterations t0+1 .. t0+T of Algorithm 1 on the stacked state x [N, m] (a copy is returned).

    I = 0 means the models are never averaged by this loop.
    ``on_step(t, x_before, G, x_after, averaged)`` is called once per iteration.
    """
    x = np.array(x, dtype=np.float64, copy=True)
    N = x.shape[0]
    for t in range(t0 + 1, t0 + T + 1):
        G = np.stack([np.asarray(grad_fn(i, t, x[i]), dtype=np.float64) for i in range(N)])
        before = x.copy() if on_step is not None else None
        averaging = I > 0 and t % I == 0
        if literal:
            if averaging:
                x = node_average(x)[None, :] - gamma * G
            else:
                x = x - gamma * G
        else:
            x = x - gamma * G
            if averaging:
                x[:] = node_average(x)[None, :]
        if on_step is not None:
            on_step(t, before, G, x.copy(), averaging)
    return x


def mlp_grad_fn(dims: Sequence[int], X: np.ndarray, Y: np.ndarray, B: int, seed: int,
                losses: Optional[dict] = None, draws: Optional[dict] = None) -> GradFn:
    """G_i^t for the MLP workload: worker i's gradient on the block draw_block(seed, i, t)."""
    n_blocks = X.shape[1] // B

    def fn(i: int, t: int, xi: np.ndarray) -> np.ndarray:
        blk = draw_block(seed, i, t, n_blocks)
        loss, g = mlp_loss_grad(xi, dims, X[i, blk * B:(blk + 1) * B], Y[i, blk * B:(blk + 1) * B])
        if losses is not None:
            losses[(i, t)] = loss
        if draws is not None:
            draws[(i, t)] = blk
        return g

    return fn


def pr_sgd_momentum(x: np.ndarray, v: np.ndarray, gamma: float, mu: float, I: int, T: int, grad_fn: GradFn,
                    t0: int = 0, average_velocity: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 1 with the local step of the paper's experiment: SGD with momentum mu (Experiment
    section, figure captions: momentum 0.9).  Per worker, in the form of the library the paper used:
        v_i <- mu * v_i + G_i ;   x_i <- x_i - gamma * v_i        (v_i starts at 0)
    On an averaging iteration the models are averaged after the step.  The paper does not say what
    happens to the momentum buffers at a restart: by default each worker keeps its own v_i;
    with average_velocity=True they are averaged like the models.  Returns (x, v), copies.
    """
    x = np.array(x, dtype=np.float64, copy=True)
    v = np.array(v, dtype=np.float64, copy=True)
    N = x.shape[0]
    for t in range(t0 + 1, t0 + T + 1):
        G = np.stack([np.asarray(grad_fn(i, t, x[i]), dtype=np.float64) for i in range(N)])
        v = mu * v + G
        x = x - gamma * v
        if I > 0 and t % I == 0:
            x[:] = node_average(x)[None, :]
            if average_velocity:
                v[:] = node_average(v)[None, :]
    return x, v


# --------------------------------------------------------------------------
# Algorithm 2 and Algorithm 3 (schedules over the same local step)
# --------------------------------------------------------------------------
def alg2_schedule(N: int, S: int) -> List[Tuple[int, float]]:
    """(K^s, gamma^s) for s = 1..S with K^s = ceil(s^(1/3) / N), gamma^s = N / s^(2/3) (Theorem 2)."""
    out = []
    for s in range(1, S + 1):
        c = round(s ** (1.0 / 3.0))
        root = float(c) if c ** 3 == s else s ** (1.0 / 3.0)  # exact at perfect cubes
        out.append((int(np.ceil(root / N)), N / root ** 2))
    return out


def pr_sgd_time_varying(x: np.ndarray, schedule: Sequence[Tuple[int, float]], grad_fn: GradFn) -> np.ndarray:
    """Algorithm 2: epoch s starts from the node average and takes K^s local steps with rate gamma^s.

    Iterations are numbered sequentially across epochs (the re-indexing in the
    paragraph after Algorithm 2).  The state returned is x_i^{S, K^S}: not averaged.
    """
    x = np.array(x, dtype=np.float64, copy=True)
    N, t = x.shape[0], 0
    for (K, g) in schedule:
        x[:] = node_average(x)[None, :]
        for _ in range(K):
            t += 1
            G = np.stack([grad_fn(i, t, x[i]) for i in range(N)])
            x = x - g * G
    return x


def pr_sgd_heterogeneous(x: np.ndarray, gamma: float, I_i: Sequence[int], S: int, grad_fn: GradFn) -> np.ndarray:
    """Algorithm 3: in each of S epochs worker i takes I_i local steps from the node average.

    Iterations are numbered t = (s-1) * max_i I_i + k; a worker with I_i < k
    keeps its point (the zero-gradient convention of the Extensions section).
    The state returned is x_i^{S, I_i}: not averaged.
    """
    x = np.array(x, dtype=np.float64, copy=True)
    N, Imax = x.shape[0], max(I_i)
    for s in range(1, S + 1):
        x[:] = node_average(x)[None, :]
        for k in range(1, Imax + 1):
            t = (s - 1) * Imax + k
            for i in range(N):
                if k <= I_i[i]:
                    x[i] = x[i] - gamma * grad_fn(i, t, x[i])
    return x
