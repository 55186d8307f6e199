"""Seeded synthetic inputs for PR-SGD runs.

This module only manufactures *inputs*: initial parameters, per-worker data
pools with their labels, and raw stacked vectors for the averaging sweep.  It
holds none of the method's arithmetic (no SGD step, no averaging, no gradient)
and imports neither the CUDA binding nor the CPU oracle, so both sides can be
fed from it without sharing any code of the method itself.

The workloads mirror the five configurations this package is measured on:

  cfg1  N=4   MLP 32-64-10          B=16  gamma=0.05 I=4   T=64    fp32
  cfg2  N=8   MLP 784-512-512-10    B=32  gamma=0.1  I=8   T=1000  fp32
  cfg3  N=16  MLP 3072-1024-1024-10 B=64  gamma=0.05 I in {1,4,16} T=512  bf16 operands
  cfg4  N=64  MLP 1024-2048-2048-1024-100 B=32 gamma=0.05 I=32 T=256     bf16 operands
  cfg5  raw [N, m] vectors, N in {8,64,256}, m in {1e6, 11e6, 25e6}

The paper itself trains ResNet20 on CIFAR10 (Section "Experiment"); that data
set is not used here.  cfg3 is only CIFAR-*shaped* (3072 = 32*32*3 inputs, 10
classes): every value is drawn from a seeded generator.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Sequence, Tuple

import numpy as np

MASTER_SEED = 20180717


@dataclass(frozen=True)
class Workload:
    name: str
    N: int                      # workers
    dims: Tuple[int, ...]       # d_0 .. d_L
    B: int                      # per-worker minibatch
    gamma: float
    I: int                      # averaging interval
    T: int                      # iterations
    precision: int              # 0 = fp32 operands, 1 = bf16 operands
    pool_samples: int           # P, samples in each worker's pool (multiple of B)
    mean_shift: float = 0.0     # std of the per-worker mean mu_i (non-identical D_i)
    gumbel: bool = False        # add Gumbel(0,1) noise to the teacher logits
    seed: int = MASTER_SEED

    @property
    def m(self) -> int:
        return sum(self.dims[l + 1] * self.dims[l] + self.dims[l + 1] for l in range(len(self.dims) - 1))

    @property
    def n_blocks(self) -> int:
        return self.pool_samples // self.B

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _pool(T: int, B: int, cap: int) -> int:
    p = min(T * B, cap)
    return max(B, (p // B) * B)


WORKLOADS = {
    "cfg1": Workload("cfg1", 4, (32, 64, 10), 16, 0.05, 4, 64, 0, _pool(64, 16, 8192), mean_shift=0.5, gumbel=True),
    "cfg2": Workload("cfg2", 8, (784, 512, 512, 10), 32, 0.1, 8, 1000, 0, _pool(1000, 32, 8192)),
    "cfg3": Workload("cfg3", 16, (3072, 1024, 1024, 10), 64, 0.05, 4, 512, 1, _pool(512, 64, 4096), mean_shift=0.5),
    "cfg4": Workload("cfg4", 64, (1024, 2048, 2048, 1024, 100), 32, 0.05, 32, 256, 1, _pool(256, 32, 1024)),
}

SWEEP_N = (8, 64, 256)
SWEEP_M = (1_000_000, 11_000_000, 25_000_000)


def _rng(seed: int, *stream: int) -> np.random.Generator:
    """Counter-based generator keyed by (seed, stream...) so every array has its own stream."""
    ss = np.random.SeedSequence([int(seed)] + [int(s) for s in stream])
    return np.random.Generator(np.random.Philox(ss))


def init_params(dims: Sequence[int], seed: int = MASTER_SEED, stream: int = 1) -> np.ndarray:
    """One draw x^0 in canonical order W_1, b_1, W_2, b_2, ... (W_l row-major [d_l, d_{l-1}]).

    Weights ~ N(0, 1/fan_in) (std = 1/sqrt(d_{l-1})), biases 0.  Drawn in fp64,
    rounded once to fp32: both the oracle and the GPU start from these fp32 values.
    """
    g = _rng(seed, stream)
    parts = []
    for l in range(len(dims) - 1):
        fan_in, fan_out = dims[l], dims[l + 1]
        parts.append((g.standard_normal(fan_out * fan_in) / np.sqrt(fan_in)).astype(np.float32))
        parts.append(np.zeros(fan_out, dtype=np.float32))
    return np.concatenate(parts)


def _teacher_logits(dims: Sequence[int], theta: np.ndarray, X: np.ndarray) -> np.ndarray:
    """Label generator: evaluates the fixed random teacher network on X (fp32, host)."""
    a = X
    off = 0
    L = len(dims) - 1
    for l in range(L):
        fi, fo = dims[l], dims[l + 1]
        W = theta[off:off + fo * fi].reshape(fo, fi)
        off += fo * fi
        b = theta[off:off + fo]
        off += fo
        a = a @ W.T + b
        if l < L - 1:
            np.maximum(a, 0.0, out=a)
    return a


def make_pools(w: Workload, first: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """Per-worker data pools X [N, P, d_0] fp32 and labels Y [N, P] int32.

    Row k holds the pool of worker first + k (a rank that owns a shard of a larger job asks for its
    own workers only; worker i's pool does not depend on which rank generates it).

    x ~ N(mu_i, I) with mu_i = mean_shift * N(0, I) per worker (mu_i = 0 when
    mean_shift = 0); label = argmax of a fixed random teacher MLP of the same
    shape (optionally with Gumbel(0,1) noise on its logits).
    """
    d0, C = w.dims[0], w.dims[-1]
    theta = init_params(w.dims, w.seed, stream=2)
    X = np.empty((w.N, w.pool_samples, d0), dtype=np.float32)
    Y = np.empty((w.N, w.pool_samples), dtype=np.int32)
    for i in range(w.N):
        g = _rng(w.seed, 3, first + i)
        xi = g.standard_normal((w.pool_samples, d0), dtype=np.float32)
        if w.mean_shift != 0.0:
            mu = (w.mean_shift * g.standard_normal(d0)).astype(np.float32)
            xi += mu
        X[i] = xi
        z = _teacher_logits(w.dims, theta, xi)
        if w.gumbel:
            u = g.random((w.pool_samples, C))
            z = z + (-np.log(-np.log(np.clip(u, 1e-300, 1.0 - 1e-16)))).astype(np.float32)
        Y[i] = np.argmax(z, axis=1).astype(np.int32)
    return X, Y


def stacked_vectors(N: int, m: int, seed: int = MASTER_SEED) -> np.ndarray:
    """[N, m] fp32 with iid N(0,1) entries (input of the averaging sweep)."""
    g = _rng(seed, 5, N, m)
    return g.standard_normal((N, m), dtype=np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    return r


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bf16, returned as fp32."""
    return (bf16_bits(x).astype(np.uint32) << 16).view(np.float32).reshape(np.shape(x))
