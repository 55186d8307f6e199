"""PR-SGD with the N workers sharded over several GPUs, one process per GPU.

Inside an epoch the workers are independent, so each rank runs its own shard with the
single-GPU library; the only exchange is the node average of Algorithm 1, obtained as the paper
suggests by an all-reduce of the local models (Section 2, "Communication Reduction"): every rank
sums its own rows, the m_pad-float row is all-reduced (sum) over ranks, and every rank restarts its
rows at sum / N.  The row is cut into column chunks so that the all-reduce of chunk c overlaps the
local sum of chunk c + 1.

Two partitions of a job over G ranks are provided by `partition`:
  strong: the job's N workers are split, rank g holds the contiguous rows
          [first_g, first_g + count_g) of `shard_bounds` (sizes differ by at most one);
  weak:   every rank holds N workers of a job of N * G workers (rows g * N .. g * N + N - 1).

This module only orchestrates: the local work is done by an *engine* object with
    local_steps(k), get_step(), m_pad, new_row(), set_lr(gamma),
    partial_sum(row, col0, ncols), assign_rows(row, divisor, col0, ncols)
and optionally local_steps_sum(k) + row0() (the last local step of a period leaves the local row sums in
every row, so the separate row-sum pass is saved)
which `paper_1807_06629_b200.binding.PRSGD` provides on the GPU (created with I = 0,
set_worker_offset(first worker of the rank) and set_global_workers(N of the job)).  The collective
is `torch.distributed.all_reduce` on whatever backend the process group uses (NCCL on GPUs).
An engine that has a `stream` attribute (a torch.cuda.Stream) enqueues its kernels there; the
collective orders itself against torch's *current* stream, so every step of the average runs with
the engine's stream made current.
"""
from __future__ import annotations

import contextlib
from typing import List, Optional, Tuple

import torch
import torch.distributed as dist


def shard_bounds(N_global: int, world: int, rank: int) -> Tuple[int, int]:
    """Workers [first, first + count) owned by `rank`: contiguous, sizes differing by at most one."""
    base, extra = divmod(N_global, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def partition(N_cfg: int, world: int, rank: int, scaling: str) -> Tuple[int, int, int]:
    """(first worker, local worker count, workers of the whole job) of `rank` for a configuration of N_cfg workers."""
    if scaling == "strong":
        if world > N_cfg:
            raise ValueError(f"strong scaling needs at least one worker per rank ({N_cfg} workers, {world} ranks)")
        first, count = shard_bounds(N_cfg, world, rank)
        return first, count, N_cfg
    if scaling == "weak":
        return rank * N_cfg, N_cfg, N_cfg * world
    raise ValueError("scaling must be 'weak' or 'strong'")


def column_chunks(m_pad: int, chunks: int) -> List[Tuple[int, int]]:
    """Cut [0, m_pad) into at most `chunks` ranges whose bounds are multiples of 4."""
    chunks = max(1, min(chunks, m_pad // 4))
    per = -(-(m_pad // 4) // chunks) * 4
    out, c0 = [], 0
    while c0 < m_pad:
        n = min(per, m_pad - c0)
        out.append((c0, n))
        c0 += n
    return out


class ShardedPRSGD:
    """Algorithm 1 over all ranks of `group`; `engine` holds this rank's shard of the workers."""

    def __init__(self, engine, N_global: int, I: int, group: Optional[dist.ProcessGroup] = None, chunks: int = 4,
                 fuse_row_sums: bool = True):
        if I < 0:
            raise ValueError("I must be >= 0")
        if getattr(engine, "average_velocity", False):
            raise ValueError("averaged momentum buffers are not supported on a sharded job: "
                             "enable momentum with average_velocity=False")
        self.engine, self.N_global, self.I, self.group = engine, N_global, I, group
        self.fuse_row_sums = fuse_row_sums     # use the engine's local_steps_sum (if it has one) instead of a row-sum pass
        self.stream = getattr(engine, "stream", None)
        with self._on_engine_stream():
            self.row = engine.new_row()
        self.chunks = column_chunks(engine.m_pad, chunks)

    def _on_engine_stream(self):
        """Make the engine's stream torch's current one (the collective orders itself against it)."""
        if isinstance(self.stream, torch.cuda.Stream):
            return torch.cuda.stream(self.stream)
        return contextlib.nullcontext()

    def average(self) -> None:
        """Node average over every worker of every rank, then restart all local rows at it."""
        with self._on_engine_stream():
            handles = []
            for (c0, n) in self.chunks:
                self.engine.partial_sum(self.row, c0, n)
                handles.append(dist.all_reduce(self.row[c0:c0 + n], op=dist.ReduceOp.SUM, group=self.group, async_op=True))
            for (c0, n), h in zip(self.chunks, handles):
                h.wait()
                self.engine.assign_rows(self.row, float(self.N_global), c0, n)

    def average_from_row_sums(self) -> None:
        """Second half of an average whose first half the engine has fused into the last local step
        (`local_steps_sum`: every local row holds the local row sum): all-reduce row 0 in place, chunk by
        chunk, and restart all local rows at sum / N."""
        with self._on_engine_stream():
            row = self.engine.row0()
            handles = [dist.all_reduce(row[c0:c0 + n], op=dist.ReduceOp.SUM, group=self.group, async_op=True)
                       for (c0, n) in self.chunks]
            for (c0, n), h in zip(self.chunks, handles):
                h.wait()
                self.engine.assign_rows(row, float(self.N_global), c0, n)

    def local_steps(self, k: int) -> None:
        """Iterations t+1 .. t+k; averages whenever I > 0 and t mod I == 0 (local step first, then the average)."""
        t = self.engine.get_step()
        end = t + k
        fused = self.fuse_row_sums and hasattr(self.engine, "local_steps_sum")
        while t < end:
            nxt = end if self.I == 0 else min(end, (t // self.I + 1) * self.I)
            averaging = self.I > 0 and nxt % self.I == 0
            if averaging and fused:           # the last local step of the period also forms the local row sums
                self.engine.local_steps_sum(nxt - t)
                self.average_from_row_sums()
            else:
                self.engine.local_steps(nxt - t)
                if averaging:
                    self.average()
            t = nxt

    def run_time_varying(self, s_begin: int, s_end: int, gamma_scale: float = 1.0) -> None:
        """Algorithm 2 over all ranks: epoch s starts from the node average of the whole job and takes
        K^s local steps with rate gamma_scale * gamma^s, both from the job's N (Theorem 2)."""
        if s_begin < 1 or s_end < s_begin:
            raise ValueError("need 1 <= s_begin <= s_end")
        from .binding import prsgd_alg2_schedule      # host-only call of the library (K^s, gamma^s of Theorem 2)
        for s in range(s_begin, s_end + 1):
            K, g = prsgd_alg2_schedule(self.N_global, s)
            self.average()
            self.engine.set_lr(g * gamma_scale)
            self.engine.local_steps(K)
