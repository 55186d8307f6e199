#!/usr/bin/env python
"""Benchmark of the PR-SGD hot path (Algorithm 1: local SGD steps + periodic node average).

One "step" of this benchmark is one full averaging period of the workload:
I local iterations of all N workers followed by the node average, i.e.
prsgd_local_steps(I).  The metric is worker-steps/s = N * I * steps / time.

Prints ONE JSON line (the last line of stdout).  `value` is timed on the device
with inputs resident in HBM; `e2e` is the same period driven through the C ABI
from pinned HOST buffers (pool upload, local steps, read-back of the node
average).  `configs` carries short runs of the other training configurations.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg4] [--scaling weak|strong] [--impl reference]

Several GPUs: one process per GPU.  Started under torchrun (WORLD_SIZE set) the
script is one rank; started plainly with --gpus N > 1 it starts the N ranks
itself (`launch_ranks`).  The workers are sharded over the ranks (`--scaling
strong`: the configuration's N workers are split; `weak`, the default: every rank
holds N workers of a job of N * G), local steps need no exchange, and the node
average is local row sums + an NCCL all-reduce + the restart.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_1807_06629_b200 import synth

DEFAULT_WORKLOAD = "cfg4"
L2_BYTES = 126 * 1024 * 1024
METRIC = "worker-steps/s"
# the other training configurations, measured briefly in the default run: (workload, I, timed periods)
OTHER_CONFIGS = (("cfg1", 4, 60), ("cfg2", 8, 40), ("cfg3", 1, 60), ("cfg3", 4, 40), ("cfg3", 16, 20))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- ranks
def rank_env():
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) for a plain start."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launch_ranks(n: int, script_args, script: str = None, capture: bool = False, timeout: float = None):
    """Start `script` (this file by default) as n ranks of one node, one process per GPU, the way the
    launcher of torch.distributed does (rendezvous on 127.0.0.1), and wait for them.  Returns the
    CompletedProcess; with capture=True stdout and stderr are captured instead of inherited."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script or os.path.abspath(__file__)]
    cmd += list(script_args)
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", "4")
    return subprocess.run(cmd, env=env, capture_output=capture, text=True, timeout=timeout)


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    """The slowest rank's figure (a multi-GPU time is the maximum over the ranks)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class CudaTimer:
    """CUDA events on torch's current stream, one pair per timed step."""

    def __init__(self, torch, steps):
        self.ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]

    def start(self, k):
        self.ev[k][0].record()

    def stop(self, k):
        self.ev[k][1].record()

    def total_ms(self):
        return sum(a.elapsed_time(b) for a, b in self.ev)


def time_periods(run_period, steps: int, warmup: int, timer, barrier, before_step=None, after_warmup=None) -> float:
    """`warmup` untimed periods, a barrier, then exactly `steps` timed periods and a barrier;
    returns this rank's summed time in ms (the caller takes the maximum over ranks)."""
    for _ in range(warmup):
        run_period()
    barrier()
    if after_warmup is not None:
        after_warmup()
    for k in range(steps):
        if before_step is not None:
            before_step(k)
        timer.start(k)
        run_period()
        timer.stop(k)
    barrier()
    return timer.total_ms()


def result_line(w_cfg: dict, value: float, ms_total: float, steps: int, warmup: int, world: int, scaling: str,
                dtype: str) -> dict:
    """The keys every line of this benchmark carries."""
    return {"metric": METRIC, "value": value, "unit": METRIC, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": scaling, "vs_baseline": None,
            "dtype": dtype, "data": "synthetic", "config": w_cfg}


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines, self.t_mark = index, None, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def mark(self):
        """Start of the timed region: earlier samples (warm-up) are dropped if later ones exist."""
        self.t_mark = time.time()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        import datetime
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]), [nm for k, nm in enumerate(names)
                                                                           if f[4 + k].lower().startswith("active")]))
            except ValueError:
                continue
        timed = [r for r in rows if self.t_mark is not None and r[0] >= self.t_mark - 0.05]
        window = "timed region"
        if not timed:
            timed, window = rows, "warm-up + timed region (timed region shorter than the sampling period)"
        sm, mx, power = [r[1] for r in timed], [r[2] for r in timed], [r[3] for r in timed]
        reasons = sorted({nm for r in timed for nm in r[4]})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "window": window, "reasons": reasons}


# ----------------------------------------------------------------------------- ncu traffic
# dram__bytes_read.sum + dram__bytes_write.sum per plain iteration of one kernel family, from a one-pass ncu
# capture of a SMALL case (cfg4 shapes with `workers` workers, a few hundred MB on the device; summary in
# profiles/).  The update kernels stream every worker's tiles once, so traffic grows in proportion to the
# number of workers: the record is scaled by N / workers.  Valid only while the kernels' source is unchanged.
NCU_TRAFFIC = {
    # profiles/tc_update_kernels_cfg4_N16.md: 556.8 MB read + 555.1 MB written by the four update launches of a plain iteration
    ("cfg4", "update"): {"workers": 16, "bytes_per_iteration": 556.8e6 + 555.1e6, "launches_per_iteration": 4,
                         "kernel_sha256": "eed39e71db2b26704b496876f2f0bfa43b234dcea97e9e5e7b74ff1fc801318f"},
}


def kernel_section_sha(family: str) -> str:
    """Hash of the source text of the kernels a family runs (update: the update kernels and their stage layouts)."""
    import hashlib
    path = os.path.join(ROOT, "paper_1807_06629_b200", "csrc", "kernels_bf16.cuh")
    with open(path) as f:
        src = f.read()
    marks = {"update": ("template <int TN, bool MOM> struct UpdCfg", "// b_l <- b_l - gamma")}
    if family not in marks:
        return ""
    a, b = src.find(marks[family][0]), src.find(marks[family][1])
    return hashlib.sha256(src[a:b].encode()).hexdigest() if 0 <= a < b else ""


def ncu_traffic_per_launch(workload: str, family: str, N: int):
    rec = NCU_TRAFFIC.get((workload.split("-")[0], family))
    if rec is None or rec["bytes_per_iteration"] is None or rec["kernel_sha256"] != kernel_section_sha(family):
        return None
    return rec["bytes_per_iteration"] * (N / rec["workers"]) / rec["launches_per_iteration"]


# ----------------------------------------------------------------------------- byte model
def period_bytes(w: synth.Workload, m_pad: int, sms: int = 148, momentum: bool = False, fused_average: bool = True,
                 fused_epilogues: bool = True, next_forward: bool = True, dx_in_update=True,
                 shared_restart: bool = True, forward_chain: bool = False, head_kernel=1, head_forward: bool = False, common_point: bool = True) -> dict:
    """Algorithmic HBM bytes and launch counts of ONE averaging period (prsgd_local_steps(I) from a period
    boundary) of all N workers, per kernel family: {family: [bytes, launches]}.

    The unit is one parameter of one worker.  bf16 path: a forward GEMM reads the bf16 copy (2 B/param), a dX
    GEMM reads it again (layers >= 2), an update reads and writes the fp32 master (4 + 4) and writes the bf16
    copy (2) (+ 4 + 4 for the momentum buffer); activations, deltas and biases are charged once per use.  fp32
    path: 4 B where bf16 has 2, no bf16 copy.  The launches follow the library's own rules: on a plain
    iteration the update of a layer >= 2 also forms dZ of the layer below when the layer has enough column
    blocks (no dX launch: the mask read and the dZ write move to the update family), and layer 1's update also
    forms the next a_1 when another iteration follows (no write of W_1's bf16 copy, a second minibatch read,
    a_1 written; the next iteration has no layer-1 forward launch); on the averaging iteration a layer with
    enough tiles takes the fused update + average (same bytes as a plain update, dX a launch of its own),
    a smaller one the plain update followed by the node average of its weight segment (8 + 2 B/param).
    Without the fused form the stand-alone average reads and writes the whole store (8 B/word, + 2 B bf16 copy).
    The class layer (at most 128 classes, last hidden width 128..1024, plain step) is one launch of its own
    family ("head"): its forward read of the bf16 copy, its update (10 B/param) and the mask read and dZ write
    of the layer below; a_{L-1} is read once for both products.  With three or more layers (and shared memory
    for a ring of two stages behind the class layer's tiles) the same launch also does the forward GEMM of layer
    L - 1, whose output then stays in shared memory.
    """
    bf = w.precision == 1
    e = 2 if bf else 4
    N, B, d, I = w.N, w.B, w.dims, max(w.I, 1)
    L = len(d) - 1
    upd_b = 8 + (2 if bf else 0) + (8 if momentum else 0)
    epi = bf and fused_epilogues and d[L] <= 128
    fam = {k: [0, 0] for k in ("forward", "softmax", "dx", "update", "update_average", "average", "misc", "head")}
    head_ok = (bf and epi and head_kernel and dx_in_update == 1 and L >= 2 and not momentum
               and d[L - 1] in (128, 256, 512, 1024) and (head_kernel == 2 or N * (d[L - 1] // 128) <= sms))

    def add(name, nbytes):
        fam[name][0] += nbytes
        fam[name][1] += 1
    cp = (d[L] + 15) // 16 * 16
    head_fixed = (8 * cp * 128 + 4 * B * 128 + 2 * B * (cp + 1) * 4 + 768 + 1023) // 1024 * 1024
    head_fwd_ok = head_ok and head_forward and L >= 3 and (227 * 1024 - head_fixed - 1024) // (2 * (16384 + B * 128)) >= 2
    a1_ready = False
    for j in range(1, I + 1):
        averaging = w.I > 0 and j == I
        fuse = averaging and fused_average and (bf or not momentum)     # (the fp32 path has no fused momentum form)
        nxt = bf and next_forward and j < I and not averaging and L > 1 and epi
        # the first iteration of a period starts from N equal rows: launches that only read the weights (and the
        # fused update + average) read one copy for all workers
        wr = 1 if (bf and shared_restart and j == 1 and w.I > 0) else N
        l_first = 2 if a1_ready else 1
        head = head_ok and not (fuse and 2 * ((d[L] + 127) // 128) * ((d[L - 1] + 63) // 64) >= sms)
        head_fwd = head and head_fwd_ok
        l_last = (L - 2 if head_fwd else L - 1) if head else L
        chained = bf and forward_chain and 2 <= l_last - l_first + 1 <= 8      # all layers' forward GEMMs in one launch
        for l in range(l_first, l_last + 1):
            add("forward", wr * d[l] * d[l - 1] * e + N * (d[l] * 4 + B * d[l - 1] * e + B * d[l] * (e if l < L else 4)))
            if chained and l > l_first:
                fam["forward"][1] -= 1
        a1_ready = False
        if not epi:
            add("softmax", N * B * d[L] * (4 + 4 + e))
        small_avg = 0
        common_layers = 0
        if head:
            add("head", N * (d[L] * d[L - 1] * e + B * d[L - 1] * e + (d[L] * d[L - 1] + d[L]) * upd_b + B * d[L - 1] * 2 * e))
            if head_fwd:       # + layer L - 1's forward: its weights and input read, its output neither written nor re-read
                fam["head"][0] += wr * d[L - 1] * d[L - 2] * e + N * (d[L - 1] * 4 + B * d[L - 2] * e) - N * B * d[L - 1] * e
        for l in range(L, 0, -1):
            wl = d[l] * d[l - 1]
            if l == L and head:
                if bf and fuse:
                    small_avg += N * wl * 10
                continue
            tiles64 = ((d[l] + 127) // 128) * ((d[l - 1] + 63) // 64)
            fuse_l = fuse and (not bf or 2 * tiles64 >= sms)
            folds = bf and epi and dx_in_update and (dx_in_update == 2 or ((d[l - 1] + 63) // 64) * N >= 3 * sms or d[l] <= 128)
            upd = N * ((wl + d[l]) * upd_b + B * (d[l] + d[l - 1]) * e)
            if l > 1 and folds and not fuse_l:
                add("update", upd + N * B * d[l - 1] * 2 * e)
            else:
                if l > 1:
                    add("dx", wr * wl * e + N * (B * d[l] * e + B * d[l - 1] * 2 * e))
                if l == 1 and nxt:
                    upd += N * (-wl * 2 + B * d[0] * e + B * d[1] * e + d[1] * 4)
                    a1_ready = True
                if fuse_l:
                    upd -= (N - wr) * wl * 4
                add("update_average" if fuse_l else "update", upd)
                if fuse_l and wr == 1 and not momentum and common_point:
                    common_layers += 1          # from a common point these layers share ONE launch after the dX launches
                    if common_layers > 1:
                        fam["update_average"][1] -= 1
            if bf and fuse and not fuse_l:
                small_avg += N * wl * 10
        if not epi and bf:
            add("misc", 0)
        if bf and fuse:
            add("misc", small_avg)        # bias segments, and the weight segments too small for the fused form, in one launch
        if averaging and not fuse:
            add("average", N * m_pad * (8 + (2 if bf else 0)))
    return fam


def flops_per_worker_step(w: synth.Workload) -> int:
    d, B = w.dims, w.B
    tot = sum(6 * B * d[l] * d[l - 1] for l in range(1, len(d)))
    return tot - 2 * B * d[1] * d[0]


# ----------------------------------------------------------------------------- oracle (CPU baseline)
def oracle_cores() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return 1


def time_oracle(w: synth.Workload, X, Y, x0, budget_s: float = 15.0):
    """Times the fp64 oracle, as it stands, on a bounded sample: all N workers for s iterations."""
    from oracle import prsgd_oracle as orc
    cores = oracle_cores()
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    state = np.tile(x0.astype(np.float64), (w.N, 1))
    t0 = time.perf_counter()
    state = orc.pr_sgd(state, w.gamma, w.I, 1, fn, t0=0)
    t1 = time.perf_counter() - t0
    s = int(max(1, min(w.I, budget_s / max(t1, 1e-6))))
    t0 = time.perf_counter()
    orc.pr_sgd(state, w.gamma, w.I, s, fn, t0=1)
    dt = time.perf_counter() - t0
    return {"value": w.N * s / dt, "unit": METRIC, "cores": cores, "kind": "oracle",
            "sample": f"all {w.N} workers x {s} consecutive iterations of {w.name} (fp64 numpy), {dt:.1f} s"}


def run_reference(args, w):
    """--impl reference: the oracle on the host cores; each step is one iteration of all N workers.
    Under a multi-rank launch rank 0 alone runs and prints; the other ranks exit without work."""
    if rank_env()[0] != 0:
        return
    from oracle import prsgd_oracle as orc
    cores = oracle_cores()
    X, Y = synth.make_pools(w)
    if w.precision == 1:
        X = synth.bf16_round(X)
    x0 = synth.init_params(w.dims, w.seed)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    state = np.tile(x0.astype(np.float64), (w.N, 1))
    t = 0
    for _ in range(args.warmup):
        state = orc.pr_sgd(state, w.gamma, w.I, 1, fn, t0=t); t += 1
    t0 = time.perf_counter()
    for _ in range(args.steps):
        state = orc.pr_sgd(state, w.gamma, w.I, 1, fn, t0=t); t += 1
    dt = time.perf_counter() - t0
    val = w.N * args.steps / dt
    sample = f"each step = 1 iteration of all {w.N} workers of {w.name} (fp64 numpy oracle)"
    line = result_line(workload_config(w), val, 1e3 * dt, args.steps, args.warmup, args.gpus, "weak", "f64")
    line.update({"impl": "reference",
                 "cpu_baseline": {"value": val, "unit": METRIC, "cores": cores, "kind": "oracle", "sample": sample},
                 "e2e": {"value": val, "unit": METRIC, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}})
    print(json.dumps(line))


def workload_config(w, extra=None, momentum=None):
    c = {"workload": w.name, "N": w.N, "dims": list(w.dims), "B": w.B, "gamma": w.gamma, "I": w.I,
         "pool_samples": w.pool_samples, "precision": "bf16 operands / fp32 master" if w.precision else "fp32",
         "step": "one averaging period = prsgd_local_steps(I)"}
    if momentum is not None:
        c["momentum"] = momentum
    if extra:
        c.update(extra)
    return c


# ----------------------------------------------------------------------------- averaging sweep
def averaging_sweep(torch, binding, peaks, dev, points=None):
    """Node-average kernel in isolation on [N, m] fp32: GB/s counting N*m*4 read + N*m*4 written."""
    out = []
    if points is None:
        points = [(N, m) for N in synth.SWEEP_N for m in synth.SWEEP_M]
    for (N, m) in points:
        if True:
            nbytes = N * m * 4
            copies = max(1, int(np.ceil(2 * L2_BYTES / nbytes))) if nbytes <= 2 * L2_BYTES else 1
            bufs = [torch.randn(N, m, device=dev, dtype=torch.float32) for _ in range(copies)]
            reps = 20
            binding.prsgd_average_rows(bufs[0], N, m)
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev[0].record()
            for r in range(reps):
                binding.prsgd_average_rows(bufs[r % copies], N, m)
            ev[1].record()
            torch.cuda.synchronize()
            ms = ev[0].elapsed_time(ev[1]) / reps
            gbs = 2 * nbytes / ms / 1e6
            out.append({"N": N, "m": m, "us": round(ms * 1e3, 2), "GBps": round(gbs, 1),
                        "frac_of_measured_copy": round(gbs / peaks["hbm_gbs"], 4),
                        "frac_of_8TBps": round(gbs / 8000.0, 4), "rotating_buffers": copies})
            del bufs
            torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- one configuration on the GPU
def measure_config(torch, w_cfg, args, dev, rank, world, scaling, steps, warmup, peaks, sharded_mode,
                   with_e2e, with_clocks):
    """Builds the context of this rank's shard of `w_cfg`, times `steps` periods on the device (CUDA events,
    maximum over ranks), repeats the region with an event pair around every launch for the roofline, and
    (with_e2e) times the same periods driven from pinned host buffers.  Returns (result dict, state for the
    CPU-oracle leg)."""
    import torch.distributed as dist
    from paper_1807_06629_b200 import binding, sharded
    first, n_local, n_global = sharded.partition(w_cfg.N, world, rank, scaling) if sharded_mode else (0, w_cfg.N, w_cfg.N)
    # the pool holds one averaging period's worth of fresh samples per worker (I blocks of B; at least 4),
    # which is what the end-to-end arm uploads from the host before every period
    w = w_cfg.with_(N=n_local, pool_samples=max(w_cfg.I, 4) * w_cfg.B)
    x0 = synth.init_params(w.dims, w.seed)              # the same x^0 on every rank
    X, Y = synth.make_pools(w, first)                   # this rank's workers of the job
    if w.precision == 1:
        X = synth.bf16_round(X)
    tdt = torch.bfloat16 if w.precision == 1 else torch.float32
    hX = torch.from_numpy(X).to(tdt).contiguous().pin_memory()
    hY = torch.from_numpy(Y).contiguous().pin_memory()
    p = binding.PRSGD(w.N, w.dims, w.B, w.gamma, 0 if sharded_mode else w.I, w.precision, w.pool_samples, w.seed,
                      device=dev)
    p.bind_data(hX.to(dev), hY.to(dev))
    p.set_params(x0)
    job = None
    if sharded_mode:          # local steps on the shard, node average = local sums + NCCL all-reduce + restart
        p.set_worker_offset(first)
        p.set_global_workers(n_global)
        job = sharded.ShardedPRSGD(p, n_global, w.I)

    def run_period():
        if job is not None:
            job.local_steps(w.I)
        else:
            p.local_steps(w.I)
    if args.update_tile is not None:
        p.set_option(binding.OPT_UPDATE_TILE, args.update_tile)
    if args.momentum is not None:
        p.enable_momentum(args.momentum)
    for flag, opt in ((args.no_fuse, binding.OPT_FUSED_AVERAGE), (args.no_dx_in_update, binding.OPT_DX_IN_UPDATE),
                      (args.no_next_forward, binding.OPT_NEXT_FORWARD), (args.no_early_loads, binding.OPT_EARLY_LOADS),
                      (args.no_fused_epilogues, binding.OPT_FUSED_EPILOGUES),
                      (args.no_shared_restart, binding.OPT_SHARED_RESTART),
                      (args.no_forward_chain, binding.OPT_FORWARD_CHAIN),
                      (args.no_head_kernel, binding.OPT_HEAD_KERNEL), (args.no_common_point, binding.OPT_COMMON_POINT),
                      (args.no_tiled_weights, binding.OPT_TILED_WEIGHTS), (args.no_overlap_update, binding.OPT_OVERLAP_UPDATE)):
        if flag:
            p.set_option(opt, 0)
    if args.head_forward:
        p.set_option(binding.OPT_HEAD_FORWARD, 1)
    if args.head_kernel_always:
        p.set_option(binding.OPT_HEAD_KERNEL, 2)
    if args.fold_all_dx:
        p.set_option(binding.OPT_DX_IN_UPDATE, 2)
    if args.dx_own_pairs:
        p.set_option(binding.OPT_DX_SHARED_PAIR, 0)
    if args.forward_chain:
        p.set_option(binding.OPT_FORWARD_CHAIN, 1)
    if args.worker_groups is not None:
        p.set_option(binding.OPT_WORKER_GROUPS, args.worker_groups)
    working_set = p.params.numel() * 4 + (p.shadow.numel() * 2 if p.shadow is not None else 0)
    need_flush = working_set <= 2 * L2_BYTES
    flush = torch.empty(3 * L2_BYTES // 4, dtype=torch.float32, device=dev) if need_flush else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def flush_l2(k):
        if flush is not None:
            flush.fill_(float(k))

    # ---- device-timed region: K periods, inputs resident in HBM -------------------------
    sampler = ClockSampler(torch.cuda.current_device()) if with_clocks else None
    if sampler:
        sampler.start()
    launches0 = [0]

    def after_warmup():
        p.sync()
        if sampler:
            sampler.mark()
        launches0[0] = p.get_launch_count()
    ms_local = time_periods(run_period, steps, warmup, CudaTimer(torch, steps), barrier, flush_l2, after_warmup)
    clocks = sampler.stop() if sampler else None
    launches = p.get_launch_count() - launches0[0]
    ms_total = max_over_ranks(ms_local, world, dev)
    worker_steps = n_global * w.I * steps          # what all ranks processed
    value = worker_steps / (ms_total * 1e-3)

    # ---- per-kernel pass (same region again with an event pair around every launch) ------
    p.set_option(binding.OPT_PROFILE, 1)
    p.get_profile()
    for k in range(steps):
        flush_l2(k)
        run_period()
    prof = p.get_profile()
    p.set_option(binding.OPT_PROFILE, 0)
    fam_model = period_bytes(w, p.m_pad, torch.cuda.get_device_properties(dev).multi_processor_count,
                             momentum=args.momentum is not None, fused_average=not args.no_fuse,
                             fused_epilogues=not args.no_fused_epilogues, next_forward=not args.no_next_forward,
                             dx_in_update=0 if args.no_dx_in_update else (2 if args.fold_all_dx else 1),
                             shared_restart=not args.no_shared_restart, forward_chain=args.forward_chain,
                             head_kernel=0 if args.no_head_kernel else (2 if args.head_kernel_always else 1),
                             head_forward=args.head_forward, common_point=not args.no_common_point)
    if sharded_mode:          # a shard's period ends with row sums fused into the last step; the restart is a pass of its own
        fam_model["average"] = [fam_model["average"][0] + p.m_pad * 4 + w.N * p.m_pad * (4 + (2 if w.precision == 1 else 0)),
                                fam_model["average"][1] + 4]
    fams = {k: v for k, v in prof.items() if v[1] > 0 and fam_model.get(k, [0, 0])[0] > 0}
    dom = max(fams, key=lambda k: fams[k][0])
    dom_ms, dom_launches = fams[dom]
    dom_bytes, dom_per_period = fam_model[dom]
    achieved = dom_bytes * steps / (dom_ms * 1e-3) / 1e9
    prof_sum = sum(x[0] for x in prof.values())
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                "traffic": ncu_traffic_per_launch(w_cfg.name, dom, w.N),
                "avg_launch_us": 1e3 * dom_ms / dom_launches,
                "algorithmic_bytes_per_launch": dom_bytes / max(dom_per_period, 1),
                "launches_per_period": {"counted": dom_launches / steps, "model": dom_per_period},
                "family_us_per_iteration": {k: round(1e3 * v[0] / (steps * max(w.I, 1)), 2) for k, v in prof.items() if v[1]},
                "share_of_step_time": {k: round(v[0] / prof_sum, 4) for k, v in prof.items() if v[1]}}
    tflops = flops_per_worker_step(w) * value / world / 1e12
    res = {"value": value, "ms_total": ms_total, "launches": launches, "roofline": roofline, "clocks": clocks,
           "gemm_tflops": tflops, "need_flush": need_flush, "n_local": n_local, "n_global": n_global, "w": w,
           "pool_samples": w.pool_samples}

    # ---- end to end through the C ABI from pinned host buffers ---------------------------
    # Every period: fresh pools come from pinned host memory (staged on a copy stream into the spare
    # device pools while the previous period computes, then swapped in), the period runs, and the node
    # average is read back into pinned host memory.
    if with_e2e:
        avg_host = [torch.empty(p.m, dtype=torch.float32).pin_memory() for _ in range(2)]
        copy_stream = torch.cuda.Stream(device=dev)
        read_stream = torch.cuda.Stream(device=dev)
        p.stage_data(hX, hY, copy_stream)
        for k in range(2):
            p.swap_data(); p.stage_data(hX, hY, copy_stream); run_period(); p.get_average_async(avg_host[k % 2], read_stream)
        read_stream.synchronize()
        barrier()
        t0 = time.perf_counter()
        for k in range(steps):
            p.swap_data()                          # pools uploaded during the previous period become current
            p.stage_data(hX, hY, copy_stream)      # H2D of the next period's pools, overlapped with this period
            run_period()
            # D2H of the result: the mean is formed on the training stream, its copy to pinned host memory overlaps
            # the next period (two host buffers; the last copy is waited for inside the timed region)
            p.get_average_async(avg_host[k % 2], read_stream)
        read_stream.synchronize()
        barrier()
        copy_stream.synchronize()
        e2e_s = max_over_ranks(time.perf_counter() - t0, world, dev)
        res["e2e"] = {"value": worker_steps / e2e_s, "unit": METRIC,
                      "h2d_bytes_per_step": hX.numel() * hX.element_size() + hY.numel() * 4,
                      "d2h_bytes_per_step": p.m * 4}
    p.sync()
    p.close()
    return res, (w, X, Y, x0)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=24)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="several GPUs: weak = N workers per rank (N * G in all), strong = the configuration's N split over the ranks")
    ap.add_argument("--interval", type=int, default=None, help="override the averaging interval I")
    ap.add_argument("--workers", type=int, default=None, help="override N (smaller cases for profiler captures)")
    ap.add_argument("--momentum", type=float, default=None, help="local step with momentum mu (the paper's experiment used 0.9)")
    ap.add_argument("--update-tile", type=int, default=None, help="tile width of the update kernel (64 or 128)")
    ap.add_argument("--no-fuse", action="store_true",
                    help="averaging iterations run as update + stand-alone averaging kernel instead of the fused pass")
    ap.add_argument("--no-fused-epilogues", action="store_true",
                    help="softmax-CE gradient and bias steps as kernels of their own instead of GEMM epilogues")
    ap.add_argument("--no-dx-in-update", action="store_true",
                    help="separate dX launches instead of forming dZ of the layer below inside the update launch")
    ap.add_argument("--dx-own-pairs", action="store_true",
                    help="64-wide update + dX with a pair of bf16 tiles per stage instead of one shared pair")
    ap.add_argument("--fold-all-dx", action="store_true",
                    help="form dZ of the layer below inside the update launch for every layer, whatever its size")
    ap.add_argument("--no-shared-restart", action="store_true",
                    help="the iteration after an average reads every worker's own copy of the common point")
    ap.add_argument("--worker-groups", type=int, default=None,
                    help="plain iterations as this many independent launch chains (one per group of workers) on streams of their own")
    ap.add_argument("--forward-chain", action="store_true", help="one forward launch for all layers")
    ap.add_argument("--no-forward-chain", action="store_true",
                    help="one forward launch per layer instead of one launch for all layers")
    ap.add_argument("--head-kernel-always", action="store_true",
                    help="the class layer as one launch of clusters even when its CTAs need more than one wave")
    ap.add_argument("--no-overlap-update", action="store_true",
                    help="layer 2's update before layer 1's, each launch after the other, instead of beside it")
    ap.add_argument("--no-tiled-weights", action="store_true",
                    help="hidden layers' weight segments row-major instead of as 128 x 64 tiles")
    ap.add_argument("--no-common-point", action="store_true",
                    help="an averaging iteration that starts from N equal rows forms and sums the N stepped models one by one")
    ap.add_argument("--head-forward", action="store_true",
                    help="the forward GEMM of layer L - 1 inside the class layer's cluster launch instead of a launch of its own")
    ap.add_argument("--no-head-kernel", action="store_true",
                    help="the class layer's forward GEMM and update as launches of their own instead of one launch of clusters")
    ap.add_argument("--no-next-forward", action="store_true",
                    help="layer 1's update does not form the next iteration's a_1")
    ap.add_argument("--no-early-loads", action="store_true",
                    help="no tile requests ahead of a kernel's dependency wait")
    ap.add_argument("--force-sharded", action="store_true",
                    help="run the multi-GPU code path (sharded workers + all-reduce average) even on one GPU")
    ap.add_argument("--no-sweep", action="store_true", help="skip the averaging-kernel sweep")
    ap.add_argument("--sweep-only", default=None, metavar="NxM[,NxM...]",
                    help="run only the averaging kernel on these [N, m] shapes (small cases for profiler captures) and print their line")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle timing")
    ap.add_argument("--no-configs", action="store_true", help="skip the short runs of the other configurations")
    args = ap.parse_args(argv)
    if args.warmup < 3:
        args.warmup = 3
    return args


def main(argv=None):
    args = parse_args(argv)
    w = synth.WORKLOADS[args.config]
    if args.interval is not None:
        w = w.with_(I=args.interval)
    if args.workers is not None:
        w = w.with_(N=args.workers, name=f"{w.name}-N{args.workers}")
    if args.impl == "reference":
        return run_reference(args, w.with_(pool_samples=max(w.I, 4) * w.B))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # a plain start that asks for several GPUs: start one rank per GPU and let rank 0 print the line
        raise SystemExit(launch_ranks(args.gpus, sys.argv[1:] if argv is None else list(argv)).returncode)

    import torch
    import torch.distributed as dist
    from paper_1807_06629_b200 import _build
    rank, local_rank, world = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    if rank == 0:
        _build.build_library()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    # everything below (torch copies, the library's kernels, the timing events) runs on one side stream:
    # the library replays captured periods as CUDA graphs, which the legacy default stream cannot capture
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))
    sharded_mode = world > 1 or args.force_sharded
    if sharded_mode:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device(dev))
        dist.barrier()            # (also: the library rank 0 may just have built is in place for every rank)
    from paper_1807_06629_b200 import binding
    peaks = load_peaks()
    if args.sweep_only:
        pts = [tuple(int(v) for v in p.lower().split("x")) for p in args.sweep_only.split(",")]
        print(json.dumps({"averaging_sweep": averaging_sweep(torch, binding, peaks, dev, pts)}), flush=True)
        return

    res, (wl, X, Y, x0) = measure_config(torch, w, args, dev, rank, world, args.scaling, args.steps, args.warmup, peaks,
                                         sharded_mode, with_e2e=True, with_clocks=True)
    if sharded_mode:
        how = (f"{args.scaling} scaling: rank g holds {res['n_local']} of the job's {res['n_global']} workers "
               f"(rows [g*N/G, (g+1)*N/G)); node average = local row sums + NCCL all-reduce + restart")
    else:
        how = "single GPU"
    cfg = workload_config(w.with_(N=res["n_global"], pool_samples=res["pool_samples"]),
                          {"l2": "L2 flushed between timed steps" if res["need_flush"] else "parameter store + shadow larger than L2",
                           "multi_gpu": how}, momentum=args.momentum)
    out = result_line(cfg, res["value"], res["ms_total"], args.steps, args.warmup, world,
                      args.scaling if world > 1 else "weak", "bf16" if w.precision else "f32")
    out.update({"clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": res["launches"], "roofline": res["roofline"],
                "gemm_tflops": res["gemm_tflops"],
                "gemm_frac_of_bf16_peak": res["gemm_tflops"] / peaks["bf16_tflops_sustained"]})
    if world == 1 and not args.force_sharded:
        default_run = args.config == DEFAULT_WORKLOAD and args.interval is None and args.workers is None
        if default_run and not args.no_configs:
            others = []
            for name, I, k in OTHER_CONFIGS:
                wo = synth.WORKLOADS[name].with_(I=I)
                r, _ = measure_config(torch, wo, args, dev, rank, world, "weak", k, 3, peaks, False,
                                      with_e2e=False, with_clocks=False)
                rf = r["roofline"]
                others.append({"workload": name, "N": wo.N, "I": I, "value": round(r["value"], 1), "unit": METRIC,
                               "steps": k, "ms_per_step": round(r["ms_total"] / k, 4),
                               "dtype": "bf16" if wo.precision else "f32",
                               "dominant_family": rf["kernel"], "achieved_GBps": round(rf["achieved"], 1),
                               "frac_of_measured_copy": round(rf["frac"], 4),
                               "family_us_per_iteration": rf["family_us_per_iteration"],
                               "gemm_tflops": round(r["gemm_tflops"], 2),
                               "l2": "L2 flushed between timed steps" if r["need_flush"] else "store larger than L2"})
                torch.cuda.empty_cache()
            out["configs"] = others
        if not args.no_sweep:
            out["averaging_sweep"] = averaging_sweep(torch, binding, peaks, dev)
        if not args.no_cpu:
            out["cpu_baseline"] = time_oracle(wl, X, Y, x0)
    if sharded_mode:
        dist.barrier()
    if rank == 0:
        sys.stdout.flush()
        print(json.dumps(out), flush=True)          # the JSON line is the last thing this run prints
    if sharded_mode:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
