"""ctypes binding of libprsgd.so: argument marshalling only.

Every function of include/prsgd.h is available under its own name on `lib`
(e.g. ``lib.prsgd_local_steps``).  The `PRSGD` class wraps a context together
with the torch tensors that own its device memory; its methods are named after
the C calls and do no arithmetic of their own.  There is no CPU fallback: if
the shared library is missing this module raises on import.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

from ._build import LIB_PATH

PRSGD_OK = 0
PRECISION_FP32, PRECISION_BF16 = 0, 1
X_FP32, X_BF16 = 0, 1
OPT_FUSED_AVERAGE = 1
OPT_PROFILE = 2
OPT_UPDATE_TILE = 3
OPT_GRAPH = 4
OPT_FUSED_EPILOGUES = 5
OPT_EARLY_LOADS = 6
OPT_NEXT_FORWARD = 7
OPT_DX_IN_UPDATE = 8
OPT_CHECK_FINITE = 9
OPT_SHARED_RESTART = 10
OPT_FORWARD_CHAIN = 11
OPT_WORKER_GROUPS = 12
OPT_DX_SHARED_PAIR = 13
OPT_HEAD_KERNEL = 14
OPT_COMMON_POINT = 15
OPT_SPLIT_BLOCKS = 16
OPT_HEAD_FORWARD = 17
OPT_MERGED_SMALL_AVERAGE = 18
OPT_TILED_WEIGHTS = 19
OPT_OVERLAP_UPDATE = 20
ERR_DEVICE_TIMEOUT, ERR_NONFINITE = -6, -7
KERNEL_FAMILIES = ("forward", "softmax", "dx", "update", "update_average", "average", "misc", "head")
MAX_LAYERS = 16

EXPORTS = [
    "prsgd_layout", "prsgd_workspace_bytes", "prsgd_create", "prsgd_destroy", "prsgd_bind_data",
    "prsgd_upload_data", "prsgd_set_params", "prsgd_set_params_stacked", "prsgd_get_params_stacked",
    "prsgd_get_params", "prsgd_local_steps", "prsgd_average", "prsgd_get_average", "prsgd_get_average_async", "prsgd_get_losses",
    "prsgd_get_draws", "prsgd_set_lr", "prsgd_set_interval", "prsgd_set_active", "prsgd_get_step",
    "prsgd_set_step", "prsgd_set_option", "prsgd_get_launch_count", "prsgd_get_profile", "prsgd_sync", "prsgd_last_error",
    "prsgd_average_rows", "prsgd_draw_block", "prsgd_mean_rows_noalloc", "prsgd_selftest_wait_expiry",
    "prsgd_clear_device_error", "prsgd_enable_momentum", "prsgd_get_velocity_stacked",
    "prsgd_set_worker_offset", "prsgd_partial_sum", "prsgd_assign_rows", "prsgd_stage_data", "prsgd_swap_data",
    "prsgd_alg2_schedule", "prsgd_run_time_varying", "prsgd_run_heterogeneous_epoch",
    "prsgd_set_global_workers", "prsgd_check_finite", "prsgd_local_steps_sum",
]
NOALLOC_MAX_M = 1 << 20


class ModelSpec(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("dims", C.POINTER(C.c_int32)), ("batch", C.c_int32),
                ("precision", C.c_int32), ("pool_samples", C.c_int64), ("draw_seed", C.c_uint64)]


class Layout(C.Structure):
    _fields_ = [("m", C.c_int64), ("m_pad", C.c_int64), ("w_off", C.c_int64 * MAX_LAYERS),
                ("b_off", C.c_int64 * MAX_LAYERS)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it first (python -m paper_1807_06629_b200._build). "
            "There is no fallback path.")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    spec_p, szp = C.POINTER(ModelSpec), C.POINTER(C.c_size_t)
    sig = {
        "prsgd_layout": (C.c_int, [spec_p, C.POINTER(Layout)]),
        "prsgd_workspace_bytes": (C.c_int, [i32, spec_p, szp, szp, szp]),
        "prsgd_create": (C.c_int, [i32, spec_p, C.c_float, i32, vp, vp, vp, vp, C.POINTER(vp)]),
        "prsgd_destroy": (C.c_int, [vp]),
        "prsgd_bind_data": (C.c_int, [vp, vp, i32, vp]),
        "prsgd_upload_data": (C.c_int, [vp, vp, vp]),
        "prsgd_set_params": (C.c_int, [vp, vp, i32, C.c_int]),
        "prsgd_set_params_stacked": (C.c_int, [vp, vp, C.c_int]),
        "prsgd_get_params_stacked": (C.c_int, [vp, vp, C.c_int]),
        "prsgd_get_params": (C.c_int, [vp, vp, i32, C.c_int]),
        "prsgd_local_steps": (C.c_int, [vp, i64]),
        "prsgd_local_steps_sum": (C.c_int, [vp, i64]),
        "prsgd_average": (C.c_int, [vp]),
        "prsgd_get_average": (C.c_int, [vp, vp, C.c_int]),
        "prsgd_get_average_async": (C.c_int, [vp, vp, vp]),
        "prsgd_get_losses": (C.c_int, [vp, vp]),
        "prsgd_get_draws": (C.c_int, [vp, vp]),
        "prsgd_set_lr": (C.c_int, [vp, C.c_float]),
        "prsgd_set_interval": (C.c_int, [vp, i32]),
        "prsgd_set_active": (C.c_int, [vp, vp]),
        "prsgd_get_step": (C.c_int, [vp, C.POINTER(i64)]),
        "prsgd_set_step": (C.c_int, [vp, i64]),
        "prsgd_set_option": (C.c_int, [vp, i32, i64]),
        "prsgd_get_launch_count": (C.c_int, [vp, C.POINTER(i64)]),
        "prsgd_get_profile": (C.c_int, [vp, i32, C.POINTER(C.c_double), C.POINTER(i64)]),
        "prsgd_sync": (C.c_int, [vp]),
        "prsgd_selftest_wait_expiry": (C.c_int, [vp, i32]),
        "prsgd_clear_device_error": (C.c_int, [vp]),
        "prsgd_enable_momentum": (C.c_int, [vp, C.c_float, vp, C.c_int]),
        "prsgd_get_velocity_stacked": (C.c_int, [vp, vp, C.c_int]),
        "prsgd_alg2_schedule": (C.c_int, [i32, i64, C.POINTER(i64), C.POINTER(C.c_float)]),
        "prsgd_run_time_varying": (C.c_int, [vp, i64, i64, C.c_float]),
        "prsgd_run_heterogeneous_epoch": (C.c_int, [vp, vp]),
        "prsgd_stage_data": (C.c_int, [vp, vp, vp, vp, vp, vp]),
        "prsgd_swap_data": (C.c_int, [vp]),
        "prsgd_set_worker_offset": (C.c_int, [vp, i32]),
        "prsgd_set_global_workers": (C.c_int, [vp, i32]),
        "prsgd_check_finite": (C.c_int, [vp, C.POINTER(i64), C.POINTER(i32)]),
        "prsgd_partial_sum": (C.c_int, [vp, vp, i64, i64]),
        "prsgd_assign_rows": (C.c_int, [vp, vp, C.c_float, i64, i64]),
        "prsgd_last_error": (C.c_char_p, [vp]),
        "prsgd_average_rows": (C.c_int, [vp, i64, i64, i64, vp]),
        "prsgd_draw_block": (u64, [u64, i32, i64, u64]),
        "prsgd_mean_rows_noalloc": (C.c_int, [vp, i64, i64, i64, vp, C.c_int, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()


class PRSGDError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"prsgd error {code}: {msg}")
        self.code = code


def _check(rc: int, ctx=None) -> None:
    if rc != PRSGD_OK:
        raise PRSGDError(rc, (lib.prsgd_last_error(ctx) or b"").decode())


def make_spec(dims: Sequence[int], batch: int, precision: int, pool_samples: int, seed: int):
    arr = (C.c_int32 * len(dims))(*dims)
    spec = ModelSpec(len(dims) - 1, C.cast(arr, C.POINTER(C.c_int32)), batch, precision, pool_samples, seed)
    spec._keep = arr
    return spec


def prsgd_layout(dims, batch, precision, pool_samples, seed=0) -> Layout:
    spec, lay = make_spec(dims, batch, precision, pool_samples, seed), Layout()
    _check(lib.prsgd_layout(C.byref(spec), C.byref(lay)))
    return lay


def prsgd_workspace_bytes(N, dims, batch, precision, pool_samples, seed=0):
    spec = make_spec(dims, batch, precision, pool_samples, seed)
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib.prsgd_workspace_bytes(N, C.byref(spec), C.byref(a), C.byref(b), C.byref(c)))
    return a.value, b.value, c.value


def prsgd_alg2_schedule(N: int, s: int):
    """(K^s, gamma^s) of Theorem 2."""
    K, g = C.c_int64(), C.c_float()
    _check(lib.prsgd_alg2_schedule(N, s, C.byref(K), C.byref(g)))
    return K.value, g.value


def prsgd_draw_block(seed: int, worker: int, t: int, n_blocks: int) -> int:
    return int(lib.prsgd_draw_block(seed, worker, t, n_blocks))


def prsgd_average_rows(P: torch.Tensor, N: int, m: int, row_stride: Optional[int] = None, stream=None) -> None:
    """In-place node average + broadcast over the rows of a device fp32 tensor."""
    assert P.is_cuda and P.dtype == torch.float32
    s = stream if stream is not None else torch.cuda.current_stream(P.device)
    with torch.cuda.device(P.device):
        _check(lib.prsgd_average_rows(P.data_ptr(), N, m, m if row_stride is None else row_stride, s.cuda_stream))


def prsgd_mean_rows_noalloc(P: torch.Tensor, N: int, m: int, row_stride: int, out, stream=None):
    """Node average of the rows of a device fp32 tensor into `out` (numpy array, or host / device tensor),
    staged through the library's fixed device row: nothing is allocated and P is left untouched."""
    assert P.is_cuda and P.dtype == torch.float32
    s = stream if stream is not None else torch.cuda.current_stream(P.device)
    if isinstance(out, np.ndarray):
        assert out.dtype == np.float32 and out.size >= m and out.flags["C_CONTIGUOUS"]
        ptr, on_dev = out.ctypes.data, 0
    else:
        assert out.dtype == torch.float32 and out.numel() >= m and out.is_contiguous()
        ptr, on_dev = out.data_ptr(), 1 if out.is_cuda else 0
    with torch.cuda.device(P.device):
        _check(lib.prsgd_mean_rows_noalloc(P.data_ptr(), N, m, row_stride, ptr, on_dev, s.cuda_stream))
    return out


def _host_ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


class PRSGD:
    """One PR-SGD context plus the device tensors that back it."""

    def __init__(self, N: int, dims: Sequence[int], batch: int, gamma: float, I: int, precision: int,
                 pool_samples: int, seed: int, device: str = "cuda:0", stream: Optional[torch.cuda.Stream] = None):
        self.N, self.dims, self.B, self.precision, self.P = N, tuple(dims), batch, precision, pool_samples
        self.device = torch.device(device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._spec = make_spec(dims, batch, precision, pool_samples, seed)
        self.layout = Layout()
        _check(lib.prsgd_layout(C.byref(self._spec), C.byref(self.layout)))
        self.m, self.m_pad = self.layout.m, self.layout.m_pad
        pb, sb, wb = prsgd_workspace_bytes(N, dims, batch, precision, pool_samples, seed)
        with torch.cuda.device(self.device):
            self.params = torch.empty(pb // 4, dtype=torch.float32, device=self.device)
            self.shadow = torch.empty(max(sb // 2, 1), dtype=torch.bfloat16, device=self.device) if sb else None
            self.scratch = torch.empty(wb, dtype=torch.uint8, device=self.device)
            ctx = C.c_void_p()
            _check(lib.prsgd_create(N, C.byref(self._spec), gamma, I, self.params.data_ptr(),
                                    self.shadow.data_ptr() if self.shadow is not None else None,
                                    self.scratch.data_ptr(), self.stream.cuda_stream, C.byref(ctx)))
        self.ctx = ctx
        self._X = self._Y = None
        self.average_velocity = False

    def _call(self, fn, *args):
        with torch.cuda.device(self.device):
            _check(fn(self.ctx, *args), self.ctx)

    def close(self):
        if getattr(self, "ctx", None):
            lib.prsgd_destroy(self.ctx)
            self.ctx = None

    __del__ = close

    # ---- data -------------------------------------------------------------------
    def bind_data(self, X: torch.Tensor, Y: torch.Tensor):
        want = torch.bfloat16 if self.precision == PRECISION_BF16 else torch.float32
        assert X.is_cuda and Y.is_cuda and X.dtype == want and Y.dtype == torch.int32
        assert X.is_contiguous() and Y.is_contiguous()
        assert tuple(X.shape) == (self.N, self.P, self.dims[0]) and tuple(Y.shape) == (self.N, self.P)
        self._X, self._Y = X, Y
        self._call(lib.prsgd_bind_data, X.data_ptr(), X_BF16 if want == torch.bfloat16 else X_FP32, Y.data_ptr())

    def upload_data(self, hX: torch.Tensor, hY: torch.Tensor):
        assert not hX.is_cuda and not hY.is_cuda and hX.is_contiguous() and hY.is_contiguous()
        self._call(lib.prsgd_upload_data, hX.data_ptr(), hY.data_ptr())

    def stage_data(self, hX: torch.Tensor, hY: torch.Tensor, copy_stream: torch.cuda.Stream):
        """Copy the next pools from (pinned) host tensors into the spare device pools on `copy_stream`."""
        assert not hX.is_cuda and not hY.is_cuda and hX.is_contiguous() and hY.is_contiguous()
        if getattr(self, "_spare", None) is None:
            self._spare = (torch.empty_like(self._X), torch.empty_like(self._Y))
        self._call(lib.prsgd_stage_data, hX.data_ptr(), hY.data_ptr(), self._spare[0].data_ptr(),
                   self._spare[1].data_ptr(), copy_stream.cuda_stream)

    def swap_data(self):
        """Make the staged pools current; the previous pools become the spare ones."""
        self._call(lib.prsgd_swap_data)
        (self._X, self._Y), self._spare = self._spare, (self._X, self._Y)

    # ---- parameters -------------------------------------------------------------
    def set_params(self, x, worker: int = -1):
        if isinstance(x, torch.Tensor) and x.is_cuda:
            assert x.dtype == torch.float32 and x.numel() == self.m and x.is_contiguous()
            self._call(lib.prsgd_set_params, x.data_ptr(), worker, 1)
        else:
            a = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
            assert a.size == self.m
            self._call(lib.prsgd_set_params, _host_ptr(a), worker, 0)

    def set_params_stacked(self, x):
        if isinstance(x, torch.Tensor) and x.is_cuda:
            assert x.dtype == torch.float32 and x.numel() == self.N * self.m and x.is_contiguous()
            self._call(lib.prsgd_set_params_stacked, x.data_ptr(), 1)
        else:
            a = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
            assert a.size == self.N * self.m
            self._call(lib.prsgd_set_params_stacked, _host_ptr(a), 0)

    def get_params_stacked(self) -> np.ndarray:
        out = np.empty((self.N, self.m), dtype=np.float32)
        self._call(lib.prsgd_get_params_stacked, _host_ptr(out), 0)
        return out

    def get_params(self, worker: int) -> np.ndarray:
        out = np.empty(self.m, dtype=np.float32)
        self._call(lib.prsgd_get_params, _host_ptr(out), worker, 0)
        return out

    # ---- Algorithm 1 ------------------------------------------------------------
    def local_steps(self, k: int):
        self._call(lib.prsgd_local_steps, k)

    def local_steps_sum(self, k: int):
        """k iterations, the last one leaving the SUM of the updated local rows in every row (see prsgd.h)."""
        self._call(lib.prsgd_local_steps_sum, k)

    def row0(self) -> torch.Tensor:
        """Row 0 of the store as a tensor of m_pad floats (the all-reduce buffer after local_steps_sum)."""
        return self.params[:self.m_pad]

    def average(self):
        self._call(lib.prsgd_average)

    def get_average(self, out=None):
        """Node average; into a host numpy array (default), a pinned host tensor or a device tensor."""
        if out is None:
            out = np.empty(self.m, dtype=np.float32)
        if isinstance(out, np.ndarray):
            self._call(lib.prsgd_get_average, _host_ptr(out), 0)
        else:
            assert out.dtype == torch.float32 and out.numel() == self.m and out.is_contiguous()
            self._call(lib.prsgd_get_average, out.data_ptr(), 1 if out.is_cuda else 0)
        return out

    def get_average_async(self, out, copy_stream):
        """Node average into a pinned host tensor through `copy_stream`; valid once that stream is synchronised."""
        assert out.dtype == torch.float32 and out.numel() == self.m and out.is_contiguous() and out.is_pinned()
        self._call(lib.prsgd_get_average_async, out.data_ptr(), copy_stream.cuda_stream)
        return out

    def get_losses(self) -> np.ndarray:
        out = np.empty(self.N, dtype=np.float32)
        self._call(lib.prsgd_get_losses, _host_ptr(out))
        return out

    def get_draws(self) -> np.ndarray:
        out = np.empty(self.N, dtype=np.int32)
        self._call(lib.prsgd_get_draws, _host_ptr(out))
        return out

    # ---- shard of a multi-GPU job ------------------------------------------------
    def set_worker_offset(self, first_worker: int):
        self._call(lib.prsgd_set_worker_offset, first_worker)

    def set_global_workers(self, N_global: int):
        self._call(lib.prsgd_set_global_workers, N_global)

    def new_row(self) -> torch.Tensor:
        """A device row of m_pad floats (the buffer an all-reduce works on)."""
        return torch.zeros(self.m_pad, dtype=torch.float32, device=self.device)

    def partial_sum(self, row: torch.Tensor, col0: int = 0, ncols: Optional[int] = None):
        assert row.is_cuda and row.dtype == torch.float32 and row.numel() == self.m_pad
        self._call(lib.prsgd_partial_sum, row.data_ptr(), col0, self.m_pad - col0 if ncols is None else ncols)

    def assign_rows(self, row: torch.Tensor, divisor: float, col0: int = 0, ncols: Optional[int] = None):
        assert row.is_cuda and row.dtype == torch.float32 and row.numel() == self.m_pad
        self._call(lib.prsgd_assign_rows, row.data_ptr(), float(divisor), col0, self.m_pad - col0 if ncols is None else ncols)

    def enable_momentum(self, mu: float, average_velocity: bool = False):
        """Allocate the momentum buffers (same size as the store) and switch the local step to SGD with momentum."""
        with torch.cuda.device(self.device):
            self.velocity = torch.empty(self.N * self.m_pad, dtype=torch.float32, device=self.device)
        self._call(lib.prsgd_enable_momentum, mu, self.velocity.data_ptr(), 1 if average_velocity else 0)
        self.average_velocity = bool(average_velocity)

    def get_velocity_stacked(self) -> np.ndarray:
        out = np.empty((self.N, self.m), dtype=np.float32)
        self._call(lib.prsgd_get_velocity_stacked, _host_ptr(out), 0)
        return out

    # ---- Algorithms 2 and 3 ------------------------------------------------------
    def run_time_varying(self, s_begin: int, s_end: int, gamma_scale: float = 1.0):
        self._call(lib.prsgd_run_time_varying, s_begin, s_end, gamma_scale)

    def run_heterogeneous_epoch(self, I_i: Sequence[int]):
        a = np.ascontiguousarray(np.asarray(I_i, dtype=np.int32))
        assert a.size == self.N
        self._call(lib.prsgd_run_heterogeneous_epoch, _host_ptr(a))

    # ---- schedule ---------------------------------------------------------------
    def set_lr(self, gamma: float):
        self._call(lib.prsgd_set_lr, gamma)

    def set_interval(self, I: int):
        self._call(lib.prsgd_set_interval, I)

    def set_active(self, mask):
        if mask is None:
            self._call(lib.prsgd_set_active, None)
        else:
            a = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
            assert a.size == self.N
            self._call(lib.prsgd_set_active, _host_ptr(a))

    def get_step(self) -> int:
        t = C.c_int64()
        self._call(lib.prsgd_get_step, C.byref(t))
        return t.value

    def set_step(self, t: int):
        self._call(lib.prsgd_set_step, t)

    def set_option(self, option: int, value: int):
        self._call(lib.prsgd_set_option, option, value)

    def get_launch_count(self) -> int:
        n = C.c_int64()
        self._call(lib.prsgd_get_launch_count, C.byref(n))
        return n.value

    def get_profile(self) -> dict:
        """{family: (ms_total, launches)} since the last call; needs OPT_PROFILE."""
        out = {}
        for k, name in enumerate(KERNEL_FAMILIES):
            ms, n = C.c_double(), C.c_int64()
            self._call(lib.prsgd_get_profile, k, C.byref(ms), C.byref(n))
            out[name] = (ms.value, n.value)
        return out

    def selftest_wait_expiry(self, limit_us: int = 1000):
        self._call(lib.prsgd_selftest_wait_expiry, limit_us)

    def clear_device_error(self):
        self._call(lib.prsgd_clear_device_error)

    def sync(self):
        self._call(lib.prsgd_sync)

    def check_finite(self):
        """(return code, count of non-finite words, lowest worker that holds one or -1); does not raise."""
        n, first = C.c_int64(), C.c_int32()
        with torch.cuda.device(self.device):
            rc = lib.prsgd_check_finite(self.ctx, C.byref(n), C.byref(first))
        return rc, n.value, first.value
