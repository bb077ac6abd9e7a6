"""ctypes binding of libmlora.so: the same names as the C ABI (include/mlora.h), plus thin
object wrappers that only marshal arguments (torch tensors -> device pointers, leading
dimensions, the current CUDA stream).  Every step of the layer runs inside the library's
kernels; nothing here computes, and there is no fallback: if the library cannot be loaded, or
no sm_100 device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libmlora.so")

MLORA_F32, MLORA_BF16 = 0, 1
(MLORA_OK, MLORA_ERR_INVALID_ARG, MLORA_ERR_SEGMENT_RANGE, MLORA_ERR_SEGMENT_OVERLAP, MLORA_ERR_ADAPTER_ID,
 MLORA_ERR_SAVE_CAPACITY, MLORA_ERR_UNSUPPORTED, MLORA_ERR_ARCH, MLORA_ERR_CUDA, MLORA_ERR_DEVICE_TIMEOUT,
 MLORA_CANCELLED) = range(11)

EXPORTS = (
    "mlora_create", "mlora_destroy", "mlora_plan_create", "mlora_plan_destroy", "mlora_plan_rows",
    "mlora_plan_ft_rows", "mlora_plan_ft_adapters", "mlora_plan_describe", "mlora_mixed_forward",
    "mlora_backward", "mlora_poll_status", "mlora_status_string", "mlora_launch_count", "mlora_set_gemm_path",
    "mlora_plan_create_ranked", "mlora_plan_create_ranked_async", "mlora_plan_lowrank_columns", "mlora_profile_enable", "mlora_profile_collect", "mlora_forward_noalloc", "mlora_adamw_update",
    "mlora_set_cancel_flag", "mlora_set_dropout", "mlora_plan_create_async", "mlora_plan_release",
    "mlora_selftest_timeout",
)
MLORA_NOALLOC_MAX_ROWS = 512


class mlora_segment_t(ctypes.Structure):
    _fields_ = [("row_start", ctypes.c_int32), ("row_len", ctypes.c_int32),
                ("adapter_id", ctypes.c_int32), ("is_finetune", ctypes.c_int32)]


class mlora_layer_t(ctypes.Structure):
    _fields_ = [("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32), ("rank", ctypes.c_int32),
                ("n_adapters", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("W", ctypes.c_void_p), ("ldw", ctypes.c_int64),
                ("A_all", ctypes.c_void_p), ("B_all", ctypes.c_void_p), ("scale", ctypes.c_void_p)]


class mlora_adamw_t(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("weight_decay", ctypes.c_float), ("step", ctypes.c_int32)]


class MloraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def load_library(build_if_missing: bool = True) -> ctypes.CDLL:
    """Load libmlora.so (building it with nvcc first when it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        from . import build as _build
        if _build.is_stale():
            _build.build()
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_28848_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    P = ctypes.POINTER
    lib.mlora_create.argtypes = [P(vp), ctypes.c_int]
    lib.mlora_create.restype = ctypes.c_int
    lib.mlora_destroy.argtypes = [vp]
    lib.mlora_destroy.restype = None
    lib.mlora_plan_create.argtypes = [vp, P(mlora_segment_t), i32, i32, i32, P(vp)]
    lib.mlora_plan_create.restype = ctypes.c_int
    lib.mlora_plan_create_ranked.argtypes = [vp, P(mlora_segment_t), i32, i32, i32, P(i32), P(vp)]
    lib.mlora_plan_create_ranked.restype = ctypes.c_int
    lib.mlora_plan_create_ranked_async.argtypes = [vp, P(mlora_segment_t), i32, i32, i32, P(i32), vp, P(vp)]
    lib.mlora_plan_create_ranked_async.restype = ctypes.c_int
    lib.mlora_plan_lowrank_columns.argtypes = [vp, i32, P(i32), i32]
    lib.mlora_plan_lowrank_columns.restype = i32
    lib.mlora_plan_destroy.argtypes = [vp]
    lib.mlora_plan_destroy.restype = None
    lib.mlora_plan_create_async.argtypes = [vp, P(mlora_segment_t), i32, i32, i32, vp, P(vp)]
    lib.mlora_plan_create_async.restype = ctypes.c_int
    lib.mlora_plan_release.argtypes = [vp, vp]
    lib.mlora_plan_release.restype = ctypes.c_int
    lib.mlora_plan_rows.argtypes = [vp]
    lib.mlora_plan_rows.restype = i32
    lib.mlora_plan_ft_rows.argtypes = [vp]
    lib.mlora_plan_ft_rows.restype = i32
    lib.mlora_plan_ft_adapters.argtypes = [vp, P(i32), i32]
    lib.mlora_plan_ft_adapters.restype = i32
    lib.mlora_plan_describe.argtypes = [vp, P(i32), P(i32)]
    lib.mlora_plan_describe.restype = ctypes.c_int
    lib.mlora_mixed_forward.argtypes = [vp, P(mlora_layer_t), vp, vp, i64, vp, i64, vp, vp, i64, i64, vp]
    lib.mlora_mixed_forward.restype = ctypes.c_int
    lib.mlora_backward.argtypes = [vp, P(mlora_layer_t), vp, vp, i64, vp, vp, vp, vp, vp, i64, i32, vp]
    lib.mlora_backward.restype = ctypes.c_int
    lib.mlora_poll_status.argtypes = [vp, vp]
    lib.mlora_poll_status.restype = ctypes.c_int
    lib.mlora_status_string.argtypes = [ctypes.c_int]
    lib.mlora_status_string.restype = ctypes.c_char_p
    lib.mlora_launch_count.argtypes = [vp]
    lib.mlora_launch_count.restype = i64
    lib.mlora_set_gemm_path.argtypes = [vp, i32]
    lib.mlora_set_gemm_path.restype = ctypes.c_int
    lib.mlora_profile_enable.argtypes = [vp, i32]
    lib.mlora_profile_enable.restype = ctypes.c_int
    lib.mlora_profile_collect.argtypes = [vp, P(i32), P(ctypes.c_float), i32]
    lib.mlora_profile_collect.restype = i32
    lib.mlora_adamw_update.argtypes = [vp, P(mlora_layer_t), vp, vp, vp, vp, vp, vp, vp, vp, vp, P(mlora_adamw_t), vp]
    lib.mlora_adamw_update.restype = ctypes.c_int
    lib.mlora_set_cancel_flag.argtypes = [vp, P(i32)]
    lib.mlora_set_cancel_flag.restype = ctypes.c_int
    lib.mlora_set_dropout.argtypes = [vp, ctypes.c_double, ctypes.c_uint64]
    lib.mlora_set_dropout.restype = ctypes.c_int
    lib.mlora_selftest_timeout.argtypes = [vp, ctypes.c_uint32, vp]
    lib.mlora_selftest_timeout.restype = ctypes.c_int
    lib.mlora_forward_noalloc.argtypes = [P(mlora_layer_t), vp, i32, vp, i64, vp, i64, vp]
    lib.mlora_forward_noalloc.restype = ctypes.c_int
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().mlora_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != MLORA_OK:
        raise MloraError(status, where)


def _segments_ctypes(segments):
    """A [n, 4] int32 array has the memory layout of mlora_segment_t[n]: pass it as it is."""
    seg = np.ascontiguousarray(np.asarray(segments, dtype=np.int32).reshape(-1, 4))
    if len(seg) == 0:
        return (mlora_segment_t * 1)(), 0
    return (mlora_segment_t * len(seg)).from_buffer_copy(seg.tobytes()), len(seg)


# --------------------------------------------------------------------------------------------
# same-name functions (raise MloraError on a non-zero status)
# --------------------------------------------------------------------------------------------
def mlora_create(device: int = 0) -> ctypes.c_void_p:
    h = ctypes.c_void_p()
    _check(load_library().mlora_create(ctypes.byref(h), int(device)), "mlora_create")
    return h


def mlora_destroy(ctx) -> None:
    load_library().mlora_destroy(ctx)


def mlora_plan_create(ctx, segments, n_rows: int, n_adapters: int) -> ctypes.c_void_p:
    arr, n = _segments_ctypes(segments)
    h = ctypes.c_void_p()
    _check(load_library().mlora_plan_create(ctx, arr, n, int(n_rows), int(n_adapters), ctypes.byref(h)),
           "mlora_plan_create")
    return h


def mlora_plan_create_ranked(ctx, segments, n_rows: int, n_adapters: int, adapter_rank) -> ctypes.c_void_p:
    """A plan for adapters with ranks of their own: ``adapter_rank`` holds one rank per adapter (host integers)."""
    arr, n = _segments_ctypes(segments)
    ranks = (ctypes.c_int32 * int(n_adapters))(*[int(r) for r in adapter_rank])
    h = ctypes.c_void_p()
    _check(load_library().mlora_plan_create_ranked(ctx, arr, n, int(n_rows), int(n_adapters), ranks, ctypes.byref(h)),
           "mlora_plan_create_ranked")
    return h


def mlora_plan_destroy(plan) -> None:
    load_library().mlora_plan_destroy(plan)


def mlora_plan_create_async(ctx, segments, n_rows: int, n_adapters: int, stream=None) -> ctypes.c_void_p:
    """Stream-ordered plan from the context's buffer pool (tables uploaded on the current or given stream)."""
    arr, n = _segments_ctypes(segments)
    h = ctypes.c_void_p()
    _check(load_library().mlora_plan_create_async(ctx, arr, n, int(n_rows), int(n_adapters), _stream_ptr(stream),
                                                  ctypes.byref(h)), "mlora_plan_create_async")
    return h


def mlora_plan_create_ranked_async(ctx, segments, n_rows: int, n_adapters: int, adapter_rank, stream=None) -> ctypes.c_void_p:
    """Stream-ordered plan for adapters with ranks of their own."""
    arr, n = _segments_ctypes(segments)
    ranks = (ctypes.c_int32 * int(n_adapters))(*[int(r) for r in adapter_rank])
    h = ctypes.c_void_p()
    _check(load_library().mlora_plan_create_ranked_async(ctx, arr, n, int(n_rows), int(n_adapters), ranks, _stream_ptr(stream),
                                                         ctypes.byref(h)), "mlora_plan_create_ranked_async")
    return h


def mlora_plan_lowrank_columns(plan, rank: int) -> List[int]:
    """Columns of the low-rank operand of every 256-row tile (the extra contraction depth of the fused expand)."""
    lib = load_library()
    n = int(lib.mlora_plan_lowrank_columns(plan, int(rank), None, 0))
    buf = (ctypes.c_int32 * max(n, 1))()
    lib.mlora_plan_lowrank_columns(plan, int(rank), buf, n)
    return [int(buf[i]) for i in range(n)]


def mlora_plan_release(plan, stream=None) -> None:
    _check(load_library().mlora_plan_release(plan, _stream_ptr(stream)), "mlora_plan_release")


def mlora_plan_rows(plan) -> int:
    return int(load_library().mlora_plan_rows(plan))


def mlora_plan_ft_rows(plan) -> int:
    return int(load_library().mlora_plan_ft_rows(plan))


def mlora_plan_ft_adapters(plan) -> List[int]:
    lib = load_library()
    n = lib.mlora_plan_ft_adapters(plan, None, 0)
    buf = (ctypes.c_int32 * max(n, 1))()
    lib.mlora_plan_ft_adapters(plan, buf, n)
    return [int(buf[i]) for i in range(n)]


def mlora_plan_describe(plan, n_segs: int):
    lib = load_library()
    n_rows = lib.mlora_plan_rows(plan)
    so = (ctypes.c_int32 * max(n_segs, 1))()
    ra = (ctypes.c_int32 * max(n_rows, 1))()
    _check(lib.mlora_plan_describe(plan, so, ra), "mlora_plan_describe")
    return np.asarray(so[:n_segs], dtype=np.int32), np.asarray(ra[:n_rows], dtype=np.int32)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


_raw_stream = None      # torch's accessor for the current stream's handle (None: not looked up yet, False: absent)


def _stream_ptr(stream=None) -> int:
    """Handle of the given torch stream, or of the current stream of the current device."""
    global _raw_stream
    import torch
    if stream is not None:
        return int(stream.cuda_stream)
    if _raw_stream is None:
        _raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", False)
    if _raw_stream:         # the handle straight from the runtime: the Stream object costs ten times the call
        return int(_raw_stream(torch.cuda.current_device()))
    return int(torch.cuda.current_stream().cuda_stream)


def make_layer(W, A_all, B_all, scale) -> mlora_layer_t:
    """Describe a projection from torch CUDA tensors (W [d_in,d_out], A_all [n,r,d_in], B_all [n,r,d_out])."""
    import torch
    assert W.is_cuda and A_all.is_cuda and B_all.is_cuda and scale.is_cuda
    assert A_all.is_contiguous() and B_all.is_contiguous() and scale.dtype == torch.float32
    assert W.dtype == A_all.dtype == B_all.dtype and W.stride(1) == 1
    dt = {torch.float32: MLORA_F32, torch.bfloat16: MLORA_BF16}[W.dtype]
    n, r, d_in = A_all.shape
    d_out = B_all.shape[2]
    assert W.shape == (d_in, d_out) and B_all.shape[:2] == (n, r) and scale.numel() == n
    return mlora_layer_t(d_in, d_out, r, n, dt, _ptr(W), W.stride(0), _ptr(A_all), _ptr(B_all), _ptr(scale))


def mlora_mixed_forward(ctx, layer: mlora_layer_t, plan, X, Y, x_save, u_save, save_row_base: int = 0,
                        save_capacity_rows: Optional[int] = None, stream=None) -> None:
    """Queue the forward on the current (or given) stream.  X, Y, x_save, u_save are torch CUDA tensors."""
    if save_capacity_rows is None:
        save_capacity_rows = 0 if u_save is None else int(u_save.shape[0])
    st = load_library().mlora_mixed_forward(
        ctx, ctypes.byref(layer), plan, _ptr(X), X.stride(0) if X is not None else 0,
        _ptr(Y), Y.stride(0) if Y is not None else 0, _ptr(x_save), _ptr(u_save),
        int(save_row_base), int(save_capacity_rows), _stream_ptr(stream))
    _check(st, "mlora_mixed_forward")


def mlora_backward(ctx, layer: mlora_layer_t, plan, dY, x_save, u_save, dA, dB, dX, accumulate: bool = False,
                   stream=None) -> None:
    """Queue the LoRA backward; all row-indexed tensors start at the first row this plan saved."""
    st = load_library().mlora_backward(
        ctx, ctypes.byref(layer), plan, _ptr(dY), dY.stride(0) if dY is not None else 0, _ptr(x_save), _ptr(u_save),
        _ptr(dA), _ptr(dB), _ptr(dX), dX.stride(0) if dX is not None else 0, int(bool(accumulate)),
        _stream_ptr(stream))
    _check(st, "mlora_backward")


def mlora_poll_status(ctx, stream=None) -> int:
    return int(load_library().mlora_poll_status(ctx, _stream_ptr(stream)))


def mlora_selftest_timeout(ctx, polls: int = 1024, stream=None) -> None:
    """Queue the kernel whose bounded wait runs out on purpose (the next poll reports the timeout)."""
    _check(load_library().mlora_selftest_timeout(ctx, int(polls), _stream_ptr(stream)), "mlora_selftest_timeout")


def mlora_launch_count(ctx) -> int:
    return int(load_library().mlora_launch_count(ctx))


def mlora_set_gemm_path(ctx, path: int) -> None:
    _check(load_library().mlora_set_gemm_path(ctx, int(path)), "mlora_set_gemm_path")


PROFILE_KINDS = ("shrink", "gemm_fwd", "gemm_bwd", "grad", "simt", "adamw", "splitk_reduce")


def mlora_adamw_update(ctx, layer: mlora_layer_t, plan, dA, dB, wA, wB, mA, vA, mB, vB, step: int, lr: float = 1e-3,
                       beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.01,
                       stream=None) -> None:
    """Queue one AdamW update of the plan's fine-tuning adapters (all tensors fp32 CUDA, slot-indexed)."""
    hp = mlora_adamw_t(lr, beta1, beta2, eps, weight_decay, int(step))
    st = load_library().mlora_adamw_update(ctx, ctypes.byref(layer), plan, _ptr(dA), _ptr(dB), _ptr(wA), _ptr(wB),
                                           _ptr(mA), _ptr(vA), _ptr(mB), _ptr(vB), ctypes.byref(hp),
                                           _stream_ptr(stream))
    _check(st, "mlora_adamw_update")


def mlora_profile_enable(ctx, max_records: int) -> None:
    _check(load_library().mlora_profile_enable(ctx, int(max_records)), "mlora_profile_enable")


def mlora_profile_collect(ctx, cap: int = 1 << 16):
    """Returns (kinds, ms) numpy arrays of the launches recorded since the last collect."""
    kinds = (ctypes.c_int32 * cap)()
    ms = (ctypes.c_float * cap)()
    n = load_library().mlora_profile_collect(ctx, kinds, ms, cap)
    n = min(n, cap)
    return np.asarray(kinds[:n], dtype=np.int32), np.asarray(ms[:n], dtype=np.float64)


def mlora_forward_noalloc(layer: mlora_layer_t, row_adapter, X, Y, stream=None) -> None:
    """Forward for a small batch of inference rows that allocates nothing: no context, no plan.

    For callers that must not allocate device memory (an engine that owns the whole memory pool,
    a worker attached to someone else's buffers).  ``row_adapter`` is an int32 CUDA tensor with one
    adapter id (or -1) per row; at most MLORA_NOALLOC_MAX_ROWS rows.  The rank-r intermediate goes
    through a scratch array built into the library and shared by every call on the device, so
    calls must not overlap on the GPU.  Make the first call on a device outside stream capture.
    """
    n_rows = int(row_adapter.numel())
    st = load_library().mlora_forward_noalloc(ctypes.byref(layer), _ptr(row_adapter), n_rows, _ptr(X),
                                              X.stride(0), _ptr(Y), Y.stride(0), _stream_ptr(stream))
    _check(st, "mlora_forward_noalloc")


def mlora_set_cancel_flag(ctx, flag) -> None:
    """Register a host flag (a ctypes.c_int32 the caller keeps alive, or None) checked before every launch."""
    ptr = None if flag is None else ctypes.pointer(flag)
    _check(load_library().mlora_set_cancel_flag(ctx, ptr), "mlora_set_cancel_flag")


def mlora_set_dropout(ctx, p: float, seed: int) -> None:
    """LoRA dropout of the fine-tuning rows' branch input for the calls that follow (p = 0: off)."""
    _check(load_library().mlora_set_dropout(ctx, float(p), int(seed) & 0xFFFFFFFFFFFFFFFF), "mlora_set_dropout")
