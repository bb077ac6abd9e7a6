"""ctypes binding of include/mlora_layer_ops.h (argument marshalling only, same names)."""
from __future__ import annotations

import ctypes

from . import binding as _b

EXPORTS = ("mlora_rmsnorm_forward", "mlora_rmsnorm_backward", "mlora_rope", "mlora_swiglu_forward",
           "mlora_swiglu_backward", "mlora_add", "mlora_attention_forward", "mlora_attention_backward",
           "mlora_layer_ops_poll_status")
_ready = False


def _lib():
    global _ready
    lib = _b.load_library()
    if _ready:
        return lib
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.mlora_rmsnorm_forward.argtypes = [vp, i64, vp, vp, i64, i32, i32, f32, vp]
    lib.mlora_rmsnorm_backward.argtypes = [vp, i64, vp, vp, i64, vp, i64, i32, i32, f32, vp]
    lib.mlora_rope.argtypes = [vp, i64, vp, i64, vp, i32, i32, i32, f32, i32, vp]
    lib.mlora_swiglu_forward.argtypes = [vp, vp, vp, i64, vp]
    lib.mlora_swiglu_backward.argtypes = [vp, vp, vp, vp, vp, i64, vp]
    lib.mlora_add.argtypes = [vp, vp, vp, i64, vp]
    lib.mlora_attention_forward.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.mlora_attention_backward.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, vp, i64, vp, i64, vp, i64, vp, i64,
                                             vp, vp, i32, i32, i32, i32, vp]
    lib.mlora_layer_ops_poll_status.argtypes = [vp]
    for name in EXPORTS:
        getattr(lib, name).restype = ctypes.c_int
    _ready = True
    return lib


def _p(t):
    return ctypes.c_void_p(t.data_ptr())


def mlora_rmsnorm_forward(x, gain, y, eps: float = 1e-5, stream=None) -> None:
    _b._check(_lib().mlora_rmsnorm_forward(_p(x), x.stride(0), _p(gain), _p(y), y.stride(0), x.shape[0], x.shape[1],
                                           float(eps), _b._stream_ptr(stream)), "mlora_rmsnorm_forward")


def mlora_rmsnorm_backward(x, gain, dy, dx, eps: float = 1e-5, stream=None) -> None:
    _b._check(_lib().mlora_rmsnorm_backward(_p(x), x.stride(0), _p(gain), _p(dy), dy.stride(0), _p(dx), dx.stride(0),
                                            x.shape[0], x.shape[1], float(eps), _b._stream_ptr(stream)),
              "mlora_rmsnorm_backward")


def mlora_rope(x, y, pos, n_heads: int, d_head: int, theta: float = 500000.0, transpose: bool = False, stream=None) -> None:
    """x, y [T, n_heads * d_head] bf16 (y may be x); pos int32 [T]."""
    _b._check(_lib().mlora_rope(_p(x), x.stride(0), _p(y), y.stride(0), _p(pos), x.shape[0], int(n_heads), int(d_head),
                                float(theta), int(bool(transpose)), _b._stream_ptr(stream)), "mlora_rope")


def mlora_swiglu_forward(g, u, m, stream=None) -> None:
    _b._check(_lib().mlora_swiglu_forward(_p(g), _p(u), _p(m), g.numel(), _b._stream_ptr(stream)), "mlora_swiglu_forward")


def mlora_swiglu_backward(g, u, dm, dg, du, stream=None) -> None:
    _b._check(_lib().mlora_swiglu_backward(_p(g), _p(u), _p(dm), _p(dg), _p(du), g.numel(), _b._stream_ptr(stream)),
              "mlora_swiglu_backward")


def mlora_add(a, b, out, stream=None) -> None:
    _b._check(_lib().mlora_add(_p(a), _p(b), _p(out), a.numel(), _b._stream_ptr(stream)), "mlora_add")


def mlora_attention_forward(q, k, v, o, lse, seq_start, seq_end, n_heads: int, n_kv: int, d_head: int, stream=None) -> None:
    """q, o [T, n_heads * d_head], k, v [T, n_kv * d_head] bf16; lse fp32 [T, n_heads]; seq_start / seq_end int32 [T]."""
    _b._check(_lib().mlora_attention_forward(_p(q), q.stride(0), _p(k), k.stride(0), _p(v), v.stride(0), _p(o), o.stride(0),
                                             _p(lse), _p(seq_start), _p(seq_end), q.shape[0], int(n_heads), int(n_kv),
                                             int(d_head), _b._stream_ptr(stream)), "mlora_attention_forward")


def mlora_attention_backward(q, k, v, o, lse, dO, dq, dk, dv, seq_start, seq_end, n_heads: int, n_kv: int, d_head: int,
                             stream=None) -> None:
    _b._check(_lib().mlora_attention_backward(_p(q), q.stride(0), _p(k), k.stride(0), _p(v), v.stride(0), _p(o), o.stride(0),
                                              _p(lse), _p(dO), dO.stride(0), _p(dq), dq.stride(0), _p(dk), dk.stride(0),
                                              _p(dv), dv.stride(0), _p(seq_start), _p(seq_end), q.shape[0], int(n_heads),
                                              int(n_kv), int(d_head), _b._stream_ptr(stream)), "mlora_attention_backward")


def mlora_layer_ops_poll_status(stream=None) -> int:
    """Synchronises the stream; returns and clears the status word of the layer pieces' bounded waits."""
    return int(_lib().mlora_layer_ops_poll_status(_b._stream_ptr(stream)))
