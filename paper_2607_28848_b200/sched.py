"""ctypes binding of the host-side scheduler entry points (include/mlora_sched.h): argument
marshalling only, same names as the C functions.  All arithmetic runs in the C library."""
from __future__ import annotations

import ctypes
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import binding as _b

EXPORTS = (
    "mlora_predict_mixed", "mlora_predict_decode", "mlora_ttft_budget", "mlora_fit_mixed",
    "mlora_sched_create", "mlora_sched_destroy", "mlora_sched_set_coef", "mlora_sched_pool_add",
    "mlora_sched_pool_size", "mlora_sched_buffer_left", "mlora_sched_set_backward_running",
    "mlora_sched_admit", "mlora_sched_requeue", "mlora_sched_buffer_release", "mlora_sched_observe",
    "mlora_sched_observations", "mlora_sched_refit",
)
MODE_EAGER, MODE_GRAPH = 0, 1
FIT_ALPHA, FIT_BETA, FIT_GAMMA, FIT_EPS, FIT_C = 1, 2, 4, 8, 16


class mlora_mixed_coef_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("alpha", "beta", "gamma", "eps", "c")]


class mlora_decode_coef_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("beta", "eps", "c")]


class mlora_observation_t(ctypes.Structure):
    _fields_ = [("prefill_lens", ctypes.POINTER(ctypes.c_int32)), ("n_prefill", ctypes.c_int32),
                ("n_decode", ctypes.c_int32), ("kv_tokens", ctypes.c_int64), ("ft_tokens", ctypes.c_int64),
                ("seconds", ctypes.c_double)]


class mlora_sched_config_t(ctypes.Structure):
    _fields_ = [("graph", mlora_mixed_coef_t), ("eager", mlora_mixed_coef_t), ("decode", mlora_decode_coef_t),
                ("t_slo_ttft", ctypes.c_double), ("t_tpot", ctypes.c_double), ("buffer_tokens", ctypes.c_int64),
                ("mixed_batch_host", ctypes.c_int32), ("host_uses_graph", ctypes.c_int32)]


class mlora_step_t(ctypes.Structure):
    _fields_ = [("prefill_lens", ctypes.POINTER(ctypes.c_int32)), ("n_prefill", ctypes.c_int32),
                ("n_decode", ctypes.c_int32), ("kv_tokens", ctypes.c_int64), ("t_now", ctypes.c_double),
                ("earliest_arrival", ctypes.c_double), ("wait_n_decode", ctypes.c_int32),
                ("wait_kv_tokens", ctypes.c_int64)]


_ready = False


def _lib() -> ctypes.CDLL:
    global _ready
    lib = _b.load_library()
    if _ready:
        return lib
    P, vp, i32, i64, dbl = ctypes.POINTER, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
    lib.mlora_predict_mixed.argtypes = [P(mlora_mixed_coef_t), P(i32), i32, i32, i64, i64]
    lib.mlora_predict_mixed.restype = dbl
    lib.mlora_predict_decode.argtypes = [P(mlora_decode_coef_t), i32, i64]
    lib.mlora_predict_decode.restype = dbl
    lib.mlora_ttft_budget.argtypes = [dbl, dbl, dbl]
    lib.mlora_ttft_budget.restype = dbl
    lib.mlora_fit_mixed.argtypes = [P(mlora_observation_t), i32, ctypes.c_uint32, P(mlora_mixed_coef_t)]
    lib.mlora_fit_mixed.restype = ctypes.c_int
    lib.mlora_sched_create.argtypes = [P(mlora_sched_config_t), P(vp)]
    lib.mlora_sched_create.restype = ctypes.c_int
    lib.mlora_sched_destroy.argtypes = [vp]
    lib.mlora_sched_destroy.restype = None
    lib.mlora_sched_set_coef.argtypes = [vp, P(mlora_mixed_coef_t), P(mlora_mixed_coef_t), P(mlora_decode_coef_t)]
    lib.mlora_sched_set_coef.restype = ctypes.c_int
    lib.mlora_sched_pool_add.argtypes = [vp, i64, i32]
    lib.mlora_sched_pool_add.restype = ctypes.c_int
    lib.mlora_sched_pool_size.argtypes = [vp]
    lib.mlora_sched_pool_size.restype = i32
    lib.mlora_sched_buffer_left.argtypes = [vp]
    lib.mlora_sched_buffer_left.restype = i64
    lib.mlora_sched_set_backward_running.argtypes = [vp, i32]
    lib.mlora_sched_set_backward_running.restype = ctypes.c_int
    lib.mlora_sched_admit.argtypes = [vp, P(mlora_step_t), P(i64), P(i32), i32, P(i32), P(dbl)]
    lib.mlora_sched_admit.restype = ctypes.c_int
    lib.mlora_sched_requeue.argtypes = [vp, P(i64), P(i32), i32]
    lib.mlora_sched_requeue.restype = ctypes.c_int
    lib.mlora_sched_buffer_release.argtypes = [vp, i64]
    lib.mlora_sched_buffer_release.restype = ctypes.c_int
    lib.mlora_sched_observe.argtypes = [vp, i32, P(mlora_observation_t)]
    lib.mlora_sched_observe.restype = ctypes.c_int
    lib.mlora_sched_observations.argtypes = [vp, i32]
    lib.mlora_sched_observations.restype = i32
    lib.mlora_sched_refit.argtypes = [vp, i32, ctypes.c_uint32, P(mlora_mixed_coef_t)]
    lib.mlora_sched_refit.restype = ctypes.c_int
    _ready = True
    return lib


def _i32_array(values: Sequence[int]):
    arr = (ctypes.c_int32 * max(len(values), 1))(*[int(v) for v in values])
    return arr


def mixed_coef(alpha=0.0, beta=0.0, gamma=0.0, eps=0.0, c=0.0) -> mlora_mixed_coef_t:
    return mlora_mixed_coef_t(alpha, beta, gamma, eps, c)


def decode_coef(beta=0.0, eps=0.0, c=0.0) -> mlora_decode_coef_t:
    return mlora_decode_coef_t(beta, eps, c)


def mlora_predict_mixed(coef: mlora_mixed_coef_t, prefill_lens: Sequence[int], n_decode: int, kv_tokens: int,
                        ft_tokens: int) -> float:
    arr = _i32_array(prefill_lens)
    return _lib().mlora_predict_mixed(ctypes.byref(coef), arr, len(prefill_lens), int(n_decode), int(kv_tokens),
                                      int(ft_tokens))


def mlora_predict_decode(coef: mlora_decode_coef_t, n_decode: int, kv_tokens: int) -> float:
    return _lib().mlora_predict_decode(ctypes.byref(coef), int(n_decode), int(kv_tokens))


def mlora_ttft_budget(t_slo: float, t_now: float, t_arrival: float) -> float:
    return _lib().mlora_ttft_budget(float(t_slo), float(t_now), float(t_arrival))


def mlora_fit_mixed(observations, fit_mask: int = 31) -> mlora_mixed_coef_t:
    """observations: iterable of (prefill_lens, n_decode, kv_tokens, ft_tokens, seconds)."""
    observations = list(observations)
    keep = []
    obs = (mlora_observation_t * max(len(observations), 1))()
    for i, (lens, bd, kv, tft, t) in enumerate(observations):
        arr = _i32_array(lens)
        keep.append(arr)
        obs[i] = mlora_observation_t(arr, len(lens), int(bd), int(kv), int(tft), float(t))
    out = mlora_mixed_coef_t()
    _b._check(_lib().mlora_fit_mixed(obs, len(observations), int(fit_mask), ctypes.byref(out)), "mlora_fit_mixed")
    return out


def mlora_sched_create(graph: mlora_mixed_coef_t, eager: mlora_mixed_coef_t, decode: mlora_decode_coef_t,
                       t_slo_ttft: float, t_tpot: float, buffer_tokens: int, mixed_batch_host: bool = True,
                       host_uses_graph: bool = False) -> ctypes.c_void_p:
    cfg = mlora_sched_config_t(graph, eager, decode, float(t_slo_ttft), float(t_tpot), int(buffer_tokens),
                               int(bool(mixed_batch_host)), int(bool(host_uses_graph)))
    h = ctypes.c_void_p()
    _b._check(_lib().mlora_sched_create(ctypes.byref(cfg), ctypes.byref(h)), "mlora_sched_create")
    return h


def mlora_sched_destroy(s) -> None:
    _lib().mlora_sched_destroy(s)


def mlora_sched_set_coef(s, graph=None, eager=None, decode=None) -> None:
    ref = lambda x: ctypes.byref(x) if x is not None else None
    _b._check(_lib().mlora_sched_set_coef(s, ref(graph), ref(eager), ref(decode)), "mlora_sched_set_coef")


def mlora_sched_pool_add(s, sample_id: int, tokens: int) -> None:
    _b._check(_lib().mlora_sched_pool_add(s, int(sample_id), int(tokens)), "mlora_sched_pool_add")


def mlora_sched_pool_size(s) -> int:
    return int(_lib().mlora_sched_pool_size(s))


def mlora_sched_buffer_left(s) -> int:
    return int(_lib().mlora_sched_buffer_left(s))


def mlora_sched_set_backward_running(s, running: bool) -> None:
    _b._check(_lib().mlora_sched_set_backward_running(s, int(bool(running))), "mlora_sched_set_backward_running")


def mlora_sched_admit(s, prefill_lens: Sequence[int], n_decode: int, kv_tokens: int, t_now: float,
                      earliest_arrival: Optional[float] = None, wait_n_decode: int = 0, wait_kv_tokens: int = 0,
                      cap: int = 4096) -> Tuple[List[int], List[int], float]:
    """Algorithm 1 with the claim.  Returns (sample ids, their token lengths, the budget Delta)."""
    arr = _i32_array(prefill_lens)
    step = mlora_step_t(arr, len(prefill_lens), int(n_decode), int(kv_tokens), float(t_now),
                        float(earliest_arrival) if earliest_arrival is not None else float("nan"),
                        int(wait_n_decode), int(wait_kv_tokens))
    ids = (ctypes.c_int64 * max(cap, 1))()
    toks = (ctypes.c_int32 * max(cap, 1))()
    n = ctypes.c_int32(0)
    budget = ctypes.c_double(0.0)
    _b._check(_lib().mlora_sched_admit(s, ctypes.byref(step), ids, toks, int(cap), ctypes.byref(n),
                                       ctypes.byref(budget)), "mlora_sched_admit")
    return list(ids[:n.value]), list(toks[:n.value]), budget.value


def mlora_sched_requeue(s, ids: Sequence[int], tokens: Sequence[int]) -> None:
    a = (ctypes.c_int64 * max(len(ids), 1))(*[int(v) for v in ids])
    t = _i32_array(tokens)
    _b._check(_lib().mlora_sched_requeue(s, a, t, len(ids)), "mlora_sched_requeue")


def mlora_sched_buffer_release(s, tokens: int) -> None:
    _b._check(_lib().mlora_sched_buffer_release(s, int(tokens)), "mlora_sched_buffer_release")


def mlora_sched_observe(s, mode: int, prefill_lens: Sequence[int], n_decode: int, kv_tokens: int, ft_tokens: int,
                        seconds: float) -> None:
    arr = _i32_array(prefill_lens)
    obs = mlora_observation_t(arr, len(prefill_lens), int(n_decode), int(kv_tokens), int(ft_tokens), float(seconds))
    _b._check(_lib().mlora_sched_observe(s, int(mode), ctypes.byref(obs)), "mlora_sched_observe")


def mlora_sched_observations(s, mode: int) -> int:
    return int(_lib().mlora_sched_observations(s, int(mode)))


def mlora_sched_refit(s, mode: int, fit_mask: int = 31) -> mlora_mixed_coef_t:
    out = mlora_mixed_coef_t()
    _b._check(_lib().mlora_sched_refit(s, int(mode), int(fit_mask), ctypes.byref(out)), "mlora_sched_refit")
    return out
