"""CPU oracle for the co-serving scheduler's arithmetic (TEST INFRASTRUCTURE ONLY).

Follows the paper's Section 4.1 (SLO budgeting) and Section 4.2 (Algorithm 1) step by step:

  Eq. I   T = alpha * sum_i (n_i + B_d)^2 + beta * (T_in + B_d) + gamma * T_ft + eps * K + c
  Eq. II  T = beta' * B_d + eps' * K + c'                              (decode-only step)
  Eq. III budget = T_SLO - (t_now - t_arrival)                         (earliest-arriving request)
  Algorithm 1: refuse when the backward runs, the buffer is full, the pool is empty, or the host
  cannot merge into a decode-only step; budget = min(TTFT slack, TPOT slack); refuse when the
  inference batch alone exceeds it; then take fine-tuning samples in increasing token length while
  the buffer holds them and the predicted mixed step stays within the budget; stop at the first
  sample that fails either test.

Readings where the paper is silent (also listed in the design notes):
  * a fine-tuning sample enters Eq. I as one more prefill entry (its length joins {n_i} and T_in:
    Section 3.2 prices it "close to one additional prefill sample") AND its tokens count in T_ft;
  * the inference-only batch is priced with the host's own mode (graph or eager coefficients), any
    batch carrying fine-tuning tokens with the eager set;
  * TTFT slack is +inf when the batch has no prefill request, TPOT slack is +inf when there is no
    decode request anywhere (neither in the step nor deferred);
  * ties in token length keep pool order (stable sort).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence


@dataclass
class MixedCoef:            # Eq. I
    alpha: float
    beta: float
    gamma: float
    eps: float
    c: float


@dataclass
class DecodeCoef:           # Eq. II
    beta: float
    eps: float
    c: float


@dataclass
class Batch:
    prefill_lens: Sequence[int] = ()
    n_decode: int = 0
    kv_tokens: int = 0


def predict_mixed(coef: MixedCoef, prefill_lens: Sequence[int], n_decode: int, kv_tokens: int, ft_tokens: int) -> float:
    attn = 0.0
    t_in = 0
    for n in prefill_lens:
        attn += float(n + n_decode) ** 2
        t_in += n
    return coef.alpha * attn + coef.beta * (t_in + n_decode) + coef.gamma * ft_tokens + coef.eps * kv_tokens + coef.c


def predict_decode(coef: DecodeCoef, n_decode: int, kv_tokens: int) -> float:
    return coef.beta * n_decode + coef.eps * kv_tokens + coef.c


def ttft_budget(t_slo: float, t_now: float, t_arrival: float) -> float:
    return t_slo - (t_now - t_arrival)


@dataclass
class AdmitState:
    backward_running: bool
    buffer_tokens_left: int                 # S_max
    mixed_batch_host: bool
    host_uses_graph: bool                   # mode of the inference-only step
    coef_graph: MixedCoef
    coef_eager: MixedCoef
    coef_decode: DecodeCoef
    t_slo_ttft: float
    t_tpot: float
    t_now: float
    earliest_arrival: Optional[float]       # of the batch's prefill requests; None: no prefill request
    deferred_decode: Optional[Batch] = None  # D_wait (hosts that run decode as its own step)


def admit(batch: Batch, pool_tokens: Sequence[int], st: AdmitState) -> List[int]:
    """Algorithm 1.  Returns the indices (into the pool) of the admitted samples, in admission order."""
    admitted: List[int] = []
    if st.backward_running or st.buffer_tokens_left <= 0 or len(pool_tokens) == 0:
        return admitted
    has_prefill = len(batch.prefill_lens) > 0
    if not st.mixed_batch_host and not has_prefill:
        return admitted
    d_tt = ttft_budget(st.t_slo_ttft, st.t_now, st.earliest_arrival) if (has_prefill and st.earliest_arrival is not None) else math.inf
    wait = st.deferred_decode
    any_decode = batch.n_decode > 0 or (wait is not None and wait.n_decode > 0)
    if any_decode:
        cost_wait = predict_decode(st.coef_decode, wait.n_decode, wait.kv_tokens) if (wait is not None and wait.n_decode > 0) else 0.0
        d_tp = st.t_tpot - cost_wait
    else:
        d_tp = math.inf
    delta = min(d_tt, d_tp)
    base_coef = st.coef_graph if st.host_uses_graph else st.coef_eager
    if predict_mixed(base_coef, batch.prefill_lens, batch.n_decode, batch.kv_tokens, 0) > delta:
        return admitted
    order = sorted(range(len(pool_tokens)), key=lambda i: (pool_tokens[i], i))
    lens = list(batch.prefill_lens)
    ft_tokens = 0
    for i in order:
        n = pool_tokens[i]
        c1 = ft_tokens + n > st.buffer_tokens_left
        c2 = predict_mixed(st.coef_eager, lens + [n], batch.n_decode, batch.kv_tokens, ft_tokens + n) > delta
        if c1 or c2:
            break
        admitted.append(i)
        lens.append(n)
        ft_tokens += n
    return admitted


def fit_mixed(observations) -> MixedCoef:
    """Least-squares fit of Eq. I's five coefficients from (prefill_lens, n_decode, kv_tokens, ft_tokens, seconds)."""
    import numpy as np
    rows, y = [], []
    for lens, bd, kv, tft, t in observations:
        rows.append([sum(float(n + bd) ** 2 for n in lens), float(sum(lens) + bd), float(tft), float(kv), 1.0])
        y.append(t)
    sol, *_ = np.linalg.lstsq(np.asarray(rows), np.asarray(y), rcond=None)
    return MixedCoef(*[float(v) for v in sol])
