"""Pins for the scheduler oracle: a hand-computed example, the equations' special cases, the
refusal conditions of Algorithm 1, and properties any correct admission must have."""
import math

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from conftest import load_golden
from oracle import sched_oracle as so

EAGER = so.MixedCoef(1e-5, 0.01, 0.002, 1e-4, 1.0)
GRAPH = so.MixedCoef(1e-5, 0.008, 0.002, 1e-4, 0.2)
DEC = so.DecodeCoef(0.02, 1e-4, 0.5)


def state(**kw):
    base = dict(backward_running=False, buffer_tokens_left=1000, mixed_batch_host=True, host_uses_graph=False,
                coef_graph=GRAPH, coef_eager=EAGER, coef_decode=DEC, t_slo_ttft=400.0, t_tpot=120.0, t_now=1000.0,
                earliest_arrival=610.0, deferred_decode=None)
    base.update(kw)
    return so.AdmitState(**base)


BATCH = so.Batch(prefill_lens=[100, 200], n_decode=10, kv_tokens=5000)
POOL = [300, 50, 120, 50]


def test_hand_computed_example():
    g = load_golden("admission_example.txt")
    assert so.predict_mixed(EAGER, BATCH.prefill_lens, 10, 5000, 0) == pytest.approx(g["inference_only_ms"][0, 0], abs=1e-12)
    assert so.ttft_budget(400.0, 1000.0, 610.0) == g["budget_ms"][0, 0]
    got = so.admit(BATCH, POOL, state())
    assert got == g["admitted_buffer_1000"][0].astype(int).tolist()
    lens, tft = [100, 200], 0
    for i, expect in zip(got, g["step_ms_after_each"][0]):
        lens.append(POOL[i]); tft += POOL[i]
        assert so.predict_mixed(EAGER, lens, 10, 5000, tft) == pytest.approx(expect, abs=1e-9)
    assert so.admit(BATCH, POOL, state(buffer_tokens_left=200)) == g["admitted_buffer_200"][0].astype(int).tolist()


def test_equation_special_cases():
    # no prefill, no fine-tuning: Eq. I collapses to beta B_d + eps K + c, the shape of Eq. II
    assert so.predict_mixed(EAGER, [], 7, 300, 0) == pytest.approx(0.01 * 7 + 1e-4 * 300 + 1.0)
    assert so.predict_decode(DEC, 7, 300) == pytest.approx(0.02 * 7 + 1e-4 * 300 + 0.5)
    # one prompt, nothing else: alpha n^2 + beta n + c
    assert so.predict_mixed(EAGER, [1000], 0, 0, 0) == pytest.approx(1e-5 * 1e6 + 10.0 + 1.0)
    # splitting a fixed prefill length across requests lowers only the quadratic term
    a = so.predict_mixed(EAGER, [400], 0, 0, 0)
    b = so.predict_mixed(EAGER, [200, 200], 0, 0, 0)
    assert a - b == pytest.approx(1e-5 * (400 ** 2 - 2 * 200 ** 2))
    assert so.ttft_budget(400, 50, 50) == 400 and so.ttft_budget(400, 500, 50) == -50


@pytest.mark.parametrize("kw", [dict(backward_running=True), dict(buffer_tokens_left=0), dict(buffer_tokens_left=-5)])
def test_refusals(kw):
    assert so.admit(BATCH, POOL, state(**kw)) == []


def test_more_refusals():
    assert so.admit(BATCH, [], state()) == []                                         # empty pool
    decode_only = so.Batch([], 32, 9000)
    assert so.admit(decode_only, POOL, state(mixed_batch_host=False, earliest_arrival=None)) == []
    assert so.admit(decode_only, POOL, state(mixed_batch_host=True, earliest_arrival=None)) != []
    assert so.admit(BATCH, POOL, state(t_now=1395.0)) == []                            # no slack even without fine-tuning
    # a deferred decode batch is charged against the TPOT slack
    wait = so.Batch([], 4000, 10 ** 6)                                                 # 80 + 100 + 0.5 ms > 120
    assert so.admit(BATCH, POOL, state(mixed_batch_host=False, deferred_decode=wait)) == []


def test_graph_mode_prices_only_the_inference_batch():
    # the inference-only check uses the graph set, every mixed batch the eager set
    tight = state(host_uses_graph=True, t_now=1000.0, earliest_arrival=1000.0 - 400.0 + 5.0)   # budget 5 ms
    assert so.predict_mixed(GRAPH, BATCH.prefill_lens, 10, 5000, 0) < 5.0 < so.predict_mixed(EAGER, BATCH.prefill_lens, 10, 5000, 0)
    assert so.admit(BATCH, POOL, tight) == []          # passes the first check, but no eager mixed batch fits


@settings(max_examples=200, deadline=None)
@given(pool=st.lists(st.integers(1, 600), min_size=0, max_size=12), buf=st.integers(-10, 1500),
       budget=st.floats(0.0, 40.0), n_dec=st.integers(0, 64), lens=st.lists(st.integers(1, 800), max_size=4))
def test_admission_properties(pool, buf, budget, n_dec, lens):
    batch = so.Batch(lens, n_dec, 1000 * n_dec)
    s = state(buffer_tokens_left=buf, t_now=1000.0, earliest_arrival=1000.0 - 400.0 + budget if lens else None,
              t_tpot=1e9)
    got = so.admit(batch, pool, s)
    order = sorted(range(len(pool)), key=lambda i: (pool[i], i))
    assert got == order[:len(got)]                                   # a prefix of the length-sorted pool
    tokens = sum(pool[i] for i in got)
    assert tokens <= max(buf, 0)
    delta = budget if lens else math.inf
    if got:
        assert so.predict_mixed(EAGER, list(lens) + [pool[i] for i in got], n_dec, batch.kv_tokens, tokens) <= delta
    if len(got) < len(pool) and buf > 0 and so.predict_mixed(EAGER, lens, n_dec, batch.kv_tokens, 0) <= delta:
        nxt = order[len(got)]                                        # the first sample left out fails a test
        over_buf = tokens + pool[nxt] > buf
        over_t = so.predict_mixed(EAGER, list(lens) + [pool[i] for i in got] + [pool[nxt]], n_dec, batch.kv_tokens,
                                  tokens + pool[nxt]) > delta
        assert over_buf or over_t


def test_fit_recovers_coefficients():
    rng = np.random.default_rng(0)
    true = so.MixedCoef(2e-6, 0.004, 0.0015, 3e-5, 0.7)
    obs = []
    for _ in range(60):
        lens = rng.integers(1, 1500, rng.integers(0, 5)).tolist()
        bd, kv, tft = int(rng.integers(0, 128)), int(rng.integers(0, 10 ** 6)), int(rng.integers(0, 2000))
        obs.append((lens, bd, kv, tft, so.predict_mixed(true, lens, bd, kv, tft)))
    fit = so.fit_mixed(obs)
    for name in ("alpha", "beta", "gamma", "eps", "c"):
        assert getattr(fit, name) == pytest.approx(getattr(true, name), rel=1e-6, abs=1e-9)
