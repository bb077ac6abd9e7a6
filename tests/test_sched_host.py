"""The C scheduler entry points against the scheduler oracle (no GPU): Eq. I/II/III values,
Algorithm 1's admitted set on random steps, the claim's bookkeeping and the calibration fit."""
import math

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from conftest import load_golden
from oracle import sched_oracle as so
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import sched as ms

EAGER = (1e-5, 0.01, 0.002, 1e-4, 1.0)
GRAPH = (1e-5, 0.008, 0.002, 1e-4, 0.2)
DEC = (0.02, 1e-4, 0.5)


def make(buffer_tokens=1000, mixed=True, graph=False, slo=400.0, tpot=120.0):
    return ms.mlora_sched_create(ms.mixed_coef(*GRAPH), ms.mixed_coef(*EAGER), ms.decode_coef(*DEC), slo, tpot,
                                 buffer_tokens, mixed, graph)


def oracle_state(**kw):
    base = dict(backward_running=False, buffer_tokens_left=1000, mixed_batch_host=True, host_uses_graph=False,
                coef_graph=so.MixedCoef(*GRAPH), coef_eager=so.MixedCoef(*EAGER), coef_decode=so.DecodeCoef(*DEC),
                t_slo_ttft=400.0, t_tpot=120.0, t_now=1000.0, earliest_arrival=610.0, deferred_decode=None)
    base.update(kw)
    return so.AdmitState(**base)


def test_hand_computed_example_through_the_library():
    g = load_golden("admission_example.txt")
    assert ms.mlora_predict_mixed(ms.mixed_coef(*EAGER), [100, 200], 10, 5000, 0) == pytest.approx(g["inference_only_ms"][0, 0], abs=1e-12)
    assert ms.mlora_ttft_budget(400.0, 1000.0, 610.0) == g["budget_ms"][0, 0]
    for buf, key in ((1000, "admitted_buffer_1000"), (200, "admitted_buffer_200")):
        s = make(buf)
        try:
            for i, n in enumerate([300, 50, 120, 50]):
                ms.mlora_sched_pool_add(s, i, n)
            ids, toks, budget = ms.mlora_sched_admit(s, [100, 200], 10, 5000, 1000.0, 610.0)
            assert ids == g[key][0].astype(int).tolist()
            assert budget == 10.0
            assert ms.mlora_sched_pool_size(s) == 4 - len(ids)
            assert ms.mlora_sched_buffer_left(s) == buf - sum(toks)
        finally:
            ms.mlora_sched_destroy(s)


@settings(max_examples=300, deadline=None)
@given(pool=st.lists(st.integers(1, 600), min_size=0, max_size=14), buf=st.integers(0, 1500),
       budget=st.floats(0.0, 40.0), n_dec=st.integers(0, 64), lens=st.lists(st.integers(1, 800), max_size=4),
       mixed=st.booleans(), graph=st.booleans(), wait=st.integers(0, 3000), bwd=st.booleans(),
       tpot=st.floats(1.0, 200.0))
def test_admit_matches_oracle(pool, buf, budget, n_dec, lens, mixed, graph, wait, bwd, tpot):
    arrival = 1000.0 - 400.0 + budget
    s = make(buf, mixed, graph, tpot=tpot)
    try:
        for i, n in enumerate(pool):
            ms.mlora_sched_pool_add(s, 100 + i, n)
        ms.mlora_sched_set_backward_running(s, bwd)
        ids, toks, _ = ms.mlora_sched_admit(s, lens, n_dec, 1000 * n_dec, 1000.0, arrival if lens else None,
                                            wait_n_decode=wait, wait_kv_tokens=500 * wait)
        expect = so.admit(so.Batch(lens, n_dec, 1000 * n_dec), pool,
                          oracle_state(backward_running=bwd, buffer_tokens_left=buf, mixed_batch_host=mixed,
                                       host_uses_graph=graph, t_tpot=tpot,
                                       earliest_arrival=arrival if lens else None,
                                       deferred_decode=so.Batch([], wait, 500 * wait) if wait else None))
        assert ids == [100 + i for i in expect]
        assert toks == [pool[i] for i in expect]
        assert ms.mlora_sched_pool_size(s) == len(pool) - len(expect)
        assert ms.mlora_sched_buffer_left(s) == buf - sum(toks)
    finally:
        ms.mlora_sched_destroy(s)


def test_claim_requeue_release():
    s = make(300)
    try:
        for i, n in enumerate([100, 100, 100, 100, 100]):
            ms.mlora_sched_pool_add(s, i, n)
        with pytest.raises(mb.MloraError):
            ms.mlora_sched_pool_add(s, 3, 10)                       # duplicate id
        with pytest.raises(mb.MloraError):
            ms.mlora_sched_pool_add(s, 9, 0)
        loose = dict(prefill_lens=[], n_decode=0, kv_tokens=0, t_now=0.0)
        ids1, toks1, budget = ms.mlora_sched_admit(s, **loose)
        assert ids1 == [0, 1, 2] and math.isinf(budget)             # buffer holds three samples
        ids2, _, _ = ms.mlora_sched_admit(s, **loose)
        assert ids2 == [] and ms.mlora_sched_buffer_left(s) == 0    # nothing is selected twice, no overcommit
        ms.mlora_sched_requeue(s, ids1[1:], toks1[1:])              # an interrupted forward returns two samples
        assert ms.mlora_sched_pool_size(s) == 4 and ms.mlora_sched_buffer_left(s) == 200
        ids3, _, _ = ms.mlora_sched_admit(s, **loose)
        assert ids3 == [3, 4]                                       # requeued samples queue behind equal lengths
        assert ms.mlora_sched_pool_size(s) == 2 and ms.mlora_sched_buffer_left(s) == 0
        with pytest.raises(mb.MloraError):
            ms.mlora_sched_requeue(s, [1], [100])                   # already in the pool
        ms.mlora_sched_buffer_release(s, 100)                       # the backward consumed one sample
        assert ms.mlora_sched_buffer_left(s) == 100
        with pytest.raises(mb.MloraError):
            ms.mlora_sched_buffer_release(s, 201)                   # more than is reserved
        ms.mlora_sched_set_backward_running(s, True)
        assert ms.mlora_sched_admit(s, **loose)[0] == []
        ms.mlora_sched_set_backward_running(s, False)
        assert ms.mlora_sched_admit(s, **loose)[0] == [1]
    finally:
        ms.mlora_sched_destroy(s)


def test_set_coef_changes_the_decision():
    s = make(10 ** 6)
    try:
        for i in range(8):
            ms.mlora_sched_pool_add(s, i, 64)
        args = dict(prefill_lens=[128], n_decode=0, kv_tokens=0, t_now=100.0, earliest_arrival=100.0)
        ms.mlora_sched_set_coef(s, eager=ms.mixed_coef(0.0, 1.0, 0.0, 0.0, 0.0))   # 1 per token, budget 400
        ids, _, _ = ms.mlora_sched_admit(s, **args)
        assert len(ids) == (400 - 128) // 64
        ms.mlora_sched_set_coef(s, eager=ms.mixed_coef(0.0, 2.0, 0.0, 0.0, 0.0))   # twice the cost per token
        ids, _, _ = ms.mlora_sched_admit(s, **args)
        assert len(ids) == (200 - 128) // 64
    finally:
        ms.mlora_sched_destroy(s)


def test_fit_matches_oracle_and_recovers_truth():
    rng = np.random.default_rng(3)
    true = so.MixedCoef(2e-6, 0.004, 0.0015, 3e-5, 0.7)
    obs = []
    for _ in range(80):
        lens = rng.integers(1, 1500, rng.integers(0, 5)).tolist()
        bd, kv, tft = int(rng.integers(0, 128)), int(rng.integers(0, 10 ** 6)), int(rng.integers(0, 2000))
        obs.append((lens, bd, kv, tft, so.predict_mixed(true, lens, bd, kv, tft) * (1 + 0.01 * rng.standard_normal())))
    got = ms.mlora_fit_mixed(obs)
    ref = so.fit_mixed(obs)
    for name in ("alpha", "beta", "gamma", "eps", "c"):
        assert getattr(got, name) == pytest.approx(getattr(ref, name), rel=1e-7, abs=1e-12)
        assert getattr(got, name) == pytest.approx(getattr(true, name), rel=0.2)
    # reduced model: only beta, gamma, c (no attention, no KV cache)
    lin = [([n], 0, 0, f, 0.003 * n + 0.001 * f + 0.05) for n in (64, 256, 1024, 2048) for f in (0, 128, 512)]
    red = ms.mlora_fit_mixed(lin, ms.FIT_BETA | ms.FIT_GAMMA | ms.FIT_C)
    assert (red.alpha, red.eps) == (0.0, 0.0)
    assert red.beta == pytest.approx(0.003, rel=1e-9) and red.gamma == pytest.approx(0.001, rel=1e-9)
    assert red.c == pytest.approx(0.05, rel=1e-9)
    with pytest.raises(mb.MloraError) as e:
        ms.mlora_fit_mixed(lin, 31)                                  # kv column is all zero: not identifiable
    assert e.value.status == mb.MLORA_ERR_UNSUPPORTED
    with pytest.raises(mb.MloraError):
        ms.mlora_fit_mixed(lin[:2], ms.FIT_BETA | ms.FIT_GAMMA | ms.FIT_C)


def test_predictors_reject_null():
    lib = mb.load_library()
    ms._lib()
    assert math.isnan(lib.mlora_predict_mixed(None, None, 0, 0, 0, 0))
    assert math.isnan(lib.mlora_predict_decode(None, 1, 1))
    assert ms.mlora_predict_decode(ms.decode_coef(*DEC), 7, 300) == pytest.approx(0.02 * 7 + 1e-4 * 300 + 0.5)


def test_online_refit_tracks_a_drift_and_changes_admission():
    """Observed steps go into a ring per execution mode; a refit installs the new coefficients, and the
    admission that follows prices batches with them."""
    s = make(10 ** 6)
    try:
        rng = np.random.default_rng(5)
        slow = so.MixedCoef(0.0, 0.004, 0.001, 0.0, 0.3)           # the eager path got 40% slower per token
        obs = []
        for _ in range(700):                                         # more than the ring holds
            lens = rng.integers(16, 900, rng.integers(1, 4)).tolist()
            bd, tft = int(rng.integers(0, 64)), int(rng.integers(0, 1024))
            t = so.predict_mixed(slow, lens, bd, 0, tft)
            obs.append((lens, bd, 0, tft, t))
            ms.mlora_sched_observe(s, ms.MODE_EAGER, lens, bd, 0, tft, t)
        assert ms.mlora_sched_observations(s, ms.MODE_EAGER) == 512 and ms.mlora_sched_observations(s, ms.MODE_GRAPH) == 0
        with pytest.raises(mb.MloraError):
            ms.mlora_sched_refit(s, ms.MODE_GRAPH)                   # nothing observed in that mode
        got = ms.mlora_sched_refit(s, ms.MODE_EAGER, ms.FIT_ALPHA | ms.FIT_BETA | ms.FIT_GAMMA | ms.FIT_C)
        ref = so.fit_mixed(obs[-512:])                                # the ring keeps the most recent 512
        assert got.beta == pytest.approx(0.004, rel=1e-9) and got.gamma == pytest.approx(0.001, rel=1e-9)
        assert got.c == pytest.approx(0.3, rel=1e-9) and got.beta == pytest.approx(ref.beta, rel=1e-6)
        assert abs(got.alpha) < 1e-12 and got.eps == EAGER[3]        # eps is outside the mask: unchanged
        for i in range(6):
            ms.mlora_sched_pool_add(s, i, 100)
        # budget 2.0: inference 0.3 + 0.004 * 200 = 1.1; a sample costs 100 * (0.004 + 0.001) = 0.5 -> one fits
        ids, _, _ = ms.mlora_sched_admit(s, [200], 0, 0, t_now=398.0, earliest_arrival=0.0)
        assert len(ids) == 1
    finally:
        ms.mlora_sched_destroy(s)
