"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates segment tables with the documented error codes, and derives the same
routing / save offsets / gradient slots as the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import mlora_oracle as orc
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2607_28848_b200 import layer_ops as mo
    from paper_2607_28848_b200 import sched as ms
    lib = mb.load_library()
    bound = {"mlora.h": set(mb.EXPORTS), "mlora_sched.h": set(ms.EXPORTS), "mlora_layer_ops.h": set(mo.EXPORTS)}
    inc = os.path.join(ROOT, "include")
    assert sorted(f for f in os.listdir(inc) if f.endswith(".h")) == sorted(bound)
    for fname, names in bound.items():
        header = open(os.path.join(inc, fname)).read()
        header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
        declared = set(re.findall(r"\b(mlora_[a-z_]+)\s*\(", header))
        assert declared == names, fname
        for name in declared:
            assert hasattr(lib, name), name


def test_status_strings():
    for s in range(11):
        assert mb.status_string(s) and mb.status_string(s) != "unknown status"
    assert mb.status_string(99) == "unknown status"


def host_plan(segs, n_rows, n_adapters):
    return mb.mlora_plan_create(None, segs, n_rows, n_adapters)


def test_plan_offsets_hand_listed():
    segs = [(10, 4, 2, 1), (0, 3, 1, 0), (3, 0, 0, 1), (20, 5, 0, 1), (4, 2, 2, 1)]
    p = host_plan(segs, 30, 3)
    try:
        assert mb.mlora_plan_rows(p) == 30
        assert mb.mlora_plan_ft_rows(p) == 11
        assert mb.mlora_plan_ft_adapters(p) == [2, 0]
        so, ra = mb.mlora_plan_describe(p, len(segs))
        assert so.tolist() == [0, -1, 4, 4, 9]
        assert ra[:7].tolist() == [1, 1, 1, -1, 2, 2, -1]
    finally:
        mb.mlora_plan_destroy(p)


@pytest.mark.parametrize("bad,code", [
    ([(0, 5, 0, 0), (4, 2, 1, 0)], mb.MLORA_ERR_SEGMENT_OVERLAP),
    ([(28, 5, 0, 0)], mb.MLORA_ERR_SEGMENT_RANGE),
    ([(-1, 2, 0, 0)], mb.MLORA_ERR_SEGMENT_RANGE),
    ([(0, -2, 0, 0)], mb.MLORA_ERR_SEGMENT_RANGE),
    ([(0, 2, 3, 0)], mb.MLORA_ERR_ADAPTER_ID),
    ([(0, 2, -2, 0)], mb.MLORA_ERR_ADAPTER_ID),
    ([(0, 2, -1, 1)], mb.MLORA_ERR_ADAPTER_ID),
])
def test_plan_refuses_bad_tables(bad, code):
    with pytest.raises(mb.MloraError) as e:
        host_plan(bad, 30, 3)
    assert e.value.status == code


def test_ranked_plan_on_the_host():
    """Per-adapter ranks do not touch routing: same offsets, slots and row table; ranks outside [1, 128] are refused;
    no rank array is the plain plan."""
    segs = [(10, 4, 2, 1), (0, 3, 1, 0), (20, 5, 0, 1), (4, 2, 2, 1)]
    plain = host_plan(segs, 30, 3)
    ranked = mb.mlora_plan_create_ranked(None, segs, 30, 3, [4, 128, 17])
    try:
        assert mb.mlora_plan_ft_adapters(ranked) == mb.mlora_plan_ft_adapters(plain) == [2, 0]
        a, b = mb.mlora_plan_describe(plain, len(segs)), mb.mlora_plan_describe(ranked, len(segs))
        assert a[0].tolist() == b[0].tolist() and a[1].tolist() == b[1].tolist()
    finally:
        mb.mlora_plan_destroy(plain)
        mb.mlora_plan_destroy(ranked)
    for bad in ([4, 0, 8], [4, 129, 8], [-1, 8, 8]):
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_plan_create_ranked(None, segs, 30, 3, bad)
        assert e.value.status == mb.MLORA_ERR_INVALID_ARG


def test_lowrank_columns_hand_listed():
    """600 rows = three 256-row tiles.  Tile 0: adapters 0 and 2; tile 1: adapters 2 (continued), 1 and 3, and a
    stretch without adapter; tile 2: adapter 3 (continued) and a fine-tuning segment of adapter 0."""
    segs = [(0, 100, 0, 0), (100, 200, 2, 0), (300, 50, 1, 0), (350, 60, -1, 0), (410, 140, 3, 0), (550, 50, 0, 1)]
    plain = host_plan(segs, 600, 4)
    ranked = mb.mlora_plan_create_ranked(None, segs, 600, 4, [8, 40, 64, 17])      # widths 16, 48, 64, 32
    try:
        assert mb.mlora_plan_lowrank_columns(plain, 64) == [2 * 64, 3 * 64, 2 * 64]
        assert mb.mlora_plan_lowrank_columns(plain, 16) == [32, 48, 32]
        assert mb.mlora_plan_lowrank_columns(ranked, 64) == [16 + 64, 64 + 48 + 32, 32 + 16]
    finally:
        mb.mlora_plan_destroy(plain)
        mb.mlora_plan_destroy(ranked)


def test_empty_table_and_empty_batch():
    p = host_plan(np.zeros((0, 4), np.int32), 5, 2)
    assert mb.mlora_plan_ft_rows(p) == 0 and mb.mlora_plan_ft_adapters(p) == []
    mb.mlora_plan_destroy(p)
    p = host_plan(np.zeros((0, 4), np.int32), 0, 2)
    assert mb.mlora_plan_rows(p) == 0
    mb.mlora_plan_destroy(p)


@settings(max_examples=60, deadline=None)
@given(seed=st.integers(0, 10 ** 6), n_rows=st.integers(1, 400), n_adapters=st.integers(1, 9))
def test_plan_matches_oracle_routing(seed, n_rows, n_adapters):
    w = synth.random_workload(seed, 8, 8, 8, n_adapters, n_rows, max_seg=50)
    row_adapter, ft, ft_rows, slots = orc.route(w.segments, n_rows, n_adapters)
    p = host_plan(w.segments, n_rows, n_adapters)
    try:
        assert mb.mlora_plan_ft_rows(p) == ft_rows
        assert mb.mlora_plan_ft_adapters(p) == slots
        so, ra = mb.mlora_plan_describe(p, len(w.segments))
        assert ra.tolist() == row_adapter.tolist()
        expect = [-1] * len(w.segments)
        it = iter(ft)
        for k, seg in enumerate(w.segments.tolist()):
            if seg[3]:
                expect[k] = next(it)[3]
        assert so.tolist() == expect
    finally:
        mb.mlora_plan_destroy(p)


def test_no_gpu_means_no_compute():
    """Without an sm_100 device the context cannot be created and the compute calls refuse to run."""
    import torch
    lib = mb.load_library()
    if not torch.cuda.is_available():
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_create(0)
        assert e.value.status == mb.MLORA_ERR_ARCH
    layer = mb.mlora_layer_t()
    st_ = lib.mlora_mixed_forward(None, ctypes.byref(layer), None, None, 0, None, 0, None, None, 0, 0, None)
    assert st_ == mb.MLORA_ERR_INVALID_ARG
    st_ = lib.mlora_backward(None, ctypes.byref(layer), None, None, 0, None, None, None, None, None, 0, 0, None)
    assert st_ == mb.MLORA_ERR_INVALID_ARG
    # a host-only plan cannot be executed either
    p = host_plan([(0, 2, 0, 1)], 4, 1)
    assert lib.mlora_mixed_forward(None, ctypes.byref(layer), p, None, 0, None, 0, None, None, 0, 0, None) \
        == mb.MLORA_ERR_INVALID_ARG
    mb.mlora_plan_destroy(p)
