"""The allocation-free forward (mlora_forward_noalloc) against the regular planned forward.

Some users of the library may not allocate device memory - an engine that gave its whole budget to
its own pool, a worker living on buffers mapped from another process - so they cannot create the
context and plan the regular path needs.  The allocation-free entry point keeps its rank-r
intermediate in a scratch array inside the library instead.  Here it is called twice in a row
through the C ABI, the second time on a smaller batch with different adapters so that whatever
the first call left in the shared scratch would show, and compared with mlora_mixed_forward and
with the CPU oracle.  A table entry outside the layer's adapters must behave like "no adapter".
This file sorts last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import mlora_oracle as orc
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import synth
from paper_2607_28848_b200.runner import LayerRun, Session

pytestmark = pytest.mark.gpu


def _reference(sess, w, t):
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows)
    run.forward()
    assert run.status() == mb.MLORA_OK
    return run


@pytest.mark.parametrize("dtype,tol", [("bf16", 2e-2), ("f32", 1e-4)])
def test_noalloc_matches_planned_forward_twice(dtype, tol):
    with Session(0) as sess:
        for seed, n_rows in ((31, 300), (32, 77)):            # two calls in a row, the second smaller
            w = synth.random_workload(seed, 128, 192, 16, 5, n_rows, dtype=dtype, max_seg=40, p_finetune=0.0)
            t = synth.make_tensors(w)
            ref = _reference(sess, w, t)
            _so, row_adapter = mb.mlora_plan_describe(ref.plan, len(w.segments))
            ra = torch.from_numpy(row_adapter).to(sess.device)
            Y = torch.full_like(ref.Y, float("nan"))
            mb.mlora_forward_noalloc(ref.layer, ra, ref.X, Y)
            torch.cuda.synchronize()
            got, want = Y.float().cpu().numpy().astype(np.float64), ref.host(ref.Y)
            assert np.isfinite(got).all()
            assert (np.abs(got - want) <= tol * (1 + np.abs(want))).all()
            oracle = orc.forward(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments)["Y"]
            assert (np.abs(got - oracle) <= tol * (1 + np.abs(oracle))).all()
            ref.close()


def test_noalloc_ids_outside_the_adapter_tables_mean_no_adapter():
    """The caller's device table cannot be checked on the host.  Rows whose id is >= n_adapters or
    below -1 must get the base product only (the oracle's result for adapter -1), and the call
    must leave the device healthy."""
    with Session(0) as sess:
        w = synth.random_workload(34, 128, 192, 16, 5, 90, dtype="bf16", max_seg=30, p_finetune=0.0)
        t = synth.make_tensors(w)
        ref = _reference(sess, w, t)
        _so, row_adapter = mb.mlora_plan_describe(ref.plan, len(w.segments))
        bad = row_adapter.copy()
        bad[3], bad[40], bad[77] = 5, 1 << 20, -7
        Y = torch.full_like(ref.Y, float("nan"))
        mb.mlora_forward_noalloc(ref.layer, torch.from_numpy(bad).to(sess.device), ref.X, Y)
        torch.cuda.synchronize()
        expect_ra = bad.copy()
        expect_ra[[3, 40, 77]] = -1
        segs = np.array([[i, 1, a, 0] for i, a in enumerate(expect_ra)], dtype=np.int32)
        oracle = orc.forward(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], segs)["Y"]
        got = Y.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert (np.abs(got - oracle) <= 2e-2 * (1 + np.abs(oracle))).all()
        assert ref.status() == mb.MLORA_OK
        ref.close()


def test_noalloc_limits_are_refused():
    with Session(0) as sess:
        w = synth.random_workload(33, 64, 64, 8, 2, 16, dtype="f32", max_seg=8, p_finetune=0.0)
        ref = _reference(sess, w, synth.make_tensors(w))
        too_many = torch.zeros(mb.MLORA_NOALLOC_MAX_ROWS + 1, dtype=torch.int32, device=sess.device)
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_forward_noalloc(ref.layer, too_many, ref.X, ref.Y)
        assert e.value.status == mb.MLORA_ERR_UNSUPPORTED
        mb.mlora_forward_noalloc(ref.layer, too_many[:0], ref.X, ref.Y)      # empty batch: no-op
        ref.close()
