"""AdamW update of the fine-tuned adapters (mlora_adamw_update) against the fp64 oracle.

fp32 arithmetic on fp32 master weights: |err| <= 1e-5 (1 + |ref|) after three steps; the stored
weights must be exactly the master weights rounded to the storage type, and adapters that are not
being fine-tuned must not change by a bit."""
import numpy as np
import pytest
import torch

from oracle import adamw_oracle as ao
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import synth
from paper_2607_28848_b200.runner import LayerRun, Session

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_adamw_three_steps(dtype):
    with Session(0) as sess:
        segs = synth.segments_array([(0, 30, 4, 1), (30, 20, 0, 0), (50, 40, 1, 1), (90, 10, 4, 1)])
        w = synth.Workload("adamw", 128, 192, 16, 6, dtype, 100, segs)
        t = synth.make_tensors(w)
        run = LayerRun(sess, dtype, t, w.segments, w.n_rows)
        slots = run.slots
        assert slots == [4, 1]
        dev = sess.device
        A0, B0 = run.A_all.clone(), run.B_all.clone()
        idx = torch.tensor(slots, device=dev)
        wA = run.A_all[idx].float().contiguous()
        wB = run.B_all[idx].float().contiguous()
        mA, vA, mB, vB = (torch.zeros_like(x) for x in (wA, wA, wB, wB))
        ref = {k: v.cpu().numpy().astype(np.float64) for k, v in (("wA", wA), ("wB", wB))}
        ref.update(mA=np.zeros_like(ref["wA"]), vA=np.zeros_like(ref["wA"]), mB=np.zeros_like(ref["wB"]),
                   vB=np.zeros_like(ref["wB"]))
        for step in (1, 2, 3):
            gA = synth.normal(step, 71, wA.numel(), std=3.0).reshape(wA.shape).astype(np.float32)
            gB = synth.normal(step, 72, wB.numel(), std=0.01).reshape(wB.shape).astype(np.float32)
            dA, dB = torch.from_numpy(gA).to(dev), torch.from_numpy(gB).to(dev)
            mb.mlora_adamw_update(sess.ctx, run.layer, run.plan, dA, dB, wA, wB, mA, vA, mB, vB, step)
            ref["wA"], ref["mA"], ref["vA"] = ao.adamw_step(ref["wA"], gA, ref["mA"], ref["vA"], step)
            ref["wB"], ref["mB"], ref["vB"] = ao.adamw_step(ref["wB"], gB, ref["mB"], ref["vB"], step)
        torch.cuda.synchronize()
        assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_OK
        for name, got in (("wA", wA), ("wB", wB), ("mA", mA), ("vA", vA), ("mB", mB), ("vB", vB)):
            g = got.cpu().numpy().astype(np.float64)
            assert (np.abs(g - ref[name]) <= 1e-5 * (1 + np.abs(ref[name]))).all(), name
        # stored weights = master weights rounded to the storage type, bit for bit
        assert torch.equal(run.A_all[idx], wA.to(run.A_all.dtype))
        assert torch.equal(run.B_all[idx], wB.to(run.B_all.dtype))
        assert not torch.equal(run.A_all[idx], A0[idx])
        others = torch.tensor([a for a in range(6) if a not in slots], device=dev)
        assert torch.equal(run.A_all[others], A0[others]) and torch.equal(run.B_all[others], B0[others])
        # argument errors launch nothing
        before = mb.mlora_launch_count(sess.ctx)
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_adamw_update(sess.ctx, run.layer, run.plan, dA, dB, wA, wB, mA, vA, mB, vB, 0)
        assert e.value.status == mb.MLORA_ERR_INVALID_ARG
        with pytest.raises(mb.MloraError):
            mb.mlora_adamw_update(sess.ctx, run.layer, run.plan, dA, None, wA, wB, mA, vA, mB, vB, 4)
        assert mb.mlora_launch_count(sess.ctx) == before
        run.close()


def test_training_loop_reduces_a_quadratic_loss():
    """Forward -> backward -> update, repeated: with dY = Y - target the adapters move towards the
    target, i.e. the three calls compose into a working fine-tuning step."""
    with Session(0) as sess:
        segs = synth.segments_array([(0, 64, 0, 1)])
        w = synth.Workload("loop", 128, 128, 16, 1, "bf16", 64, segs)
        t = synth.make_tensors(w)
        t["B_all"] = synth.round_to_bf16(synth.normal(9, 5, t["B_all"].size, std=0.02).reshape(t["B_all"].shape))
        run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
        dev = sess.device
        target = (run.X.float() @ run.W.float()) + 0.5 * torch.randn(64, 128, device=dev, generator=torch.Generator(dev).manual_seed(0))
        wA, wB = run.A_all.float().contiguous(), run.B_all.float().contiguous()
        mA, vA, mB, vB = (torch.zeros_like(x) for x in (wA, wA, wB, wB))
        losses = []
        for step in range(1, 41):
            run.forward()
            diff = run.Y.float() - target
            losses.append(float((diff * diff).mean()))
            run.dY = diff.to(torch.bfloat16).contiguous()
            run.backward(want_dx=False)
            mb.mlora_adamw_update(sess.ctx, run.layer, run.plan, run.dA, run.dB, wA, wB, mA, vA, mB, vB, step, lr=1e-2,
                                  weight_decay=0.0)
        assert losses[-1] < 0.8 * losses[0], losses[::8]
        run.close()
