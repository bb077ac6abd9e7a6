"""Forward (with activation save) and backward captured in a CUDA graph and replayed.

The paper's co-serving step has to run eagerly because its activation capture lives in Python
hooks that cannot run inside a replayed graph (Section 4, "Execution-mode coefficients").  Here the
save is part of a kernel, the calls allocate nothing and never synchronise, so a whole
forward + backward + update can be captured once and replayed on new inputs."""
import numpy as np
import pytest
import torch

from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import synth
from paper_2607_28848_b200.runner import LayerRun, Session

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", ["mixed", "long_k_split", "dropout", "one_finetune_adapter", "rank_128", "uneven_tiles"])
def test_graph_replay_matches_eager_on_new_inputs(case):
    with Session(0) as sess:
        if case == "long_k_split":      # few output tiles and K = 8192: the K-split GEMM and its reduction kernel
            w = synth.random_workload(62, 8192, 256, 16, 3, 200, max_seg=80, p_finetune=0.5)
        elif case == "one_finetune_adapter":   # gradient groups split over rows: partial sums and arrival counters inside the graph
            segs = synth.segments_array([(0, 60, 2, 0), (60, 900, 0, 1), (960, 40, 1, 0)])
            w = synth.Workload("one_slot", 512, 768, 16, 3, "bf16", 1000, segs, seed=63)
        elif case == "rank_128":          # tcgen05 shrink + finish kernel, operand split + tcgen05 gradient kernel
            w = synth.random_workload(66, 512, 640, 128, 4, 700, max_seg=200, p_decode=0.05, p_finetune=0.5)
        elif case == "uneven_tiles":      # the cost-balanced unit list of the GEMM is made in the warm-up and found by the capture
            segs = [(0, 256, 0, 0)] + [(256 + i, 1, 1 + i, 0) for i in range(200)] + [(456, 312, 201, 1), (768, 256, 202, 1)]
            w = synth.Workload("uneven", 512, 5120, 32, 203, "bf16", 1024, synth.segments_array(segs), seed=67)
        else:
            w = synth.random_workload(61, 256, 384, 16, 5, 420, max_seg=130, p_finetune=0.4)
        if case == "dropout":           # the seed is part of the captured launch parameters
            mb.mlora_set_dropout(sess.ctx, 0.1, 4321)
        t = synth.make_tensors(w)
        run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
        dev = sess.device
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            for _ in range(2):                      # warm-up: one-time function attributes are set here
                run.forward()
                run.backward()
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                run.forward()
                run.backward()
            # new inputs in the same buffers
            x2 = torch.from_numpy(synth.round_to_bf16(synth.normal(5, 1, run.X.numel()).reshape(run.X.shape))).to(dev).to(torch.bfloat16)
            dy2 = torch.from_numpy(synth.round_to_bf16(synth.normal(5, 2, run.dY.numel()).reshape(run.dY.shape))).to(dev).to(torch.bfloat16)
            run.X.copy_(x2)
            run.dY.copy_(dy2)
            for buf in (run.Y, run.x_save, run.u_save, run.dA, run.dB, run.dX):
                buf.zero_()
            graph.replay()
            stream.synchronize()
            replayed = [b.clone() for b in (run.Y, run.x_save, run.u_save, run.dA, run.dB, run.dX)]
            for buf in (run.Y, run.x_save, run.u_save, run.dA, run.dB, run.dX):
                buf.zero_()
            run.forward()
            run.backward()
            stream.synchronize()
        assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_OK
        for a, b in zip(replayed, (run.Y, run.x_save, run.u_save, run.dA, run.dB, run.dX)):
            assert torch.equal(a, b)
        assert float(run.Y.float().abs().max()) > 0
        run.close()


def test_a_larger_plan_after_capture_leaves_the_graph_valid():
    """A plan for a larger batch makes the context replace its workspaces by larger ones.  The blocks they
    replace stay allocated, so a graph captured before still runs on memory of its own: its replay gives
    the eager result, and so does the large batch."""
    with Session(0) as sess:
        w = synth.random_workload(64, 256, 384, 16, 5, 300, max_seg=90, p_finetune=0.4)
        t = synth.make_tensors(w)
        run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
        stream = torch.cuda.Stream(device=sess.device)
        with torch.cuda.stream(stream):
            for _ in range(2):
                run.forward(); run.backward()
            stream.synchronize()
            eager = [b.clone() for b in (run.Y, run.u_save, run.dA, run.dB, run.dX)]
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                run.forward(); run.backward()
            # many more rows, items and adapter groups than anything this context has seen
            big = synth.random_workload(65, 256, 384, 16, 40, 9000, max_seg=60, p_decode=0.6, p_finetune=0.3)
            tb = synth.make_tensors(big)
            run_big = LayerRun(sess, "bf16", tb, big.segments, big.n_rows)
            run_big.forward(); run_big.backward()
            stream.synchronize()
            for b in (run.Y, run.u_save, run.dA, run.dB, run.dX):
                b.zero_()
            graph.replay()
            stream.synchronize()
        assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_OK
        for a, b in zip(eager, (run.Y, run.u_save, run.dA, run.dB, run.dX)):
            assert torch.equal(a, b)
        from oracle import mlora_oracle as orc
        ref = orc.forward_blocked(tb["X"], tb["W"], tb["A_all"], tb["B_all"], tb["scale"], big.segments)["Y"]
        got = run_big.host(run_big.Y)
        assert (np.abs(got - ref) <= 2e-2 * (1 + np.abs(ref))).all()
        run.close(); run_big.close()
