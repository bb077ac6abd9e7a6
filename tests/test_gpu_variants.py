"""GPU parity of the variants with the oracle: LoRA dropout on the fine-tuning rows (mask checked
bit for bit with an exact probe, values within the layer's tolerance) and adapters of different
ranks stored with zero padding."""
import numpy as np
import pytest
import torch

from oracle import mlora_oracle as orc
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import synth
from paper_2607_28848_b200.runner import LayerRun, Session
from test_gpu_parity import TOL, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sess():
    s = Session(0)
    yield s
    mb.mlora_set_dropout(s.ctx, 0.0, 0)
    s.close()


def check_dropout(sess, w, t, p, seed, path=0, blocked=False, base=0, cap=None):
    tol = TOL[w.dtype]
    mb.mlora_set_gemm_path(sess.ctx, path)
    mb.mlora_set_dropout(sess.ctx, p, seed)
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows, save_row_base=base, save_capacity_rows=cap, guard=True)
    try:
        run.forward()
        assert run.status() == mb.MLORA_OK
        drop = (p, seed) if p > 0 else None
        fwd = (orc.forward_blocked if blocked else orc.forward)(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"],
                                                                 w.segments, dropout=drop)
        assert_close("Y", run.host(run.Y), fwd["Y"], tol)
        n = run.ft_rows
        assert n == fwd["ft_rows"] and n > 0
        assert np.array_equal(run.host(run.x_save)[base:base + n], fwd["x_save"][:n]), "x_save keeps the undropped rows"
        assert_close("u_save", run.host(run.u_save)[base:base + n], fwd["u_save"][:n], min(tol, 1e-3))
        run.backward()
        assert run.status() == mb.MLORA_OK
        bwd = (orc.backward_blocked if blocked else orc.backward)(
            t["dY"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments, fwd["x_save"], fwd["u_save"],
            n_rows=w.n_rows, dropout=drop)
        assert_close("dX", run.host(run.dX)[:n], bwd["dX"], tol)
        assert_close("dA", run.host(run.dA), bwd["dA"], tol)
        assert_close("dB", run.host(run.dB), bwd["dB"], tol)
    finally:
        mb.mlora_set_dropout(sess.ctx, 0.0, 0)
        mb.mlora_set_gemm_path(sess.ctx, 0)
        run.close()


@pytest.mark.parametrize("rank", [8, 16, 32, 64, 128])
def test_dropout_every_rank(sess, rank):
    """Ranks up to 64: the streaming kernels mask the rows as they pass; rank 128: the per-item kernels do, V comes
    from the tcgen05 shrink (no mask enters it), and the input gradient is the base product plus the masked expand."""
    # ragged table: gathered single rows, partial items, fine-tuning segments of every length
    w = synth.random_workload(40 + rank, 512, 384, rank, 5, 700, max_seg=150, p_finetune=0.45)
    check_dropout(sess, w, synth.make_tensors(w), 0.3, 2 ** 40 + rank)


def test_dropout_paper_rate_full_items_and_append(sess):
    # full 32-row items (block-saved through the tensor-map store) with the paper's p = 0.05,
    # saved behind rows of an earlier step
    segs = synth.segments_array([(0, 96, 1, 0), (96, 256, 0, 1), (352, 40, 2, 0), (392, 128, 3, 1)])
    w = synth.Workload("dropout_full_items", 1024, 512, 16, 4, "bf16", 520, segs, seed=5)
    check_dropout(sess, w, synth.make_tensors(w), 0.05, 123456789, base=64, cap=64 + 384 + 16)


def test_dropout_cuda_core_path_and_fp32(sess):
    w = synth.random_workload(77, 256, 192, 16, 4, 300, max_seg=90, p_finetune=0.5)
    check_dropout(sess, w, synth.make_tensors(w), 0.25, 99, path=1)
    w32 = synth.cfg1_tiny()
    check_dropout(sess, w32, synth.make_tensors(w32), 0.5, 7)


def test_dropout_off_is_the_plain_layer(sess):
    w = synth.random_workload(78, 256, 256, 16, 4, 200, p_finetune=0.5)
    check_dropout(sess, w, synth.make_tensors(w), 0.0, 1234)


def test_dropout_mask_bit_exact(sess):
    """Exact probe: with A[q, k] = [k mod r == q], X = 1, W = 0, B[q, j] = [j == q], dY[m, j] = [j < r], s = 1
    the forward's U[m, q] is (number of kept columns of class q) / (1 - p) and the input gradient is
    keep[m, k] / (1 - p): every element of the mask shows up exactly."""
    d_in, d_out, r, n_ad = 512, 256, 16, 2
    segs = synth.segments_array([(0, 70, 0, 1), (70, 10, 1, 0), (80, 37, 1, 1)])
    T, n_ft = 117, 107
    p, seed = 0.4, 0xDEADBEEFCAFE
    k = np.arange(d_in)
    A = (k[None, :] % r == np.arange(r)[:, None]).astype(np.float32)
    B = (np.arange(d_out)[None, :] == np.arange(r)[:, None]).astype(np.float32)
    t = {"X": np.ones((T, d_in), np.float32), "W": np.zeros((d_in, d_out), np.float32),
         "A_all": np.stack([A] * n_ad), "B_all": np.stack([B] * n_ad), "scale": np.ones(n_ad, np.float32),
         "dY": np.concatenate([np.ones((n_ft, r), np.float32), np.zeros((n_ft, d_out - r), np.float32)], axis=1)}
    keep = orc.dropout_keep_vectorised(seed, n_ft, d_in, p)
    ks = np.float32(1.0 / (1.0 - p))
    mb.mlora_set_dropout(sess.ctx, p, seed)
    run = LayerRun(sess, "bf16", t, segs, T)
    try:
        run.forward()
        run.backward()
        assert run.status() == mb.MLORA_OK
        counts = np.stack([keep[:, q::r].sum(axis=1) for q in range(r)], axis=1).astype(np.float32)
        got_u = run.u_save[:n_ft].cpu().numpy()
        assert np.array_equal(got_u, counts * ks)
        got_dx = run.dX[:n_ft].float().cpu().numpy()
        ks_bf16 = torch.tensor(float(ks)).to(torch.bfloat16).float().item()
        assert np.array_equal(got_dx, np.where(keep, np.float32(ks_bf16), np.float32(0.0)))
        # inference rows (70..79) see no dropout: Y = U B with U = d_in / r per class
        y = run.Y[70:80].float().cpu().numpy()
        assert np.array_equal(y[:, :r], np.full((10, r), d_in / r, np.float32)) and not y[:, r:].any()
    finally:
        mb.mlora_set_dropout(sess.ctx, 0.0, 0)
        run.close()


def test_dropout_refusals(sess):
    """The per-item kernels of kernel variant 2 carry the mask only at rank 128; a rate of 1 is no rate."""
    w = synth.random_workload(79, 256, 256, 16, 3, 200, p_finetune=0.5)
    t = synth.make_tensors(w)
    mb.mlora_set_dropout(sess.ctx, 0.1, 1)
    mb.mlora_set_gemm_path(sess.ctx, 2)
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows)
    try:
        with pytest.raises(mb.MloraError) as e:
            run.forward()
        assert e.value.status == mb.MLORA_ERR_UNSUPPORTED
        with pytest.raises(mb.MloraError):
            mb.mlora_set_dropout(sess.ctx, 1.0, 1)
    finally:
        mb.mlora_set_dropout(sess.ctx, 0.0, 0)
        mb.mlora_set_gemm_path(sess.ctx, 0)
        run.close()


def test_dropout_rank_128_llama_projection(sess):
    """4096 -> 4096 at rank 128, 1600 rows with 2 x 256 fine-tuning rows, p = 0.05, against the blocked oracle."""
    w0 = synth.cfg2_single_projection()
    w = synth.Workload("cfg2_rank128", w0.d_in, w0.d_out, 128, w0.n_adapters, "bf16", w0.n_rows, w0.segments, seed=31)
    check_dropout(sess, w, synth.make_tensors(w), 0.05, 777, blocked=True)


def test_dropout_llama_projection_sampled(sess):
    """4096 -> 4096, 1600 rows (1024 prefill + 64 decode + 2 x 256 fine-tune), p = 0.05: full check with
    the blocked oracle."""
    w = synth.cfg2_single_projection()
    check_dropout(sess, w, synth.make_tensors(w), 0.05, 2024, blocked=True)


def test_different_ranks_through_zero_padding(sess):
    rng_ranks = [4, 16, 8, 12, 16, 1]
    w = synth.random_workload(81, 512, 320, 16, len(rng_ranks), 600, max_seg=120, p_finetune=0.4)
    t = synth.make_tensors(w)
    A_list, B_list = [], []
    for a, ra in enumerate(rng_ranks):
        t["A_all"][a, ra:] = 0.0
        t["B_all"][a, ra:] = 0.0
        A_list.append(t["A_all"][a, :ra].copy())
        B_list.append(t["B_all"][a, :ra].copy())
        t["scale"][a] = 32.0 / ra                          # alpha / r_a
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows)
    try:
        run.forward()
        run.backward()
        assert run.status() == mb.MLORA_OK
        ref = orc.forward_ragged(t["X"], t["W"], A_list, B_list, t["scale"], w.segments)
        assert_close("Y", run.host(run.Y), ref, TOL["bf16"])
        dA, dB = run.host(run.dA), run.host(run.dB)
        fwd = orc.forward(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments)
        rag = orc.backward_ragged(t["dY"], t["W"], A_list, B_list, t["scale"], w.segments, fwd["x_save"], n_rows=w.n_rows)
        assert rag["ft_adapters"] == run.slots
        for g, a in enumerate(run.slots):
            ra = rng_ranks[a]                              # gradients of the padding rows are exactly zero,
            assert not dA[g, ra:].any() and not dB[g, ra:].any()
            assert_close(f"dA[{g}]", dA[g, :ra], rag["dA"][g], TOL["bf16"])      # the others those of the adapter's own rank
            assert_close(f"dB[{g}]", dB[g, :ra], rag["dB"][g], TOL["bf16"])
        assert_close("dX", run.host(run.dX)[:run.ft_rows], rag["dX"], TOL["bf16"])
    finally:
        run.close()


def _ragged_case(seed, d_in, d_out, R, ranks, n_rows, **kw):
    w = synth.random_workload(seed, d_in, d_out, R, len(ranks), n_rows, **kw)
    t = synth.make_tensors(w)
    A_list, B_list = [], []
    for a, ra in enumerate(ranks):
        t["A_all"][a, ra:] = 0.0
        t["B_all"][a, ra:] = 0.0
        A_list.append(t["A_all"][a, :ra].copy())
        B_list.append(t["B_all"][a, :ra].copy())
        t["scale"][a] = 32.0 / ra
    return w, t, A_list, B_list


def _check_ragged(run, w, t, A_list, B_list, ranks):
    run.forward()
    run.backward()
    assert run.status() == mb.MLORA_OK
    ref = orc.forward_ragged(t["X"], t["W"], A_list, B_list, t["scale"], w.segments)
    assert_close("Y", run.host(run.Y), ref, TOL["bf16"])
    fwd = orc.forward(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments)
    rag = orc.backward_ragged(t["dY"], t["W"], A_list, B_list, t["scale"], w.segments, fwd["x_save"], n_rows=w.n_rows)
    assert rag["ft_adapters"] == run.slots
    dA, dB = run.host(run.dA), run.host(run.dB)
    for g, a in enumerate(run.slots):
        ra = ranks[a]
        assert not dA[g, ra:].any() and not dB[g, ra:].any()
        assert_close(f"dA[{g}]", dA[g, :ra], rag["dA"][g], TOL["bf16"])
        assert_close(f"dB[{g}]", dB[g, :ra], rag["dB"][g], TOL["bf16"])
    assert_close("dX", run.host(run.dX)[:run.ft_rows], rag["dX"], TOL["bf16"])


@pytest.mark.parametrize("R,path", [(16, 0), (32, 0), (64, 0), (128, 0), (64, 2), (32, 6), (64, 7)])
def test_plans_with_per_adapter_ranks(sess, R, path):
    """mlora_plan_create_ranked: the fused expand packs every group of a tile by its own rank (rounded up to 16)
    instead of the layer's padded rank.  Same numbers as the per-rank oracle, forward and backward, on ragged tables
    with single-row groups, on every kernel that writes the GEMM's low-rank operand (streaming shrink, per-item
    shrink = kernel variant 2, tcgen05 finish kernel = ranks 64 / 128 and kernel variant 6)."""
    ranks = [r for r in (1, 4, 8, 12, 16, 24, 32, 48, 64, 100, 128) if r <= R]
    ranks = (ranks * 3)[:max(6, len(ranks))]
    w, t, A_list, B_list = _ragged_case(300 + R + path, 384, 768, R, ranks, 900, max_seg=140, p_decode=0.4, p_finetune=0.35)
    mb.mlora_set_gemm_path(sess.ctx, path)
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows, adapter_rank=ranks)
    try:
        _check_ragged(run, w, t, A_list, B_list, ranks)
    finally:
        mb.mlora_set_gemm_path(sess.ctx, 0)
        run.close()


def test_ranked_plan_gives_the_padded_plan_s_numbers_bit_for_bit(sess):
    """Packing the groups changes which zero columns the tensor cores multiply, not a single product that counts:
    a ranked plan and a plain plan over the same zero-padded adapters give identical bits."""
    ranks = [16, 64, 32, 16, 48, 8, 16, 64]
    w, t, _, _ = _ragged_case(77, 512, 1024, 64, ranks, 1100, max_seg=60, p_decode=0.5, p_finetune=0.3)
    outs = []
    for ar in (None, ranks):
        run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows, adapter_rank=ar)
        try:
            run.forward(); run.backward()
            assert run.status() == mb.MLORA_OK
            outs.append([b.clone() for b in (run.Y, run.dX, run.dA, run.dB)])
        finally:
            run.close()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_ranked_plan_refusals(sess):
    w = synth.random_workload(78, 128, 128, 8, 3, 100, p_finetune=0.4)
    t = synth.make_tensors(w)
    with pytest.raises(mb.MloraError) as e:                 # rank outside [1, 128]
        mb.mlora_plan_create_ranked(sess.ctx, w.segments, w.n_rows, 3, [4, 0, 8])
    assert e.value.status == mb.MLORA_ERR_INVALID_ARG
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows, adapter_rank=[4, 8, 8])      # layer rank 8: not a multiple of 16
    try:
        with pytest.raises(mb.MloraError) as e:
            run.forward()
        assert e.value.status == mb.MLORA_ERR_INVALID_ARG
    finally:
        run.close()
    w16 = synth.random_workload(79, 128, 128, 16, 3, 100, p_finetune=0.4)
    run = LayerRun(sess, w16.dtype, synth.make_tensors(w16), w16.segments, w16.n_rows, adapter_rank=[4, 32, 8])   # an adapter wider than the layer
    try:
        with pytest.raises(mb.MloraError) as e:
            run.forward()
        assert e.value.status == mb.MLORA_ERR_INVALID_ARG
    finally:
        run.close()
