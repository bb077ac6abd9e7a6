"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Tolerances: bf16 layers  |err| <= 2e-2 (1 + |ref|)  (bf16 storage, fp32 accumulation);
fp32 layers |err| <= 1e-4 (1 + |ref|).  Routing and the activation-save indexing are checked
bit for bit (saved rows of X, and the exact-integer probe where every output is an integer).
"""
import numpy as np
import pytest
import torch

from oracle import mlora_oracle as orc
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import synth
from paper_2607_28848_b200.runner import LayerRun, Session
from probes import integer_probe

pytestmark = pytest.mark.gpu

TOL = {"bf16": 2e-2, "f32": 1e-4}


@pytest.fixture(scope="module")
def sess():
    s = Session(0)
    yield s
    s.close()


def assert_close(name, got, ref, tol):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    excess = np.abs(got - ref) - tol * (1.0 + np.abs(ref))
    if excess.size and excess.max() > 0:
        i = np.unravel_index(np.argmax(excess), excess.shape)
        raise AssertionError(f"{name}: |err| {abs(got[i] - ref[i]):.4g} at {i} (got {got[i]:.6g}, ref {ref[i]:.6g}), "
                             f"{int((excess > 0).sum())} of {excess.size} outside tolerance {tol}")


def run_and_check(sess, w, t, path=0, check_backward=True, tol=None, base=0, cap=None, blocked=False):
    tol = TOL[w.dtype] if tol is None else tol
    mb.mlora_set_gemm_path(sess.ctx, path)
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows, save_row_base=base, save_capacity_rows=cap, guard=True)
    try:
        run.forward()
        assert run.status() == mb.MLORA_OK
        fwd = (orc.forward_blocked if blocked else orc.forward)(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"],
                                                                 w.segments)
        assert_close("Y", run.host(run.Y), fwd["Y"], tol)
        n = run.ft_rows
        assert n == fwd["ft_rows"] and run.slots == fwd["ft_adapters"]
        if n:
            xs = run.host(run.x_save)[base:base + n]
            assert np.array_equal(xs, fwd["x_save"][:n]), "saved rows of X must be bit-exact copies"
            assert_close("u_save", run.host(run.u_save)[base:base + n], fwd["u_save"][:n], min(tol, 1e-3))
        # guard: rows of the activation buffer outside [base, base + n) are untouched
        assert torch.isnan(run.u_save[:base]).all() and torch.isnan(run.u_save[base + n:]).all()
        assert torch.isnan(run.x_save[:base].float()).all() and torch.isnan(run.x_save[base + n:].float()).all()
        if check_backward and n:
            run.backward()
            assert run.status() == mb.MLORA_OK
            bwd = (orc.backward_blocked if blocked else orc.backward)(
                t["dY"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments, fwd["x_save"], fwd["u_save"],
                n_rows=w.n_rows)
            assert_close("dX", run.host(run.dX)[:n], bwd["dX"], tol)
            assert_close("dA", run.host(run.dA), bwd["dA"], tol)
            assert_close("dB", run.host(run.dB), bwd["dB"], tol)
        return run
    finally:
        mb.mlora_set_gemm_path(sess.ctx, 0)
        run.close()


# ------------------------------------------------------------------------------------------
def test_cfg1_tiny_fp32(sess):
    w = synth.cfg1_tiny()
    run_and_check(sess, w, synth.make_tensors(w))


@pytest.mark.parametrize("path", [0, 1, 2, 3, 4, 5, 6])
def test_bf16_ragged_multi_tile(sess, path):
    w = synth.random_workload(5, 256, 512, 16, 6, 389, max_seg=150)
    run_and_check(sess, w, synth.make_tensors(w), path=path)


def test_fp32_ragged(sess):
    w = synth.random_workload(6, 96, 160, 12, 5, 201, dtype="f32", max_seg=60)
    run_and_check(sess, w, synth.make_tensors(w))


@pytest.mark.parametrize("rank", [8, 16, 32, 64, 128])
def test_rank_sweep(sess, rank):
    w = synth.random_workload(10 + rank, 320, 448, rank, 7, 300, max_seg=90)
    run_and_check(sess, w, synth.make_tensors(w))


@pytest.mark.parametrize("rank", [8, 16, 128])
def test_no_split_k(sess, rank):
    """The two-SM kernel without K slices on a small problem (kernel variant 4); the default splits it."""
    w = synth.random_workload(10 + rank, 320, 448, rank, 7, 300, max_seg=90)
    run_and_check(sess, w, synth.make_tensors(w), path=4)


@pytest.mark.parametrize("k", [8192, 8192 + 64 * 37, 16384])
def test_split_k_slices(sess, k):
    """Long contractions with few output tiles: 4 to 8 K slices (also a K that the slices do not divide evenly)."""
    segs = synth.segments_array([(0, 100, 0, 0), (100, 60, 1, 1), (160, 30, 2, 0), (190, 64, 0, 1)])
    w = synth.Workload("split_k", k, 256, 16, 3, "bf16", 254, segs, seed=k)
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)
    w2 = synth.Workload("split_k_bwd", 256, k, 16, 3, "bf16", 254, segs, seed=k + 1)      # long K in the backward GEMM
    run_and_check(sess, w2, synth.make_tensors(w2), blocked=True)


@pytest.mark.parametrize("d_in,d_out", [(8192, 4096), (4096, 8192)])
def test_k_split_of_the_last_wave_only(sess, d_in, d_out):
    """More output tiles than CTA pairs with a small last wave on a long contraction: 5 x 16 tiles of
    the forward (d_in = 8192) or of the input-gradient product (d_out = 8192) leave 6 tiles for the last
    wave, which are cut into 8 K slices while the other 74 run whole.  Checked against the blocked oracle;
    the variant without any K split must give the same numbers up to the rounding of the partial sums."""
    segs = synth.segments_array([(0, 1130, 0, 1), (1130, 70, 1, 0)])
    w = synth.Workload("tail_split", d_in, d_out, 16, 2, "bf16", 1200, segs, seed=d_in + 1)
    t = synth.make_tensors(w)
    run_and_check(sess, w, t, blocked=True)
    run_and_check(sess, w, t, path=4, blocked=True)


@pytest.mark.parametrize("rank", [32, 128])
def test_tensor_core_rank_r_kernels_are_bit_reproducible(sess, rank):
    """The tcgen05 shrink adds its runs in CTA order and the gradient kernel its pieces likewise: ten forward + backward
    passes over a batch whose blocks are shared by many CTAs (one adapter, long contraction) give the same bits."""
    segs = synth.segments_array([(0, 700, 0, 1), (700, 300, 1, 0), (1000, 500, 0, 1)])
    w = synth.Workload("repro_tc", 4096, 1024, rank, 2, "bf16", 1500, segs, seed=600 + rank)
    t = synth.make_tensors(w)
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows)
    try:
        first = None
        for it in range(10):
            for b in (run.Y, run.u_save, run.dA, run.dB, run.dX):
                b.zero_()
            run.forward(); run.backward()
            torch.cuda.synchronize()
            got = [b.clone() for b in (run.Y, run.u_save, run.dA, run.dB, run.dX)]
            if first is None:
                first = got
            else:
                for a, b in zip(first, got):
                    assert torch.equal(a, b), it
        assert run.status() == mb.MLORA_OK
    finally:
        run.close()


@pytest.mark.parametrize("rank", [64, 128])
def test_high_rank_large_batch(sess, rank):
    """8192 rows over 40 adapters at rank 64 / 128 (2048 -> 4096): the tcgen05 shrink with a few hundred blocks and runs
    shared by several CTAs, its finish kernel's zero rows, the operand images of ~30 gradient blocks, unit lists."""
    w = synth.random_workload(500 + rank, 2048, 4096, rank, 40, 8192, max_seg=300, p_decode=0.35, p_finetune=0.4)
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)


@pytest.mark.parametrize("rank", [32, 128])
def test_row_tiles_of_unequal_cost_get_balanced_unit_lists(sess, rank):
    """One 256-row tile of 200 single-row adapters between tiles of one group each: the heavy tile carries
    100 (rank 32) or 400 (rank 128) low-rank K-blocks against 8 main ones, so the units of the two-SM
    kernel are dealt out by cost from a list kept with the plan instead of round robin (5 x 20 tiles on
    74 pairs).  Same numbers as the oracle's, and bit for bit those of the round-robin variant (7): which
    pair computes a tile does not enter its arithmetic.  The second pass finds the list cached."""
    segs = [(0, 256, 0, 0)] + [(256 + i, 1, 1 + i, 0) for i in range(200)] + [(456, 56, 201, 0), (512, 300, 202, 1),
                                                                               (812, 212, 203, 1), (1024, 90, 3, 0)]
    w = synth.Workload("uneven_tiles", 512, 5120, rank, 204, "bf16", 1114, synth.segments_array(segs), seed=70 + rank)
    t = synth.make_tensors(w)
    outs = []
    for path in (0, 0, 7):
        run = None
        mb.mlora_set_gemm_path(sess.ctx, path)
        run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows)
        try:
            for _ in range(2):
                run.forward(); run.backward()
            assert run.status() == mb.MLORA_OK
            outs.append([b.clone() for b in (run.Y, run.dX, run.dA, run.dB)])
        finally:
            mb.mlora_set_gemm_path(sess.ctx, 0)
            run.close()
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    for a, b in zip(outs[0], outs[2]):
        assert torch.equal(a, b)
    run_and_check(sess, w, t, blocked=True)


@pytest.mark.parametrize("path", [0, 3])
@pytest.mark.parametrize("d_in,d_out", [(64, 128), (128, 64), (320, 448), (192, 320)])
def test_output_width_not_a_multiple_of_the_column_tile(sess, path, d_in, d_out):
    """Output widths that leave 1, 2 or 3 of the four 64-column chunks of the last column tile:
    the epilogue's two staging buffers alternate per chunk whether or not the chunk is stored, so
    a chunk past the edge must not overwrite a buffer whose store is still in flight.  Repeated on
    a warm context, since a slip here is a race (it showed as zeros in the last rows of a 32-row box)."""
    w = synth.random_workload(900 + d_in + d_out, d_in, d_out, 32, 20, 183, max_seg=60, p_finetune=0.9)
    t = synth.make_tensors(w)
    for _ in range(6):
        run_and_check(sess, w, t, path=path, blocked=True)


@pytest.mark.parametrize("seed", range(4))
def test_random_shapes_tables_and_kernel_variants(sess, seed):
    """Seeded random layer shapes, ranks, adapter counts, segment tables, save offsets and kernel
    variants on one warm context, each checked element by element (forward, saves, backward)."""
    rng = np.random.default_rng(7000 + seed)
    for it in range(10):
        d_in = int(rng.choice([64, 128, 192, 256, 320, 512, 576, 1024, 2048]))
        d_out = int(rng.choice([64, 128, 192, 256, 448, 512, 704, 1024, 4096]))
        rank = int(rng.choice([8, 16, 32, 64, 128]))
        w = synth.random_workload(7000 + 100 * seed + it, d_in, d_out, rank, int(rng.integers(1, 40)),
                                  int(rng.integers(1, 1200)), max_seg=int(rng.integers(1, 400)),
                                  p_decode=float(rng.uniform(0, 0.9)), p_finetune=float(rng.uniform(0, 0.7)))
        cap = None if rng.random() < 0.5 else int(w.ft_rows + 30)
        run_and_check(sess, w, synth.make_tensors(w), path=int(rng.choice([0, 0, 0, 2, 3, 4, 5, 6, 7])), blocked=True,
                      base=int(rng.integers(0, 3)) * 7, cap=cap)


@pytest.mark.parametrize("path", [5, 6])
@pytest.mark.parametrize("rank", [8, 16, 32, 64, 128])
def test_gradient_kernel_variants_rank_sweep(sess, rank, path):
    """Both gradient kernels on every rank: variant 5 = the mma.sync kernels (per-item kernel at rank 128), variant 6 =
    the tcgen05 gradient kernel (the default only at rank 128)."""
    w = synth.random_workload(60 + rank, 320, 448, rank, 7, 420, max_seg=150, p_finetune=0.5)
    run_and_check(sess, w, synth.make_tensors(w), path=path)


@pytest.mark.parametrize("lens", [(1100, 40), (2048,), (256,), (70, 700, 3)])
def test_tensor_core_gradient_kernel_on_split_strips(sess, lens):
    """The tcgen05 gradient kernel (kernel variant 6) where a slot's strips are shared by several CTAs: pieces summed by the
    last arrival in CTA order, slots of very different sizes, short last blocks, overwrite and accumulate, and the
    same bits from run to run."""
    segs, row = [(0, 37, 3, 0)], 37
    for a, n in enumerate(lens):
        segs.append((row, n, a, 1))
        row += n
    segs.append((row, 20, 0, 0))
    row += 20
    w = synth.Workload("few_slots_tc", 512, 1024, 16, 4, "bf16", row, synth.segments_array(segs), seed=400 + len(lens))
    t = synth.make_tensors(w)
    run_and_check(sess, w, t, blocked=True, path=6)
    mb.mlora_set_gemm_path(sess.ctx, 6)
    try:
        run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
        run.forward()
        outs = []
        for _ in range(3):
            run.backward(accumulate=False)
            outs.append((run.dA.clone(), run.dB.clone()))
        for dA, dB in outs[1:]:
            assert torch.equal(dA, outs[0][0]) and torch.equal(dB, outs[0][1])
        run.backward(accumulate=True, want_dx=False)
        assert_close("dA x2", run.host(run.dA), 2 * run.host(outs[0][0]), 1e-5)
        assert_close("dB x2", run.host(run.dB), 2 * run.host(outs[0][1]), 1e-5)
        assert run.status() == mb.MLORA_OK
        run.close()
    finally:
        mb.mlora_set_gemm_path(sess.ctx, 0)


def test_tensor_core_gradient_kernel_full_size(sess):
    """Kernel variant 6 on the widest projection of the layer set (plain ranges with shared strips at this size)."""
    w = synth.cfg3_layer_set(projections=["gate"])[0]
    run_and_check(sess, w, synth.make_tensors(w), blocked=True, path=6)


@pytest.mark.parametrize("rank", [8, 128])
def test_one_sm_gemm_kernel(sess, rank):
    """The one-SM tensor-core kernel (kernel variant 3) on ranks at both ends."""
    w = synth.random_workload(40 + rank, 320, 448, rank, 7, 300, max_seg=90)
    run_and_check(sess, w, synth.make_tensors(w), path=3)


@pytest.mark.parametrize("rank", [8, 32])
def test_every_row_its_own_adapter(sess, rank):
    """Decode-style tiles: up to 128 distinct adapters inside one 128-row tile."""
    n = 150
    ad = np.random.default_rng(1).permutation(n)
    segs = [(i, 1, int(ad[i]), 0) for i in range(n)] + [(n, 70, 3, 1)]
    w = synth.Workload("decode_tile", 256, 320, rank, n, "bf16", n + 70, synth.segments_array(segs))
    run_and_check(sess, w, synth.make_tensors(w))


@pytest.mark.parametrize("lens", [[0, 1, 127, 128, 129], [128, 128], [1], [300]])
def test_segment_lengths_around_a_tile(sess, lens):
    segs, row = [], 0
    for i, ln in enumerate(lens):
        segs.append((row, ln, i % 3, i % 2))
        row += ln
    w = synth.Workload("edges", 128, 256, 16, 3, "bf16", max(row, 1), synth.segments_array(segs))
    run_and_check(sess, w, synth.make_tensors(w))


@pytest.mark.parametrize("path", [0, 1, 2])
def test_finetune_slot_without_rows(sess, path):
    """A zero-length fine-tuning segment still opens a gradient slot: its dA / dB are written as zeros."""
    segs = [(0, 40, 0, 1), (40, 0, 2, 1), (40, 70, 1, 1), (110, 20, 2, 0)]
    w = synth.Workload("empty_slot", 256, 192, 16, 3, "bf16", 130, synth.segments_array(segs))
    run = run_and_check(sess, w, synth.make_tensors(w), path=path)
    assert run.slots == [0, 2, 1]
    assert not run.host(run.dA)[1].any() and not run.host(run.dB)[1].any()


@pytest.mark.parametrize("n_rows", [5, 129, 257])
def test_small_batches(sess, n_rows):
    """Fewer rows than one tile, and batches that leave the second CTA of a pair tile (almost) empty."""
    segs = [(0, n_rows // 2, 1, 0), (n_rows // 2, n_rows - n_rows // 2, 0, 1)]
    w = synth.Workload("small", 192, 320, 16, 2, "bf16", n_rows, synth.segments_array(segs))
    run_and_check(sess, w, synth.make_tensors(w))


def test_gathered_and_contiguous_items(sess):
    """Rows of one adapter scattered between other rows (gathered shrink items) next to long
    contiguous segments, with base-only rows inside tiles that have adapters."""
    segs, row = [], 0
    for i in range(60):                              # decode-style rows cycling over 5 adapters, some without adapter
        segs.append((row, 1, (i % 6) - 1, 0))
        row += 1
    segs.append((row, 150, 2, 1)); row += 150        # fine-tune segment
    row += 7                                         # uncovered rows
    segs.append((row, 90, 4, 0)); row += 90
    for i in range(40):
        segs.append((row, 1, i % 5, 0))
        row += 1
    w = synth.Workload("mixed_items", 2048, 320, 16, 5, "bf16", row, synth.segments_array(segs))
    run_and_check(sess, w, synth.make_tensors(w))


def test_block_save_only_when_save_offsets_run_with_the_rows(sess):
    """Full 32-row items of fine-tuning rows are saved as one block only when their save offsets are
    consecutive.  Here adjacent fine-tuning segments of ONE adapter sit in the table out of row order,
    so 32 adjacent rows map to permuted / interleaved save offsets; next to them a segment whose
    items can be block-saved, a mixed inference + fine-tune item, and a partial item."""
    segs = [(0, 8, 0, 1), (16, 8, 0, 1), (8, 8, 0, 1), (24, 8, 0, 1),        # rows 0..31 adjacent, saves 0-7,16-23,8-15,24-31
            (64, 32, 1, 1), (32, 32, 1, 1),                                   # two full items, second saved first
            (96, 96, 2, 1),                                                   # three block-saved items
            (192, 10, 3, 0), (202, 54, 3, 1),                                 # item mixing inference and fine-tune rows
            (256, 45, 0, 1)]                                                  # full item + partial item, adapter 0 again
    for path in (0, 2):
        w = synth.Workload("block_save_order", 768, 256, 16, 4, "bf16", 301, synth.segments_array(segs), seed=path)
        run_and_check(sess, w, synth.make_tensors(w), path=path, base=5, cap=5 + 291 + 9)


def test_stream_ordered_plans_from_the_pool(sess):
    """Plans created and released on a stream, step after step (buffers come back from the pool while
    earlier steps may still be running): every step's outputs equal those of an ordinary plan."""
    w0 = synth.random_workload(90, 256, 320, 16, 5, 600, max_seg=100, p_finetune=0.3)
    t = synth.make_tensors(w0)
    run = LayerRun(sess, "bf16", t, w0.segments, w0.n_rows, save_capacity_rows=700)
    outs, tables = [], []
    try:
        for step in range(12):
            w = synth.random_workload(100 + step, 256, 320, 16, 5, 200 + 31 * step, max_seg=60 + 5 * step, p_finetune=0.3)
            plan = mb.mlora_plan_create_async(sess.ctx, w.segments, w.n_rows, 5)
            y = torch.zeros((w.n_rows, 320), dtype=torch.bfloat16, device=sess.device)
            mb.mlora_mixed_forward(sess.ctx, run.layer, plan, run.X, y, run.x_save, run.u_save, 0, run.capacity)
            mb.mlora_plan_release(plan)
            outs.append(y)
            tables.append(w)
        torch.cuda.synchronize()
        assert run.status() == mb.MLORA_OK
        for y, w in zip(outs, tables):
            plan = mb.mlora_plan_create(sess.ctx, w.segments, w.n_rows, 5)
            y2 = torch.zeros_like(y)
            mb.mlora_mixed_forward(sess.ctx, run.layer, plan, run.X, y2, run.x_save, run.u_save, 0, run.capacity)
            torch.cuda.synchronize()
            mb.mlora_plan_destroy(plan)
            assert torch.equal(y, y2)
        ref = orc.forward(t["X"][:tables[3].n_rows], t["W"], t["A_all"], t["B_all"], t["scale"], tables[3].segments)
        assert_close("Y", run.host(outs[3]), ref["Y"], TOL["bf16"])
        # a pooled plan may also be destroyed the ordinary way
        plan = mb.mlora_plan_create_async(sess.ctx, w0.segments, w0.n_rows, 5)
        mb.mlora_plan_destroy(plan)
        # stream-ordered plans with per-adapter ranks (all 16 here, the layer's own): the same bits as the plain plan's
        w = tables[5]
        plan = mb.mlora_plan_create_ranked_async(sess.ctx, w.segments, w.n_rows, 5, [16] * 5)
        y3 = torch.zeros_like(outs[5])
        mb.mlora_mixed_forward(sess.ctx, run.layer, plan, run.X, y3, run.x_save, run.u_save, 0, run.capacity)
        mb.mlora_plan_release(plan)
        torch.cuda.synchronize()
        assert torch.equal(y3, outs[5])
    finally:
        run.close()


def test_blocking_plans_reuse_the_pool(sess):
    """mlora_plan_create / mlora_plan_destroy take their buffer pair from the context's pool and give it back: three
    hundred plans of mixed sizes later the device holds no more memory than after the first few, and a plan made
    this way computes what the oracle says."""
    tables = [synth.random_workload(90 + i, 128, 128, 16, 6, 100 + 700 * i, max_seg=50 + 40 * i) for i in range(4)]
    for w in tables:
        mb.mlora_plan_destroy(mb.mlora_plan_create(sess.ctx, w.segments, w.n_rows, w.n_adapters))
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for i in range(300):
        w = tables[i % 4]
        mb.mlora_plan_destroy(mb.mlora_plan_create(sess.ctx, w.segments, w.n_rows, w.n_adapters))
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < (8 << 20), (free0, free1)
    run_and_check(sess, tables[1], synth.make_tensors(tables[1]))


def test_many_rows_many_adapters(sess):
    """16384 rows (64 pair tiles), 96 adapters, 5000 fine-tuning rows in ragged segments: the workspaces grow,
    tables and counters stay in range."""
    w = synth.random_workload(123, 1024, 768, 16, 96, 16384, max_seg=700, p_finetune=0.3)
    assert w.ft_rows > 3000
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)


@pytest.mark.parametrize("rows,d_in,d_out,rank,n_ad,kw", [
    (70000, 512, 1024, 128, 32, dict(max_seg=5000, p_decode=0.1, p_finetune=0.6)),
    (50000, 1024, 512, 32, 500, dict(max_seg=40, p_decode=0.8, p_finetune=0.3)),
])
def test_batches_beyond_the_tensor_core_rank_r_kernels_limits(sess, rows, d_in, d_out, rank, n_ad, kw):
    """Tens of thousands of rows: 39616 fine-tuning rows at rank 128 (more 128-row blocks than the operand
    workspace of the tcgen05 gradient kernel holds), and 8762 segments over 500 adapters (unit lists, item tables
    and partial-sum workspaces at their largest).  Every element against the oracle."""
    w = synth.random_workload(7, d_in, d_out, rank, n_ad, rows, **kw)
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)


def test_base_only_rows_and_no_finetune(sess):
    segs = [(0, 40, -1, 0), (60, 30, 1, 0)]      # rows 40..59 and 90..99 uncovered
    w = synth.Workload("base_only", 192, 256, 16, 2, "bf16", 100, synth.segments_array(segs))
    t = synth.make_tensors(w)
    run = run_and_check(sess, w, t)
    assert run.ft_rows == 0
    w2 = synth.Workload("no_segments", 192, 256, 16, 2, "bf16", 100, np.zeros((0, 4), np.int32))
    run_and_check(sess, w2, synth.make_tensors(w2))


def test_empty_batch_is_a_no_op(sess):
    plan = mb.mlora_plan_create(sess.ctx, np.zeros((0, 4), np.int32), 0, 2)
    w = synth.Workload("x", 64, 64, 8, 2, "bf16", 4, synth.segments_array([(0, 4, 0, 0)]))
    run = LayerRun(sess, "bf16", synth.make_tensors(w), w.segments, 4)
    mb.mlora_mixed_forward(sess.ctx, run.layer, plan, None, None, None, None, 0, 0)
    mb.mlora_backward(sess.ctx, run.layer, plan, None, None, None, None, None, None)
    assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_OK
    mb.mlora_plan_destroy(plan)
    run.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_integer_probe_bit_exact(sess, dtype):
    p = integer_probe(n_rows=333, d_in=128, d_out=192, rank=16, n_adapters=9, seed=4, dtype=dtype)
    w = synth.Workload("probe", 128, 192, 16, 9, dtype, 333, p["segments"])
    fwd = orc.forward(p["X"], p["W"], p["A_all"], p["B_all"], p["scale"], p["segments"])
    run = LayerRun(sess, dtype, p, p["segments"], 333, guard=True)
    try:
        run.forward()
        assert run.status() == mb.MLORA_OK
        n = run.ft_rows
        assert np.array_equal(run.host(run.Y), fwd["Y"])
        assert np.array_equal(run.host(run.x_save)[:n], fwd["x_save"])
        assert np.array_equal(run.host(run.u_save)[:n], fwd["u_save"])
        run.backward()
        bwd = orc.backward(p["dY"], p["W"], p["A_all"], p["B_all"], p["scale"], p["segments"], fwd["x_save"],
                           fwd["u_save"], n_rows=333)
        assert np.array_equal(run.host(run.dX)[:n], bwd["dX"])
        assert np.array_equal(run.host(run.dA), bwd["dA"])
        assert np.array_equal(run.host(run.dB), bwd["dB"])
    finally:
        run.close()


@pytest.mark.parametrize("path", [0, 6])
@pytest.mark.parametrize("seed", range(8))
def test_random_tables_route_bit_exactly(sess, seed, path):
    """Random valid segment tables (ragged lengths, single rows, gaps, adapter -1, shuffled order,
    several fine-tune segments per adapter) on the exact-integer probe: every output must equal the
    oracle bit for bit, so any mis-routed row, wrong scale or mis-indexed save row shows.  Under kernel
    variant 6 every rank-r product runs on the tcgen05 kernels (blocks, run sums, operand images)."""
    rng = np.random.default_rng(seed)
    n_rows = int(rng.integers(1, 700))
    n_adapters = int(rng.integers(1, 40))
    rank = int(rng.choice([8, 16, 32, 64, 128]))
    d_in, d_out = int(rng.choice([64, 128, 192])), int(rng.choice([64, 256, 320]))
    p = integer_probe(n_rows=n_rows, d_in=d_in, d_out=d_out, rank=rank, n_adapters=n_adapters, seed=100 + seed,
                      max_seg=int(rng.integers(2, 300)))
    fwd = orc.forward(p["X"], p["W"], p["A_all"], p["B_all"], p["scale"], p["segments"])
    mb.mlora_set_gemm_path(sess.ctx, path)
    run = LayerRun(sess, "bf16", p, p["segments"], n_rows, guard=True)
    try:
        run.forward()
        assert run.status() == mb.MLORA_OK
        n = run.ft_rows
        assert n == fwd["ft_rows"] and run.slots == fwd["ft_adapters"]
        assert np.array_equal(run.host(run.Y), fwd["Y"])
        assert np.array_equal(run.host(run.x_save)[:n], fwd["x_save"])
        assert np.array_equal(run.host(run.u_save)[:n], fwd["u_save"])
        if n:
            run.backward()
            bwd = orc.backward(p["dY"], p["W"], p["A_all"], p["B_all"], p["scale"], p["segments"], fwd["x_save"],
                               fwd["u_save"], n_rows=n_rows)
            assert np.array_equal(run.host(run.dX)[:n], bwd["dX"])
            assert np.array_equal(run.host(run.dA), bwd["dA"])
            assert np.array_equal(run.host(run.dB), bwd["dB"])
    finally:
        mb.mlora_set_gemm_path(sess.ctx, 0)
        run.close()


def test_append_two_steps_then_one_backward(sess):
    """Two forward steps append into one activation buffer; one backward consumes both
    (activations accumulate until a backward batch is full)."""
    d_in, d_out, r, n_ad = 128, 192, 16, 4
    w1 = synth.Workload("s1", d_in, d_out, r, n_ad, "bf16", 90, synth.segments_array([(0, 50, 0, 0), (50, 40, 2, 1)]))
    w2 = synth.Workload("s2", d_in, d_out, r, n_ad, "bf16", 70, synth.segments_array([(0, 30, 3, 1), (30, 40, 1, 0)]),
                        tag_base=50)
    t1, t2 = synth.make_tensors(w1), synth.make_tensors(w2)
    t2["W"], t2["A_all"], t2["B_all"] = t1["W"], t1["A_all"], t1["B_all"]
    cap = 70
    r1 = LayerRun(sess, "bf16", t1, w1.segments, 90, save_row_base=0, save_capacity_rows=cap)
    r2 = LayerRun(sess, "bf16", t2, w2.segments, 70, save_row_base=40, save_capacity_rows=cap)
    r2.x_save, r2.u_save = r1.x_save, r1.u_save          # one shared activation buffer
    r1.forward()
    r2.forward()
    # backward over all 70 saved rows: a fine-tune-only table in save order
    segs_b = synth.segments_array([(0, 40, 2, 1), (40, 30, 3, 1)])
    dY = np.concatenate([t1["dY"], t2["dY"]])
    tb = dict(t1, X=np.zeros((70, d_in), np.float32), dY=dY)
    rb = LayerRun(sess, "bf16", tb, segs_b, 70)
    rb.x_save, rb.u_save = r1.x_save, r1.u_save
    rb.backward()
    assert rb.status() == mb.MLORA_OK
    f1 = orc.forward(t1["X"], t1["W"], t1["A_all"], t1["B_all"], t1["scale"], w1.segments)
    f2 = orc.forward(t2["X"], t1["W"], t1["A_all"], t1["B_all"], t1["scale"], w2.segments)
    xs = np.concatenate([f1["x_save"], f2["x_save"]])
    us = np.concatenate([f1["u_save"], f2["u_save"]])
    assert np.array_equal(rb.host(r1.x_save)[:70], xs)
    ref = orc.backward(dY, t1["W"], t1["A_all"], t1["B_all"], t1["scale"], segs_b, xs, us, n_rows=70)
    assert rb.slots == ref["ft_adapters"] == [2, 3]
    assert_close("dA", rb.host(rb.dA), ref["dA"], 2e-2)
    assert_close("dB", rb.host(rb.dB), ref["dB"], 2e-2)
    assert_close("dX", rb.host(rb.dX), ref["dX"], 2e-2)
    # the buffer is full now: one more fine-tuning row must be refused before anything runs
    with pytest.raises(mb.MloraError) as e:
        mb.mlora_mixed_forward(sess.ctx, r2.layer, r2.plan, r2.X, r2.Y, r1.x_save, r1.u_save, 41, cap)
    assert e.value.status == mb.MLORA_ERR_SAVE_CAPACITY
    for r_ in (r1, r2, rb):
        r_.close()


def test_accumulate_and_optional_outputs(sess):
    w = synth.random_workload(21, 128, 192, 16, 4, 260, max_seg=80, p_finetune=0.5)
    t = synth.make_tensors(w)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows, save_x=True)
    run.forward()
    run.backward(accumulate=False)
    dA1, dB1 = run.host(run.dA), run.host(run.dB)
    run.backward(accumulate=True, want_dx=False)
    assert_close("dA x2", run.host(run.dA), 2 * dA1, 1e-5)
    assert_close("dB x2", run.host(run.dB), 2 * dB1, 1e-5)
    # x_save = NULL skips the copy but still produces Y and u_save
    run2 = LayerRun(sess, "bf16", t, w.segments, w.n_rows, save_x=False)
    run2.forward()
    assert torch.equal(run2.Y, run.Y) and torch.equal(run2.u_save, run.u_save)
    run.close()
    run2.close()


@pytest.mark.parametrize("rank", [8, 16, 32, 64])
@pytest.mark.parametrize("lens", [(1100, 40), (2048,), (256,), (70, 700, 3)])
def test_gradient_groups_split_over_rows(sess, rank, lens):
    """One to three fine-tuning adapters leave the gradient kernel fewer (slot, strip) groups than
    half the SMs: the row blocks of a slot are then dealt out over several CTAs per group and the
    last one to arrive adds the partial sums in index order.  Slots of very different sizes (parts
    without any block), overwrite and accumulate, and bit-identical results from run to run."""
    segs, row = [(0, 37, 3, 0)], 37
    for a, n in enumerate(lens):
        segs.append((row, n, a, 1))
        row += n
    segs.append((row, 20, 0, 0))
    row += 20
    w = synth.Workload("few_slots", 512, 1024, rank, 4, "bf16", row, synth.segments_array(segs), seed=300 + rank)
    t = synth.make_tensors(w)
    run = run_and_check(sess, w, t, blocked=True)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    run.forward()
    outs = []
    for _ in range(3):
        run.backward(accumulate=False)
        outs.append((run.dA.clone(), run.dB.clone()))
    for dA, dB in outs[1:]:
        assert torch.equal(dA, outs[0][0]) and torch.equal(dB, outs[0][1])
    run.backward(accumulate=True, want_dx=False)
    assert_close("dA x2", run.host(run.dA), 2 * run.host(outs[0][0]), 1e-5)
    assert_close("dB x2", run.host(run.dB), 2 * run.host(outs[0][1]), 1e-5)
    assert run.status() == mb.MLORA_OK
    run.close()


def test_strided_inputs_and_outputs(sess):
    w = synth.random_workload(22, 128, 256, 16, 3, 200, max_seg=70)
    t = synth.make_tensors(w)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    big_x = torch.zeros((w.n_rows, 128 + 64), dtype=torch.bfloat16, device=sess.device)
    big_x[:, 64:] = run.X
    big_y = torch.full((w.n_rows, 256 + 128), 7.0, dtype=torch.bfloat16, device=sess.device)
    run.forward()
    y_ref = run.Y.clone()
    run.X, run.Y = big_x[:, 64:], big_y[:, 128:]
    run.forward()
    assert torch.equal(run.Y, y_ref)
    assert (big_y[:, :128] == 7.0).all()
    run.close()


@pytest.mark.parametrize("rank,path", [(8, 0), (16, 2), (32, 0), (64, 0), (128, 0), (16, 6)])
def test_row_strides_on_every_operand(sess, rank, path):
    """X, Y, dY and dX as column slices of wider buffers (row strides 8 to 200 elements beyond the width): the same bits
    as with packed operands on every kernel family (streaming, per-item, tcgen05 rank-r kernels), nothing written outside."""
    w = synth.random_workload(500 + rank, 512, 448, rank, 6, 700, max_seg=150, p_decode=0.3, p_finetune=0.5)
    t = synth.make_tensors(w)
    mb.mlora_set_gemm_path(sess.ctx, path)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    try:
        run.forward(); run.backward()
        ref = [x.clone() for x in (run.Y, run.u_save, run.x_save, run.dA, run.dB, run.dX)]
        dev, n = sess.device, run.ft_rows
        bx = torch.full((w.n_rows, 512 + 24), 3.0, dtype=torch.bfloat16, device=dev); bx[:, 24:] = run.X
        by = torch.full((w.n_rows, 448 + 200), 7.0, dtype=torch.bfloat16, device=dev)
        bdy = torch.full((run.dY.shape[0], 448 + 8), 5.0, dtype=torch.bfloat16, device=dev); bdy[:, :448] = run.dY
        bdx = torch.full((run.dX.shape[0], 512 + 64), 9.0, dtype=torch.bfloat16, device=dev)
        run.X, run.Y, run.dY, run.dX = bx[:, 24:], by[:, :448], bdy[:, :448], bdx[:, 64:]
        run.u_save.fill_(float("nan")); run.x_save.fill_(float("nan")); run.dA.fill_(float("nan")); run.dB.fill_(float("nan"))
        run.forward(); run.backward()
        assert run.status() == mb.MLORA_OK
        got = (run.Y, run.u_save, run.x_save, run.dA, run.dB, run.dX)
        for i, (g, r) in enumerate(zip(got, ref)):
            assert torch.equal(g[:n], r[:n]) if i in (1, 2, 5) else torch.equal(g, r), i
        assert (by[:, 448:] == 7.0).all() and (bdx[:, :64] == 9.0).all()
    finally:
        mb.mlora_set_gemm_path(sess.ctx, 0)
        run.close()


def test_run_to_run_determinism(sess):
    w = synth.random_workload(23, 256, 320, 32, 5, 500, max_seg=120, p_finetune=0.5)
    t = synth.make_tensors(w)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    outs = []
    for _ in range(2):
        run.forward()
        run.backward()
        outs.append([x.clone() for x in (run.Y, run.u_save, run.dA, run.dB, run.dX)])
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    run.close()


def test_argument_errors_launch_nothing(sess):
    w = synth.random_workload(24, 128, 128, 16, 3, 64, max_seg=20, p_finetune=0.6)
    t = synth.make_tensors(w)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    before = mb.mlora_launch_count(sess.ctx)
    with pytest.raises(mb.MloraError) as e:                     # capacity too small
        mb.mlora_mixed_forward(sess.ctx, run.layer, run.plan, run.X, run.Y, run.x_save, run.u_save, 0, run.ft_rows - 1)
    assert e.value.status == mb.MLORA_ERR_SAVE_CAPACITY
    with pytest.raises(mb.MloraError) as e:                     # u_save missing
        mb.mlora_mixed_forward(sess.ctx, run.layer, run.plan, run.X, run.Y, run.x_save, None, 0, 1000)
    assert e.value.status == mb.MLORA_ERR_INVALID_ARG
    few = mb.make_layer(run.W, run.A_all[:2].contiguous(), run.B_all[:2].contiguous(), run.scale[:2].contiguous())
    with pytest.raises(mb.MloraError) as e:                     # plan built for more adapters than the layer has
        mb.mlora_mixed_forward(sess.ctx, few, run.plan, run.X, run.Y, run.x_save, run.u_save, 0, 1000)
    assert e.value.status == mb.MLORA_ERR_ADAPTER_ID
    odd = mb.make_layer(run.W, run.A_all, run.B_all, run.scale)
    odd.rank = 24
    with pytest.raises(mb.MloraError) as e:
        mb.mlora_mixed_forward(sess.ctx, odd, run.plan, run.X, run.Y, run.x_save, run.u_save, 0, 1000)
    assert e.value.status == mb.MLORA_ERR_UNSUPPORTED
    assert mb.mlora_launch_count(sess.ctx) == before
    run.close()


def test_cancel_flag_stops_between_kernels(sess):
    """The caller's host flag is read before every launch: once raised, a call launches nothing
    more and reports MLORA_CANCELLED; once lowered, the same step runs normally (the interrupted
    step is simply repeated, its partial activations overwritten)."""
    import ctypes
    w = synth.random_workload(25, 128, 192, 16, 3, 200, max_seg=60, p_finetune=0.5)
    t = synth.make_tensors(w)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    run.forward()
    run.backward()
    ref = [x.clone() for x in (run.Y, run.u_save, run.dA, run.dB, run.dX)]
    flag = ctypes.c_int32(0)
    mb.mlora_set_cancel_flag(sess.ctx, flag)
    try:
        flag.value = 1
        before = mb.mlora_launch_count(sess.ctx)
        for call in (run.forward, run.backward):
            with pytest.raises(mb.MloraError) as e:
                call()
            assert e.value.status == mb.MLORA_CANCELLED
        assert mb.mlora_launch_count(sess.ctx) == before
        flag.value = 0
        run.Y.zero_()
        run.forward()
        run.backward()
        for a, b in zip(ref, (run.Y, run.u_save, run.dA, run.dB, run.dX)):
            assert torch.equal(a, b)
    finally:
        mb.mlora_set_cancel_flag(sess.ctx, None)
    run.close()


def test_bounded_wait_runs_out_and_is_reported(sess):
    """A wait inside a kernel that can never be satisfied gives up after its poll limit, the kernel returns,
    and the status word carries MLORA_ERR_DEVICE_TIMEOUT until it is polled; the poll clears it (and the
    arrival counters), and the same forward + backward before and after are bit-identical.  Nothing faults
    or hangs: the kernel is the library's own self-test, one warp waiting 1024 polls on a barrier nobody
    arrives at."""
    segs = synth.segments_array([(0, 37, 3, 0), (37, 2048, 0, 1), (2085, 20, 1, 0)])     # one slot: row-split gradient groups
    w = synth.Workload("timeout_probe", 2048, 512, 16, 4, "bf16", 2105, segs, seed=77)
    t = synth.make_tensors(w)
    run = LayerRun(sess, "bf16", t, w.segments, w.n_rows)
    run.forward(); run.backward()
    before = [x.clone() for x in (run.Y, run.u_save, run.dA, run.dB, run.dX)]
    assert run.status() == mb.MLORA_OK
    mb.mlora_selftest_timeout(sess.ctx, 1024)
    assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_ERR_DEVICE_TIMEOUT
    assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_OK
    for b in (run.Y, run.u_save, run.dA, run.dB, run.dX):
        b.zero_()
    run.forward(); run.backward()
    assert run.status() == mb.MLORA_OK
    for a, b in zip(before, (run.Y, run.u_save, run.dA, run.dB, run.dX)):
        assert torch.equal(a, b)
    run.close()


# ---- full-size configurations: every element of every output against the oracle --------------------
def test_cfg2_full_size(sess):
    w = synth.cfg2_single_projection()
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)


@pytest.mark.parametrize("proj", ["q", "k", "v", "o", "gate", "up", "down"])
def test_cfg3_projection_full_size(sess, proj):
    """The benchmark's launch configuration (banded tile order and the K split of the last wave included):
    Y, the saved rows, u_save, dX, dA and dB element by element against oracle.forward_blocked /
    oracle.backward_blocked."""
    w = synth.cfg3_layer_set(projections=[proj])[0]
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)


@pytest.mark.parametrize("mode", ["decode", "finetune", "mixed"])
def test_cfg5_decode_heavy_full_size(sess, mode):
    """The three runs the decode-heavy configuration reports: decode rows only, the fine-tuning segment
    only, and both in one batch."""
    w = synth.cfg5_decode_heavy(mode=mode)
    run_and_check(sess, w, synth.make_tensors(w), blocked=True)


_CFG4_CACHE = {}


def _cfg4_tensors(w):
    """synth.make_tensors for a sweep point, keeping the tensors that do not change from point to point
    (X and W always, the adapters per (rank, adapter count)): every tensor is a pure function of
    (seed, tag, shape), so the cached arrays are exactly what make_tensors would draw again."""
    def draw(key, tag, shape, std):
        if key not in _CFG4_CACHE:
            n = int(np.prod(shape))
            _CFG4_CACHE[key] = synth.round_to_storage(synth.normal(w.seed, w.tag_base + tag, n, std=std).reshape(shape), w.dtype)
        return _CFG4_CACHE[key]
    for k in [k for k in _CFG4_CACHE if k[0] in ("A", "B") and k[1:] != (w.rank, w.n_adapters)]:
        del _CFG4_CACHE[k]                           # one adapter set at a time (the largest is 2.4 GB)
    t = {"X": draw(("X",), 1, (w.n_rows, w.d_in), 1.0), "W": draw(("W",), 2, (w.d_in, w.d_out), w.d_in ** -0.5),
         "A_all": draw(("A", w.rank, w.n_adapters), 3, (w.n_adapters, w.rank, w.d_in), 0.02),
         "B_all": draw(("B", w.rank, w.n_adapters), 4, (w.n_adapters, w.rank, w.d_out), 0.02),
         "scale": np.full(w.n_adapters, w.lora_scale, dtype=np.float32)}
    n = w.ft_rows
    t["dY"] = synth.round_to_storage(synth.normal(w.seed, w.tag_base + 5, n * w.d_out).reshape(n, w.d_out), w.dtype)
    return t


def test_cfg4_cached_tensors_are_the_generator_s(sess):
    w = synth.cfg4_sweep_point(8, 1, 0.5)
    a, b = _cfg4_tensors(w), synth.make_tensors(w)
    assert all(np.array_equal(a[k], b[k]) for k in b)


CFG4_GRID = [(r, n, f, True) for r in (8, 16, 32, 64, 128) for n in (1, 256) for f in (0.0, 0.5)] + [(16, 64, 0.25, False)]


@pytest.mark.parametrize("rank,n_adapters,f,sorted_rows", CFG4_GRID)
def test_cfg4_sweep_grid_full_size(sess, rank, n_adapters, f, sorted_rows):
    """Every rank x {1, 256} adapters x fine-tune fraction {0, 0.5} of the sweep on 4096 -> 14336, plus one
    point with unsorted rows (every row its own segment), each compared element by element."""
    w = synth.cfg4_sweep_point(rank, n_adapters, f, sorted_rows=sorted_rows)
    run_and_check(sess, w, _cfg4_tensors(w), blocked=True)


def test_two_contexts_on_two_host_threads():
    """Contexts are independent across host threads (the per-device caches of one-time kernel attributes are shared and
    locked): two threads, each with its own context, stream and plans, run different ranks at the same time on the same
    device; each checks its own results against the oracle."""
    import threading
    errors = []

    def worker(seed, rank):
        try:
            stream = torch.cuda.Stream(device=torch.device("cuda", 0))
            with torch.cuda.stream(stream):
                with Session(0) as s2:
                    for it in range(3):
                        w = synth.random_workload(seed + it, 256, 384, rank, 5, 500, max_seg=120, p_finetune=0.4)
                        run_and_check(s2, w, synth.make_tensors(w))
        except Exception as e:          # noqa: BLE001 - reported below, in the main thread
            errors.append((seed, rank, repr(e)))

    threads = [threading.Thread(target=worker, args=(910, 16)), threading.Thread(target=worker, args=(920, 64))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
