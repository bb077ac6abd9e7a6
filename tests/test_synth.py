"""The seeded input generators: determinism, storage rounding, and the shapes of the five configs."""
import numpy as np
import torch

from paper_2607_28848_b200 import synth


def test_counter_based_streams_are_reproducible_and_piecewise():
    a = synth.normal(0, 7, 1000)
    b = synth.normal(0, 7, 1000)
    assert np.array_equal(a, b)
    whole = synth.uniform01(3, 9, 0, 100)
    assert np.array_equal(whole[40:60], synth.uniform01(3, 9, 40, 20))
    assert not np.array_equal(synth.normal(0, 7, 100), synth.normal(1, 7, 100))
    assert not np.array_equal(synth.normal(0, 7, 100), synth.normal(0, 8, 100))


def test_normal_moments():
    x = synth.normal(0, 1, 400000, std=0.5)
    assert abs(x.mean()) < 5e-3
    assert abs(x.std() - 0.5) < 5e-3


def test_bf16_rounding_matches_torch():
    x = synth.normal(0, 2, 20000).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -3.0e-39, 65504.0]     # ties and a subnormal
    ours = synth.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours, ref)


def _check_table(w):
    seg = w.segments
    assert seg.dtype == np.int32 and seg.shape[1] == 4
    covered = np.zeros(w.n_rows, dtype=int)
    for st, ln, ad, ft in seg.tolist():
        assert 0 <= st and st + ln <= w.n_rows and -1 <= ad < w.n_adapters
        covered[st:st + ln] += 1
    assert covered.max() <= 1


def test_config_shapes():
    c1 = synth.cfg1_tiny()
    assert (c1.d_in, c1.d_out, c1.rank, c1.n_adapters, c1.n_rows, c1.ft_rows, c1.dtype) == (256, 256, 8, 4, 64, 16, "f32")
    c2 = synth.cfg2_single_projection()
    assert (c2.n_rows, c2.ft_rows, len(c2.segments)) == (1600, 512, 8 + 64 + 2)
    c3 = synth.cfg3_layer_set()
    assert [w.name for w in c3] == ["cfg3_q", "cfg3_k", "cfg3_v", "cfg3_o", "cfg3_gate", "cfg3_up", "cfg3_down"]
    assert all(w.n_rows == 4096 and w.ft_rows == 2048 and len(w.segments) == 12 + 1024 + 4 for w in c3)
    assert (c3[4].d_in, c3[4].d_out, c3[6].d_in, c3[6].d_out, c3[1].d_out) == (4096, 14336, 14336, 4096, 1024)
    c5 = synth.cfg5_decode_heavy()
    assert (c5.n_rows, c5.ft_rows, c5.rank, c5.n_adapters) == (2560, 2048, 32, 128)
    assert synth.cfg5_decode_heavy(mode="decode").n_rows == 512
    for w in [c1, c2, c5] + c3:
        _check_table(w)


def test_cfg4_sweep_points():
    for r in (8, 128):
        for n in (1, 8, 64, 256):
            for f in (0.0, 0.25, 0.5, 0.75):
                w = synth.cfg4_sweep_point(r, n, f)
                assert w.n_rows == 2048 and w.ft_rows == int(2048 * f)
                _check_table(w)
    w = synth.cfg4_sweep_point(16, 64, 0.25, sorted_rows=False)
    assert len(w.segments) == 1536 + 2
    z = synth.zipf_adapters(0, 401, 200000, 8)
    share = np.bincount(z, minlength=8) / len(z)
    assert abs(share[0] - 0.40) < 0.01          # top adapter's share for Zipf(1.1) over 8 adapters


def test_make_tensors_layouts_and_storage():
    w = synth.random_workload(1, 24, 40, 8, 3, 50)
    t = synth.make_tensors(w)
    assert t["X"].shape == (50, 24) and t["W"].shape == (24, 40)
    assert t["A_all"].shape == (3, 8, 24) and t["B_all"].shape == (3, 8, 40)
    assert t["dY"].shape == (w.ft_rows, 40)
    for k in ("X", "W", "A_all", "B_all", "dY"):
        assert np.array_equal(t[k], synth.round_to_bf16(t[k]))       # already bf16 values
    _check_table(w)
