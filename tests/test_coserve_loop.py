"""The co-serving loop's host logic against a recording executor (no GPU): every admitted sample is
forwarded once and trained once, the activation buffer is never overcommitted, the backward table
lists the saved rows in save order, the backward yields to steps with prompts, and an interrupted
forward returns its samples."""
import numpy as np

from oracle import mlora_oracle as orc
from paper_2607_28848_b200 import sched as ms
from paper_2607_28848_b200.coserve import CoServeLoop, synthetic_arrivals


class RecordingExecutor:
    def __init__(self, buffer_tokens):
        self.cap = buffer_tokens
        self.saved = 0
        self.forwards, self.backwards, self.updates = [], [], 0

    def forward(self, table, n_rows, save_base, cancel=False):
        if cancel:
            return False
        _, ft_segments, ft_rows, _ = orc.route(table, n_rows, 8)      # the table is valid for the layer
        assert save_base == self.saved and save_base + ft_rows <= self.cap
        self.saved += ft_rows
        self.forwards.append((table.copy(), n_rows, save_base))
        return True

    def backward(self, table, n_rows):
        _, ft_segments, ft_rows, _ = orc.route(table, n_rows, 8)
        assert ft_rows == n_rows == self.saved                        # exactly the saved rows, compact
        assert [off for *_x, off in ft_segments] == sorted(off for *_x, off in ft_segments)
        self.backwards.append(table.copy())
        self.saved = 0

    def update(self, table, n_rows):
        self.updates += 1


def make_sched(buf, per_token=1e-3, slo=1.0, tpot=1.0):
    c = ms.mixed_coef(0.0, per_token, 0.0, 0.0, 0.01)
    return ms.mlora_sched_create(c, c, ms.decode_coef(), slo, tpot, buf)


def test_loop_trains_every_admitted_sample_once():
    buf = 1024
    s = make_sched(buf)
    ex = RecordingExecutor(buf)
    loop = CoServeLoop(ex, s, 8, ft_adapter_of=lambda sid: sid % 3, backward_batch=256)
    try:
        for i in range(40):
            ms.mlora_sched_pool_add(s, i, 64 + 32 * (i % 5))
        admitted = []
        for prefill, dec, kv in synthetic_arrivals(120, 3, 8):
            lens = [n for n, _ in prefill]
            out = loop.step(prefill, dec, kv, t_now=0.2, earliest_arrival=0.0 if lens else None)
            admitted += out["admitted"]
            assert out["ft_tokens"] <= buf and loop.saved_tokens <= buf
            assert ms.mlora_sched_buffer_left(s) == buf - loop.saved_tokens
            if out["backward"]:
                assert not lens                                         # the backward yields to steps with prompts
        assert len(admitted) == len(set(admitted))                     # nothing is selected twice
        still_saved = [smp.sample_id for smp in loop.saved]
        assert sorted(loop.trained + still_saved) == sorted(admitted)
        assert loop.n_backward == len(ex.backwards) == ex.updates and loop.n_backward > 0
        assert ms.mlora_sched_pool_size(s) == 40 - len(admitted)
    finally:
        ms.mlora_sched_destroy(s)


def test_step_table_layout_and_budget():
    s = make_sched(4096, per_token=1e-3, slo=1.0)
    ex = RecordingExecutor(4096)
    loop = CoServeLoop(ex, s, 8, ft_adapter_of=lambda sid: 5)
    try:
        for i, n in enumerate([300, 100, 200]):
            ms.mlora_sched_pool_add(s, i, n)
        # budget 0.5: inference 0.01 + (128 + 2) * 0.001 = 0.14; samples cost 0.1, 0.2, 0.3 -> 100 and 200 fit (0.44)
        out = loop.step([(128, 1)], [2, 3], 0, t_now=0.5, earliest_arrival=0.0)
        assert out["admitted"] == [1, 2] and out["ft_tokens"] == 300 and abs(out["budget"] - 0.5) < 1e-12
        table, n_rows, base = ex.forwards[-1]
        assert n_rows == 128 + 2 + 300 and base == 0
        assert table.tolist() == [[0, 128, 1, 0], [128, 1, 2, 0], [129, 1, 3, 0], [130, 100, 5, 1], [230, 200, 5, 1]]
        assert not out["backward"]                                     # the step had a prompt
        out = loop.step([], [0], 0, t_now=0.0, earliest_arrival=None)  # decode-only step: backward may run
        assert out["backward"] and ex.backwards[-1].tolist()[:2] == [[0, 100, 5, 1], [100, 200, 5, 1]]
    finally:
        ms.mlora_sched_destroy(s)


def test_interrupted_forward_returns_its_samples():
    s = make_sched(1024)
    ex = RecordingExecutor(1024)
    loop = CoServeLoop(ex, s, 8)
    try:
        for i in range(4):
            ms.mlora_sched_pool_add(s, i, 128)
        out = loop.step([], [], 0, t_now=0.0, earliest_arrival=None, interrupt=True)   # a fine-tuning-only step, aborted
        assert out["interrupted"] and out["admitted"] == []
        assert ms.mlora_sched_pool_size(s) == 4 and ms.mlora_sched_buffer_left(s) == 1024 and loop.saved_tokens == 0
        out = loop.step([], [], 0, t_now=0.0, earliest_arrival=None)
        assert sorted(out["admitted"]) == [0, 1, 2, 3] and out["backward"]
    finally:
        ms.mlora_sched_destroy(s)


def test_sequence_tables_of_the_layer_module_match_a_plain_loop():
    """Host-side tables of the decoder-layer module (position, first and one-past-last row of each row's
    sequence) against the obvious loop, on random sequence layouts with gaps and single-row sequences."""
    import numpy as np
    from paper_2607_28848_b200.layer import sequence_tables
    rng = np.random.default_rng(3)
    for _ in range(20):
        seqs, row = [], 0
        for _ in range(int(rng.integers(0, 30))):
            row += int(rng.integers(0, 3))                    # rows that belong to no sequence
            n = int(rng.integers(0, 50)) if rng.random() < 0.7 else 1
            seqs.append((row, n))
            row += n
        T = row + int(rng.integers(0, 4))
        pos, start, end = sequence_tables(T, seqs)
        p_ref, s_ref = np.zeros(T, np.int32), np.arange(T, dtype=np.int32)
        e_ref = s_ref + 1
        for s0, n in seqs:
            p_ref[s0:s0 + n] = np.arange(n)
            s_ref[s0:s0 + n] = s0
            e_ref[s0:s0 + n] = s0 + n
        assert np.array_equal(pos, p_ref) and np.array_equal(start, s_ref) and np.array_equal(end, e_ref)
        assert pos.dtype == start.dtype == end.dtype == np.int32
