"""The co-serving loop on the GPU: steps appended to the activation buffer over several forwards,
then one backward over the compact table; its gradients are checked against the oracle."""
import numpy as np
import pytest
import torch

from oracle import mlora_oracle as orc
from paper_2607_28848_b200 import binding as mb
from paper_2607_28848_b200 import sched as ms
from paper_2607_28848_b200.coserve import CoServeLoop, GpuExecutor
from paper_2607_28848_b200.runner import LayerRun, Session
from test_gpu_parity import TOL, assert_close

pytestmark = pytest.mark.gpu


class Recording(GpuExecutor):
    def __init__(self, *a, **k):
        super().__init__(*a, **k)
        self.tables = []
        self.first = None

    def forward(self, table, n_rows, save_base, cancel=False):
        ok = super().forward(table, n_rows, save_base, cancel)
        if ok:
            self.tables.append((table.copy(), n_rows, save_base))
        return ok

    def backward(self, table, n_rows):
        A0, B0 = self.A.clone(), self.B.clone()
        super().backward(table, n_rows)
        if self.first is None:
            self.first = (table.copy(), n_rows, list(self.tables), A0, B0, self.dA.clone(), self.dB.clone(), list(self.slots),
                          self.dX[:n_rows].clone())
        self.tables = []


def test_loop_backward_matches_oracle():
    buf = 512
    with Session(0) as sess:
        ex = Recording(sess, 256, 384, 16, 6, 1024, buf, seed=3)
        c = ms.mixed_coef(0.0, 1e-3, 0.0, 0.0, 0.01)
        s = ms.mlora_sched_create(c, c, ms.decode_coef(), 1.0, 1.0, buf)
        loop = CoServeLoop(ex, s, 6, ft_adapter_of=lambda sid: sid % 3, backward_batch=256)
        try:
            for i in range(12):
                ms.mlora_sched_pool_add(s, i, 40 + 24 * (i % 4))
            # three steps with prompts (tight budgets: a few samples each), then a decode-only step
            for t_now in (0.75, 0.7, 0.72):
                loop.step([(100, 4), (37, 5)], [0, 1, 2, 3], 0, t_now=t_now, earliest_arrival=0.0)
            out = loop.step([], [1, 2], 0, t_now=0.0, earliest_arrival=None)
            assert out["backward"] and ex.first is not None
            assert mb.mlora_poll_status(sess.ctx) == mb.MLORA_OK
            table_b, rows_b, tables, A0, B0, dA, dB, slots, dX = ex.first
            host = LayerRun.host
            X, W, scale = host(ex.X), host(ex.W), ex.scale.cpu().numpy().astype(np.float64)
            A0h, B0h = host(A0), host(B0)
            xs = np.zeros((rows_b, 256))
            us = np.zeros((rows_b, 16))
            for table, n_rows, base in tables:                        # what each forward must have appended
                _, ft_segments, ft_rows, _ = orc.route(table, n_rows, 6)
                for start, length, a, off in ft_segments:
                    xs[base + off:base + off + length] = X[start:start + length]
                    us[base + off:base + off + length] = X[start:start + length] @ A0h[a].T
            assert np.array_equal(host(ex.x_save[:rows_b]), xs)
            ref = orc.backward(host(ex.dY[:rows_b]), W, A0h, B0h, scale, table_b, xs, us, n_rows=rows_b)
            assert slots == ref["ft_adapters"]
            assert_close("dA", host(dA), ref["dA"], TOL["bf16"])
            assert_close("dB", host(dB), ref["dB"], TOL["bf16"])
            assert_close("dX", host(dX), ref["dX"], TOL["bf16"])
            assert loop.saved_tokens == 0 and ms.mlora_sched_buffer_left(s) == buf
        finally:
            ms.mlora_sched_destroy(s)
