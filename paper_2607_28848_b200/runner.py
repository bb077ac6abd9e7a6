"""Convenience driver used by the tests, the smoke check and the benchmark: uploads a workload's
tensors, owns the output / activation buffers, and calls the C ABI through the binding.
It only moves data and marshals arguments; all arithmetic happens in the library's kernels.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding as mb


def torch_dtype(dtype: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]


class Session:
    """One context on one device."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the multi-LoRA layer has no CPU fallback")
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.ctx = mb.mlora_create(device)

    def close(self):
        if self.ctx is not None:
            mb.mlora_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def to_device(self, arr: np.ndarray, dtype: str) -> torch.Tensor:
        return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(self.device).to(torch_dtype(dtype))


class LayerRun:
    """Device-resident tensors of one projection + one batch, ready for forward / backward."""

    def __init__(self, sess: Session, dtype: str, tensors: Dict[str, np.ndarray], segments: np.ndarray,
                 n_rows: int, save_row_base: int = 0, save_capacity_rows: Optional[int] = None,
                 save_x: bool = True, guard: bool = False, adapter_rank=None):
        self.sess, self.dtype = sess, dtype
        td = torch_dtype(dtype)
        dev = sess.device
        self.W = sess.to_device(tensors["W"], dtype)
        self.A_all = sess.to_device(tensors["A_all"], dtype)
        self.B_all = sess.to_device(tensors["B_all"], dtype)
        self.scale = torch.from_numpy(np.asarray(tensors["scale"], dtype=np.float32)).to(dev)
        self.X = sess.to_device(tensors["X"], dtype)
        self.n_adapters, self.rank, self.d_in = self.A_all.shape
        self.d_out = self.B_all.shape[2]
        self.n_rows = n_rows
        self.segments = np.asarray(segments, dtype=np.int32).reshape(-1, 4)
        if adapter_rank is None:
            self.plan = mb.mlora_plan_create(sess.ctx, self.segments, n_rows, self.n_adapters)
        else:               # adapters with ranks of their own (stored padded to the layer's rank)
            self.plan = mb.mlora_plan_create_ranked(sess.ctx, self.segments, n_rows, self.n_adapters, adapter_rank)
        self.ft_rows = mb.mlora_plan_ft_rows(self.plan)
        self.slots = mb.mlora_plan_ft_adapters(self.plan)
        self.layer = mb.make_layer(self.W, self.A_all, self.B_all, self.scale)
        self.save_row_base = save_row_base
        cap = save_row_base + self.ft_rows if save_capacity_rows is None else save_capacity_rows
        self.capacity = cap
        fill = float("nan") if guard else 0.0
        self.Y = torch.full((n_rows, self.d_out), fill, dtype=td, device=dev)
        self.x_save = torch.full((max(cap, 1), self.d_in), fill, dtype=td, device=dev) if save_x else None
        self.u_save = torch.full((max(cap, 1), self.rank), fill, dtype=torch.float32, device=dev)
        n_slots = max(len(self.slots), 1)
        self.dA = torch.full((n_slots, self.rank, self.d_in), fill, dtype=torch.float32, device=dev)
        self.dB = torch.full((n_slots, self.rank, self.d_out), fill, dtype=torch.float32, device=dev)
        self.dX = torch.full((max(self.ft_rows, 1), self.d_in), fill, dtype=td, device=dev)
        self.dY = sess.to_device(tensors["dY"], dtype) if "dY" in tensors and self.ft_rows else None

    def forward(self):
        mb.mlora_mixed_forward(self.sess.ctx, self.layer, self.plan, self.X, self.Y, self.x_save, self.u_save,
                               self.save_row_base, self.capacity)

    def backward(self, accumulate: bool = False, want_dx: bool = True):
        b = self.save_row_base
        xs = self.x_save[b:] if self.x_save is not None else None
        mb.mlora_backward(self.sess.ctx, self.layer, self.plan, self.dY, xs, self.u_save[b:], self.dA, self.dB,
                          self.dX if want_dx else None, accumulate)

    def status(self) -> int:
        return mb.mlora_poll_status(self.sess.ctx)

    def close(self):
        if self.plan is not None:
            mb.mlora_plan_destroy(self.plan)
            self.plan = None

    @staticmethod
    def host(t: torch.Tensor) -> np.ndarray:
        return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)
