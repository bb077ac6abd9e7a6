"""Multi-GPU helpers for the replica mode.

Rows of a batch are independent in the forward and in dX, and this build runs one GPU per
replica with no exchange on the data path (the paper's multi-GPU deployment is engine replicas
too).  What N processes share is only the measurement protocol: a barrier on both sides of the
timed region and the slowest rank's time.  These helpers work on any torch.distributed backend
(nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """The largest of the ranks' values (every rank gets it)."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank_per_step: float, steps: int, ms_this_rank: float,
                         device: torch.device | str = "cpu") -> dict:
    """Whole-job throughput of N replicas: all ranks' units divided by the slowest rank's time."""
    ms = max_over_ranks(ms_this_rank, device)
    n = world()
    return {"n_gpus": n, "ms_per_step": ms / steps, "value": n * units_per_rank_per_step * steps / (ms * 1e-3)}


def shard_segments(segments: Sequence[Sequence[int]], n_shards: int) -> List[list]:
    """Split a segment table by whole segments into n_shards batches of similar size (requests
    never straddle replicas); each shard's rows are renumbered from 0.  Greedy by descending length."""
    order = sorted(range(len(segments)), key=lambda k: -int(segments[k][1]))
    loads = [0] * n_shards
    picks: List[List[int]] = [[] for _ in range(n_shards)]
    for k in order:
        s = min(range(n_shards), key=lambda i: loads[i])
        picks[s].append(k)
        loads[s] += int(segments[k][1])
    out = []
    for s in range(n_shards):
        row, table = 0, []
        for k in sorted(picks[s]):
            _st, ln, ad, ft = (int(v) for v in segments[k])
            table.append((row, ln, ad, ft))
            row += ln
        out.append(table)
    return out
