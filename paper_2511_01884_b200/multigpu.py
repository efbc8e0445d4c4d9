"""Host-side logic of the multi-GPU run: one process per GPU, rows of X sharded over ranks.

Every reduction of the operator runs along N, so rows are independent: a rank computes its
block of rows with replicated W, b, gamma, beta and no collective touches the data path.
The only exchange is the timing one: the slowest rank's time decides the aggregate rate.
"""
from __future__ import annotations

from typing import Tuple

from . import workloads as wk


def rank_rows_weak(wl: wk.Workload, rank: int) -> Tuple[int, int]:
    """Weak scaling: every rank gets wl.M rows of a global input of world * wl.M rows.
    Returns (M, row_offset) for ``workloads.make_inputs``."""
    return wl.M, rank * wl.M


def rank_rows_strong(wl: wk.Workload, rank: int, world: int) -> Tuple[int, int]:
    """Strong scaling: the wl.M rows are split into contiguous blocks."""
    lo, hi = wk.shard_rows(wl.M, rank, world)
    return hi - lo, lo


def max_over_ranks(ms: float, dist=None, device=None) -> float:
    """Max of a per-rank time over all ranks (identity when not distributed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Whole-job rate: the units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / (ms_max * 1e-3)
