"""Host-side logic of the multi-GPU run: one process per GPU.

Rows of X sharded over ranks (the default): every reduction of the operator runs along N, so rows
are independent; a rank computes its block of rows with replicated W, b, gamma, beta and no
collective touches the data path.  The only exchange is the timing one: the slowest rank's
time decides the aggregate rate.

Columns (rows of W) sharded over ranks, for the skinny-M problems whose whole cost is streaming
W: every rank holds N / world rows of W and the matching slice of b, runs the same fused kernel
on its slice and gets a partial out[M]; the partials are combined by one small all-reduce of M
floats (sum or max).  That exchange is a real step of the path, so it is a collective (NCCL on
GPUs); nothing else is computed outside the kernels.
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


def rank_cols(wl: wk.Workload, rank: int, world: int) -> Tuple[int, int]:
    """Column sharding: contiguous block [lo, hi) of the N rows of W (multiples of 8, the
    16-bit kernels' row pitch rule) owned by ``rank``."""
    groups = wl.N // 8
    if groups * 8 != wl.N or groups < world:
        raise ValueError("column sharding needs N to be a multiple of 8 with at least one group per rank")
    lo, hi = wk.shard_rows(groups, rank, world)
    return 8 * lo, 8 * hi


COLUMN_SHARDABLE = (wk.RED_SUM, wk.RED_MAX)


def combine_column_partials(partial, red: int, dist=None):
    """Combine the per-rank out[M] of a column-sharded run in place (a torch tensor on the rank's
    device) and return it: all-reduce SUM for the row sum, MAX for the row max."""
    if red not in COLUMN_SHARDABLE:
        raise ValueError("only row sum and row max combine across column shards by a plain all-reduce")
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return partial
    dist.all_reduce(partial, op=dist.ReduceOp.SUM if red == wk.RED_SUM else dist.ReduceOp.MAX)
    return partial
