"""World-size-2 run of the multi-GPU host logic on CPU (gloo): row sharding, that the shards
reproduce the single-process result when evaluated by the oracle, and the max-over-ranks
timing exchange."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_01884_b200 import multigpu
from paper_2511_01884_b200 import workloads as wk


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, strong, q):
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = wk.custom_workload("mr", wk.F32, 37, 24, 16, wk.ACT_SILU, wk.RED_SUM, seed=5)
    M, off = multigpu.rank_rows_strong(wl, rank, world) if strong else multigpu.rank_rows_weak(wl, rank)
    inp = wk.make_inputs(wl, M=M, row_offset=off)
    out = oracle.fused_linear(inp["X"], inp["W"], inp["b"], act=wl.act, scale=wl.scale, red=wl.red)
    ms = multigpu.max_over_ranks(10.0 * (rank + 1), dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, (off, out))
    if rank == 0:
        q.put((ms, gathered))
    dist.barrier()
    dist.destroy_process_group()


def _run(strong):
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, strong, q)) for r in range(2)]
    for p in procs:
        p.start()
    ms, gathered = q.get()
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    return ms, gathered


def _single(M_total):
    import oracle
    wl = wk.custom_workload("mr", wk.F32, 37, 24, 16, wk.ACT_SILU, wk.RED_SUM, seed=5)
    inp = wk.make_inputs(wl, M=M_total)
    return oracle.fused_linear(inp["X"], inp["W"], inp["b"], act=wl.act, scale=wl.scale, red=wl.red)


def test_strong_sharding_reproduces_single_process():
    ms, gathered = _run(strong=True)
    assert ms == 20.0                                   # slowest rank decides
    got = np.concatenate([o for _, o in sorted(gathered, key=lambda t: t[0])])
    assert np.array_equal(got, _single(37))


def test_weak_sharding_tiles_a_global_input():
    ms, gathered = _run(strong=False)
    got = np.concatenate([o for _, o in sorted(gathered, key=lambda t: t[0])])
    assert np.array_equal(got, _single(74))             # two ranks x 37 rows of one global X
    assert multigpu.aggregate_rate(100.0, 2, ms) == 2 * 100.0 / 0.020


def test_single_process_helpers():
    assert multigpu.max_over_ranks(3.5) == 3.5
    wl = wk.WORKLOADS["c3"]
    assert multigpu.rank_rows_weak(wl, 3) == (8192, 3 * 8192)
    assert multigpu.rank_rows_strong(wl, 1, 4) == (2048, 2048)


def _col_worker(rank, world, port, red, q):
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = wk.custom_workload("mc", wk.F32, 9, 40, 24, wk.ACT_GELU_ERF, red, seed=3)
    inp = wk.make_inputs(wl)
    lo, hi = multigpu.rank_cols(wl, rank, world)
    part = oracle.fused_linear(inp["X"], inp["W"][lo:hi], inp["b"][lo:hi], act=wl.act, scale=wl.scale, red=wl.red)
    out = multigpu.combine_column_partials(torch.from_numpy(np.ascontiguousarray(part)), red, dist)
    if rank == 0:
        q.put(((lo, hi), out.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_column_shards_combine_to_the_unsharded_result():
    """W split by rows over two ranks; the per-rank row sums / maxima (here from the
    oracle) combined by the small collective give the unsharded operator's output."""
    import oracle
    for red in multigpu.COLUMN_SHARDABLE:
        ctx = mp.get_context("spawn")
        q = ctx.SimpleQueue()
        port = _free_port()
        procs = [ctx.Process(target=_col_worker, args=(r, 2, port, red, q)) for r in range(2)]
        for p in procs:
            p.start()
        (lo, hi), got = q.get()
        for p in procs:
            p.join(60)
            assert p.exitcode == 0
        assert (lo, hi) == (0, 24)                           # 5 groups of 8 columns: 3 + 2
        wl = wk.custom_workload("mc", wk.F32, 9, 40, 24, wk.ACT_GELU_ERF, red, seed=3)
        inp = wk.make_inputs(wl)
        want = oracle.fused_linear(inp["X"], inp["W"], inp["b"], act=wl.act, scale=wl.scale, red=wl.red)
        assert np.allclose(got, want, rtol=1e-13, atol=1e-13), red
    wl = wk.WORKLOADS["c4"]
    assert [multigpu.rank_cols(wl, r, 8) for r in (0, 7)] == [(0, 2048), (14336, 16384)]
    with np.testing.assert_raises(ValueError):
        multigpu.combine_column_partials(torch.zeros(3), wk.RED_LAYERNORM)
