"""GPU parity of the bf16 tcgen05 path (TMA -> shared-memory ring -> tcgen05.mma -> TMEM ->
fused epilogue) against the CPU oracle."""
import dataclasses

import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]


def _case(M, N, K, act, red, seed=0, scale=1.0, has_bias=True):
    return wk.custom_workload(f"bf16_{M}x{N}x{K}", wk.BF16, M, N, K, act, red, scale=scale, seed=seed,
                              has_bias=has_bias)


def test_one_tile_one_k_block_identity_weight():
    """W = I (N = K = 64 padded into one 256-wide tile): Y must reproduce bf16(X) exactly --
    any mistake in the shared-memory / instruction descriptors or the swizzle shows here."""
    wl = _case(128, 64, 64, wk.ACT_IDENTITY, wk.RED_NONE, has_bias=False)
    inp = wk.make_inputs(wl)
    inp["W"] = np.eye(64, dtype=np.float32)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05
    assert np.array_equal(g, inp["X"].astype(np.float64))


def test_k_steps_inside_and_across_swizzle_atoms():
    for K in (16, 32, 64, 128, 136, 512):
        wl = _case(128, 256, K, wk.ACT_IDENTITY, wk.RED_NONE, seed=K)
        inp = wk.make_inputs(wl)
        g, _ = pu.run_gpu(wl, inp)
        pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"K={K}")


SHAPES = [(33, 8, 8), (128, 256, 64), (129, 264, 72), (300, 520, 200), (1000, 776, 328), (2048, 1024, 512)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("red", [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX])
def test_shapes_and_reductions(M, N, K, red):
    act = ACTS[(M + N + K + red) % len(ACTS)]
    wl = _case(M, N, K, act, red, seed=M + K, scale=0.75)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"act={act} red={red}")


@pytest.mark.parametrize("act", ACTS)
def test_every_activation(act):
    wl = _case(256, 512, 128, act, wk.RED_NONE, seed=act, scale=1.25)
    inp = wk.make_inputs(wl)
    inp["W"] = wk.round_to_storage(inp["W"] * 4.0, wk.BF16)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_more_tiles_than_sms_and_both_accumulator_buffers():
    wl = _case(128 * 20, 256 * 9, 192, wk.ACT_SILU, wk.RED_NONE, seed=5)      # 180 tiles on 148 CTAs
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["grid"] <= 148
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_freivalds_covers_every_output_element():
    wl = _case(1536, 1280, 640, wk.ACT_IDENTITY, wk.RED_NONE, seed=2)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    rng = np.random.default_rng(0)
    r = rng.standard_normal(wl.N)
    want = inp["X"].astype(np.float64) @ (inp["W"].astype(np.float64).T @ r) + inp["b"].astype(np.float64) @ r
    # bf16 rounding of each output (2^-9 relative) averages out over N terms
    assert np.max(np.abs(g @ r - want)) <= 2e-2 * np.sqrt(np.mean(want * want))


def test_repeatable_bits_and_workspace_reuse():
    wl = _case(700, 1304, 256, wk.ACT_GELU_TANH, wk.RED_MAX, seed=3)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


def test_c3_sampled_rows_full_size():
    wl = wk.WORKLOADS["c3"]
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05
    assert np.isfinite(g).all()
    rows = wk.sample_rows(wl.M)
    pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))


@pytest.mark.parametrize("M,N,K,grid", [(64, 2048, 4096, 8 * 4), (112, 2048, 4096, 8 * 4), (300, 520, 4096, 2 * 6 * 4), (128, 16384, 2048, 64 * 2)])
@pytest.mark.parametrize("red", [wk.RED_NONE, wk.RED_SUM, wk.RED_MEAN_GELU_RESIDUAL, wk.RED_CROSS_ENTROPY])
def test_tiles_of_the_last_wave_cut_along_k(M, N, K, grid, red):
    """Fewer tiles than CTAs (or CTA pairs): every tile is computed by several of them, a slice of K
    each, and put together by the first.  Same bits on every run (the arrival flags only ever grow).  (With at most
    96 rows only the chain takes this kernel; the other reductions go to the skinny kernel and are checked all the same.)"""
    wl = wk.custom_workload(f"bf16_ksplit_{M}", wk.BF16, M, N, K, wk.ACT_GELU_TANH, red, seed=M + red, w_std=0.02)
    st, plan = B.forge_fused_linear_query_plan(pu.desc_of(wl))
    if M <= 96 and red != wk.RED_MEAN_GELU_RESIDUAL:
        assert st == B.FORGE_OK and plan.kernel == B.FORGE_KERNEL_BF16_SKINNY
    else:
        assert st == B.FORGE_OK and plan.kernel == B.FORGE_KERNEL_BF16_TCGEN05 and plan.grid == grid
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)
    rows = np.unique(np.concatenate([np.arange(0, M, 7), [M - 1]]))
    pu.assert_parity(wl, a[rows], pu.run_oracle(wl, inp, rows))


@pytest.mark.parametrize("red", [wk.RED_NONE, wk.RED_SUM])
def test_one_wave_then_a_k_cut_tail_walked_downwards(red):
    """90 pair tiles on 74 CTA pairs with operands past half of L2: every pair computes one whole tile (K upwards),
    then 16 tiles are left, each cut into 4 parts along K, and these second items walk their k-blocks downwards
    (the K serpentine).  The ring, the part ranges and the hand-over must not care about the direction."""
    M, N, K = 512, 256 * 45, 4096
    wl = wk.custom_workload("bf16_wave_tail_serpentine", wk.BF16, M, N, K, wk.ACT_SILU, red, seed=77 + red, w_std=0.02)
    st, plan = B.forge_fused_linear_query_plan(pu.desc_of(wl))
    assert st == B.FORGE_OK and plan.kernel == B.FORGE_KERNEL_BF16_TCGEN05 and plan.cluster == 2 and plan.grid == 148
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op, repeats=2)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)
    rows = np.unique(np.concatenate([np.arange(0, M, 5), [M - 1]]))
    pu.assert_parity(wl, a[rows], pu.run_oracle(wl, inp, rows))


def test_row_counts_between_the_skinny_kernel_and_a_full_tile():
    """M = 48, 64, 96, 112 against a 32768 x 8192 weight: fewer rows than a 128-row tile -- the problem is bound by
    the stream of W.  Up to 96 rows the skinny kernel serves it, beyond that this kernel (one CTA per tile, the last
    wave cut along K); every output element against the oracle."""
    base = wk.EXTRA_WORKLOADS["m64"]
    full = wk.make_inputs(dataclasses.replace(base, M=112))
    for M in (48, 64, 96, 112):
        wl = dataclasses.replace(base, name=f"m{M}", M=M)
        inp = dict(full)
        inp["X"] = np.ascontiguousarray(full["X"][:M])
        g, plan = pu.run_gpu(wl, inp)
        assert plan["kernel"] == (B.FORGE_KERNEL_BF16_SKINNY if M <= 96 else B.FORGE_KERNEL_BF16_TCGEN05) and plan["cluster"] == 1
        pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"M={M}")
