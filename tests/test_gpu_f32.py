"""GPU parity of the fp32 path (register-tiled FFMA kernel) against the CPU oracle."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]
REDS = [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX, wk.RED_LAYERNORM]


def test_c1_full():
    wl = wk.WORKLOADS["c1"]
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_F32_FFMA
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_c2_sampled_rows_full_size():
    wl = wk.WORKLOADS["c2"]
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    rows = wk.sample_rows(wl.M)
    pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
    assert np.isfinite(g).all()


# several tiles in both directions plus ragged tails; K not a multiple of 4 takes the scalar loads
SHAPES = [(1, 1, 1), (3, 5, 7), (128, 128, 16), (129, 257, 33), (200, 130, 64), (64, 300, 100), (257, 96, 19)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_shapes_and_reductions(M, N, K, red):
    act = ACTS[(M + N + K + red) % len(ACTS)]
    wl = wk.custom_workload(f"f32_{M}x{N}x{K}", wk.F32, M, N, K, act, red, scale=0.75, seed=M + N)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"act={act} red={red}")


@pytest.mark.parametrize("act", ACTS)
def test_every_activation(act):
    wl = wk.custom_workload("f32_act", wk.F32, 150, 140, 72, act, wk.RED_NONE, scale=1.25, seed=act)
    inp = wk.make_inputs(wl)
    # widen the pre-activations so that the tails of the activation are exercised
    inp["W"] = wk.round_to_storage(inp["W"] * 4.0, wk.F32)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


# one tile per strip, 8 and 9 tiles (past the width a thread-block cluster would span), 32 tiles with many strips
# per CTA (several waves of persistent CTAs), a row as wide as a language-model head with few rows
@pytest.mark.parametrize("M,N,K,bias", [(130, 1024, 40, False), (70, 1032, 36, True), (1500, 4096, 64, True),
                                        (40, 32768, 24, True), (128 * 5 + 3, 128 * 59 + 8, 20, True),
                                        (130, 128 * 300 + 5, 12, True)])      # more tiles per strip than CTAs: two passes
def test_layernorm_of_wide_rows(M, N, K, bias):
    wl = wk.custom_workload(f"f32_ln_{N}", wk.F32, M, N, K, wk.ACT_GELU_ERF, wk.RED_LAYERNORM, has_bias=bias, seed=4)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    g, plan = pu.run_gpu(wl, inp, op=op, repeats=3)           # the strip counters are never reset between runs
    op.close()
    assert plan["kernel"] == B.FORGE_KERNEL_F32_FFMA and plan["cluster"] == 1 and plan["grid"] <= 2 * 148
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_layernorm_rows_wider_than_the_grid_are_planned():
    # the tiles of a strip wait for one another; with more 128-column tiles than resident CTAs every tile is computed twice
    for N in (128 * 296, 128 * 296 + 1, 1 << 20):
        st, p = B.forge_fused_linear_query_plan(B.make_desc(8, N, 8, wk.F32, 0, wk.RED_LAYERNORM))
        assert st == B.FORGE_OK and p.grid <= 296


def test_layernorm_constant_rows_give_beta():
    wl = wk.custom_workload("f32_ln_const", wk.F32, 5, 200, 12, wk.ACT_RELU, wk.RED_LAYERNORM, seed=1)
    inp = wk.make_inputs(wl)
    inp["X"][:] = -np.abs(inp["X"])
    inp["W"][:] = np.abs(inp["W"])
    inp["b"][:] = -0.5                      # every pre-activation negative: ReLU output is all zero
    g, _ = pu.run_gpu(wl, inp)
    assert np.array_equal(g, np.tile(inp["beta"].astype(np.float64), (5, 1)))


def test_freivalds_covers_every_output_element():
    """act = identity: Y r must equal X (W^T r) + (b . r) for random r (checks all of Y in O(MN))."""
    wl = wk.custom_workload("f32_freivalds", wk.F32, 1000, 900, 520, wk.ACT_IDENTITY, wk.RED_NONE, seed=2)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    rng = np.random.default_rng(0)
    for _ in range(3):
        r = rng.standard_normal(wl.N)
        want = inp["X"].astype(np.float64) @ (inp["W"].astype(np.float64).T @ r) + inp["b"].astype(np.float64) @ r
        got = g @ r
        assert np.max(np.abs(got - want)) <= 1e-4 * (np.sqrt(np.mean(want * want)))


def test_repeatable_bits_and_workspace_reuse():
    wl = wk.custom_workload("f32_rep", wk.F32, 300, 700, 64, wk.ACT_SILU, wk.RED_SUM, seed=3)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op)          # second run reuses counters reset by the first
    op.close()
    assert np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


# few 64x64 tiles and a long K: K is cut into slices that run on different SMs and are summed, in slice
# order, by the CTA that arrives last (ragged last slice, scalar loads when K % 4 != 0)
SLICED = [(100, 200, 520), (7, 70, 1000), (33, 65, 333), (128, 512, 256)]


@pytest.mark.parametrize("M,N,K", SLICED)
@pytest.mark.parametrize("red", [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX, wk.RED_MEAN_GELU_RESIDUAL, wk.RED_LOGSUMEXP, wk.RED_CROSS_ENTROPY])
def test_small_grids_cut_along_k(M, N, K, red):
    act = ACTS[(M + red) % len(ACTS)]
    wl = wk.custom_workload(f"f32_sl_{M}x{N}x{K}", wk.F32, M, N, K, act, red, scale=1.5, seed=K + red)
    st, plan = B.forge_fused_linear_query_plan(pu.desc_of(wl))
    tiles = -(-M // 64) * -(-N // 64)
    assert st == B.FORGE_OK and plan.tile_m == 64 and plan.grid > tiles
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)                 # fixed summation order, counters back at zero
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp), f"act={act} red={red}")
