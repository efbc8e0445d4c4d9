"""GPU parity of the fp32-storage path whose contraction runs on the tensor cores as three TF32
products (head*head + head*tail + tail*head) against the CPU oracle, at the fp32 tolerance."""
import dataclasses

import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

T = wk.F32_TF32X3
ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]
REDS = [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX, wk.RED_LAYERNORM, wk.RED_MEAN_GELU_RESIDUAL, wk.RED_LOGSUMEXP, wk.RED_CROSS_ENTROPY]


def test_identity_weight_reproduces_full_fp32_mantissas():
    """W = I: Y must be X to fp32 accuracy although a TF32 operand keeps only 10 fraction bits.
    The inputs carry every low-order bit pattern (a head-only product would be off by 2^-11, and a
    tail computed against the wrong rounding of the head by 2^-10)."""
    wl = wk.custom_workload("t_identity", T, 300, 256, 256, wk.ACT_IDENTITY, wk.RED_NONE)
    inp = wk.make_inputs(wl)
    x = inp["X"].view(np.uint32).copy()
    low = (np.arange(x.size, dtype=np.uint32).reshape(x.shape) * np.uint32(2654435761)) & np.uint32(0x1FFF)
    inp["X"] = ((x & np.uint32(0xFFFFE000)) | low).view(np.float32)          # all 8192 tails occur
    inp["W"] = np.eye(256, dtype=np.float32)
    inp["b"][:] = 0.0
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_F32_TF32X3 and plan["cluster"] == 2
    X = inp["X"].astype(np.float64)
    assert np.max(np.abs(g - X) / np.abs(X)) <= 2.0 ** -20


def test_c2_tensors_sampled_rows_full_size():
    wl = wk.EXTRA_WORKLOADS["c2t"]
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    rows = wk.sample_rows(wl.M)
    e = pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
    assert e <= 1e-5, e        # the split leaves about 2^-21 per product: far inside the 1e-4 budget
    assert np.isfinite(g).all()


# several pair tiles in both directions, ragged tails in M, N and K (K % 32 != 0: zero-filled
# TMA boxes), M <= 128 (the second CTA of the pair has no rows), many ring passes
SHAPES = [(4, 4, 4), (100, 260, 36), (129, 256, 32), (300, 520, 132), (513, 1028, 68), (260, 300, 1000)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_shapes_and_reductions(M, N, K, red):
    act = ACTS[(M + N + K + red) % len(ACTS)]
    wl = wk.custom_workload(f"t_{M}x{N}x{K}", T, M, N, K, act, red, scale=0.75, seed=M + N)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"act={act} red={red}")


@pytest.mark.parametrize("act", ACTS)
def test_every_activation(act):
    wl = wk.custom_workload("t_act", T, 150, 140, 72, act, wk.RED_NONE, scale=1.25, seed=act)
    inp = wk.make_inputs(wl)
    inp["W"] = wk.round_to_storage(inp["W"] * 4.0, T)       # widen the pre-activations: tails of the activation
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_same_sign_operands_do_not_accumulate_the_truncation_bias():
    """All products positive: the dropped part of every tail has the same sign, the worst case for
    the split.  Row sums over K = 4096 must still sit far inside the tolerance."""
    wl = wk.custom_workload("t_bias", T, 260, 512, 4096, wk.ACT_IDENTITY, wk.RED_SUM, seed=9)
    inp = wk.make_inputs(wl)
    inp["X"] = np.abs(inp["X"])
    inp["W"] = np.abs(inp["W"])
    g, _ = pu.run_gpu(wl, inp)
    rows = np.arange(0, 260, 7)
    e = pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
    assert e <= 1e-5, e


def test_freivalds_covers_every_output_element():
    wl = wk.custom_workload("t_freivalds", T, 1000, 900, 520, wk.ACT_IDENTITY, wk.RED_NONE, seed=2)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    rng = np.random.default_rng(0)
    for _ in range(3):
        r = rng.standard_normal(wl.N)
        want = inp["X"].astype(np.float64) @ (inp["W"].astype(np.float64).T @ r) + inp["b"].astype(np.float64) @ r
        assert np.max(np.abs(g @ r - want)) <= 1e-4 * np.sqrt(np.mean(want * want))


def test_repeatable_bits_no_bias_and_workspace_reuse():
    wl = wk.custom_workload("t_rep", T, 600, 700, 64, wk.ACT_SILU, wk.RED_SUM, seed=3, has_bias=False)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


@pytest.mark.parametrize("red", [wk.RED_NONE, wk.RED_MAX, wk.RED_MEAN_GELU_RESIDUAL, wk.RED_CROSS_ENTROPY])
def test_tiles_of_the_last_wave_cut_along_k(red):
    """6 pair tiles on 74 clusters, K = 2048: every tile is computed by 4 clusters, a quarter of K each,
    and put together by the first of them.  Same bits on every run (the arrival flags only ever grow)."""
    wl = wk.custom_workload("t_ksplit", T, 300, 520, 2048, wk.ACT_GELU_ERF, red, seed=11)
    st, plan = B.forge_fused_linear_query_plan(pu.desc_of(wl))
    assert st == B.FORGE_OK and plan.grid == 2 * 6 * 4
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)
    e = pu.assert_parity(wl, a, pu.run_oracle(wl, inp))
    assert e <= 1e-5, e


def test_agrees_with_the_ffma_kernel_far_inside_the_tolerance():
    base = wk.custom_workload("t_vs_ffma", wk.F32, 512, 768, 2048, wk.ACT_GELU_ERF, wk.RED_NONE, seed=5)
    inp = wk.make_inputs(base)
    f, pf = pu.run_gpu(base, inp)
    t, pt = pu.run_gpu(dataclasses.replace(base, dtype=T), inp)
    assert pf["kernel"] == B.FORGE_KERNEL_F32_FFMA and pt["kernel"] == B.FORGE_KERNEL_F32_TF32X3
    assert pu.rel_err(t, f) <= 1e-5


def test_layernorm_of_wide_rows():
    """N = 4096 (16 tiles per row strip), many strips, several launches on one handle (the strip counters only
    ever grow)."""
    wl = wk.custom_workload("t_ln_wide", T, 1500, 4096, 256, wk.ACT_GELU_TANH, wk.RED_LAYERNORM, seed=6)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    b, _ = pu.run_gpu(wl, inp, op=op)
    op.close()
    assert np.array_equal(a, b)
    rows = wk.sample_rows(wl.M)
    e = pu.assert_parity(wl, a[rows], pu.run_oracle(wl, inp, rows))
    assert e <= 2e-5, e


def test_layernorm_constant_rows_give_beta():
    wl = wk.custom_workload("t_ln_const", T, 5, 520, 12, wk.ACT_RELU, wk.RED_LAYERNORM, seed=1)
    inp = wk.make_inputs(wl)
    inp["X"][:] = -np.abs(inp["X"])
    inp["W"][:] = np.abs(inp["W"])
    inp["b"][:] = -0.5                      # every pre-activation negative: ReLU output is all zero
    g, _ = pu.run_gpu(wl, inp)
    assert np.array_equal(g, np.tile(inp["beta"].astype(np.float64), (5, 1)))


def test_what_the_kernel_does_not_serve_is_refused():
    for M, N, K, red in [(64, 64, 66, wk.RED_NONE), (64, 66, 64, wk.RED_NONE)]:
        st, _ = B.forge_fused_linear_query_plan(B.make_desc(M, N, K, T, 0, red))
        assert st == B.FORGE_ERR_UNSUPPORTED


def test_layernorm_rows_with_more_tiles_than_cta_pairs():
    """More 256-column tiles per row strip than the grid has CTA pairs: every tile is computed twice (statistics,
    then normalisation); the strip counters carry over from run to run."""
    wl = wk.custom_workload("t_ln_2pass", T, 140, 256 * 80 + 8, 64, wk.ACT_GELU_TANH, wk.RED_LAYERNORM, seed=9)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    g, plan = pu.run_gpu(wl, inp, op=op, repeats=3)
    op.close()
    assert plan["kernel"] == B.FORGE_KERNEL_F32_TF32X3
    e = pu.assert_parity(wl, g, pu.run_oracle(wl, inp))
    assert e <= 2e-5, e
