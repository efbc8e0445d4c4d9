"""GPU parity of the case-study chain (Linear, subtract, row mean, GELU, residual add) on the
fp32 and bf16 paths against the CPU oracle."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

# one N-tile and several; ragged M, N, K; K not a multiple of 4 (scalar residual path)
SHAPES = [(1, 1, 1), (5, 100, 7), (128, 128, 16), (130, 300, 36), (257, 1000, 64), (300, 96, 19), (1000, 2048, 128)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_shapes(M, N, K):
    wl = wk.custom_workload(f"chain_{M}x{N}x{K}", wk.F32, M, N, K, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL, seed=M + N)
    inp = wk.make_inputs(wl)
    # spread the row means over the curved part of the GELU
    inp["b"] = wk.round_to_storage(inp["b"] + np.linspace(-2, 2, N).astype(np.float32) * 0 + 0.7, wk.F32)
    g, plan = pu.run_gpu(wl, inp)
    assert g.shape == (M, K) and plan["kernel"] == B.FORGE_KERNEL_F32_FFMA
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


BF16_SHAPES = [(17, 8, 8), (128, 256, 64), (130, 264, 72), (300, 1000, 200), (1000, 1536, 128), (16, 512, 64)]


@pytest.mark.parametrize("M,N,K", BF16_SHAPES)
def test_bf16_shapes(M, N, K):
    wl = wk.custom_workload(f"chain_bf16_{M}x{N}x{K}", wk.BF16, M, N, K, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL,
                            seed=M + N, w_std=0.1)
    inp = wk.make_inputs(wl)
    inp["b"] = wk.round_to_storage(inp["b"] + 0.7, wk.BF16)
    g, plan = pu.run_gpu(wl, inp)
    assert g.shape == (M, K) and plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05          # also for M <= 16
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_bf16_repeats_and_no_subtract_vector():
    wl = wk.custom_workload("chain_bf16_rep", wk.BF16, 700, 1304, 256, wk.ACT_SILU, wk.RED_MEAN_GELU_RESIDUAL, seed=4, w_std=0.1)
    inp = wk.make_inputs(wl)
    inp["sub"] = None
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    op.close()
    assert np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


def test_with_activation_scale_and_no_subtract_vector():
    wl = wk.custom_workload("chain_act", wk.F32, 200, 260, 48, wk.ACT_RELU, wk.RED_MEAN_GELU_RESIDUAL, scale=3.0, seed=9)
    inp = wk.make_inputs(wl)
    inp["sub"] = None
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_zero_mean_returns_the_input_bits():
    wl = wk.custom_workload("chain_zero", wk.F32, 140, 256, 32, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL, seed=3)
    inp = wk.make_inputs(wl)
    inp["W"][:] = 0.0
    inp["sub"] = inp["b"].copy()
    g, _ = pu.run_gpu(wl, inp)
    assert np.array_equal(g, inp["X"].astype(np.float64))


def test_two_runs_on_one_handle():
    wl = wk.custom_workload("chain_rep", wk.F32, 300, 700, 64, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL, seed=4)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    op.close()
    assert np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


def test_n1_sampled_rows_full_size():
    wl = wk.EXTRA_WORKLOADS["n1"]
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    rows = wk.sample_rows(wl.M)
    pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
    assert np.isfinite(g).all()


@pytest.mark.parametrize("name", ["n1t", "n1b"])
def test_chain_on_the_tensor_core_kernels_sampled_rows_full_size(name):
    """The bench's launch configurations: the residual rows are written by the whole grid after all
    strips have published gelu(mean) (cooperative launch); n1t also cuts its last wave along K."""
    wl = wk.EXTRA_WORKLOADS[name]
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp, repeats=2)
    assert plan["cluster"] == 2
    rows = wk.sample_rows(wl.M)
    pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
    assert np.isfinite(g).all()
