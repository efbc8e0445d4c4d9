"""GPU parity of the softmax row statistics -- log-sum-exp and per-row cross-entropy, merged
across output tiles as (max, sum of exponentials) pairs -- on the fp32 and bf16 paths."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

REDS = [wk.RED_LOGSUMEXP, wk.RED_CROSS_ENTROPY]
F32_SHAPES = [(1, 1, 1), (5, 100, 7), (128, 128, 16), (130, 300, 36), (257, 1000, 64), (64, 2500, 19)]
BF16_SHAPES = [(128, 256, 64), (300, 520, 200), (1000, 776, 328), (260, 4104, 64),
               # M <= 96: skinny kernel, rows of X padded to a multiple of 16
               (17, 8, 8), (16, 1024, 128), (1, 64, 16), (7, 20000, 264), (16, 148 * 8 * 17, 128), (3, 1184 * 13, 2048),
               (30, 20000, 264), (32, 148 * 8 * 17, 128), (21, 1184 * 13, 2048), (70, 20000, 264), (96, 1184 * 13, 512)]


@pytest.mark.parametrize("M,N,K", F32_SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_fp32(M, N, K, red):
    wl = wk.custom_workload(f"lse_f32_{M}x{N}x{K}", wk.F32, M, N, K, wk.ACT_IDENTITY, red, scale=3.0, seed=M + N)
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert g.shape == (M,) and plan["kernel"] == B.FORGE_KERNEL_F32_FFMA
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


@pytest.mark.parametrize("M,N,K", BF16_SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_bf16(M, N, K, red):
    wl = wk.custom_workload(f"lse_bf16_{M}x{N}x{K}", wk.BF16, M, N, K, wk.ACT_IDENTITY, red, scale=2.0, seed=M + N)
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == (B.FORGE_KERNEL_BF16_SKINNY if M <= 96 else B.FORGE_KERNEL_BF16_TCGEN05)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_large_logits_do_not_overflow_and_runs_repeat():
    wl = wk.custom_workload("lse_big", wk.F32, 200, 700, 32, wk.ACT_IDENTITY, wk.RED_CROSS_ENTROPY, scale=40.0, seed=6)
    inp = wk.make_inputs(wl)
    ref = pu.run_oracle(wl, inp)
    assert ref.max() > 50                                         # exp of these logits overflows fp32 without the max shift
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    op.close()
    assert np.array_equal(a, b) and np.isfinite(a).all()
    pu.assert_parity(wl, a, ref)


def test_cross_entropy_needs_its_targets():
    import torch
    wl = wk.custom_workload("lse_args", wk.BF16, 64, 64, 64, wk.ACT_IDENTITY, wk.RED_CROSS_ENTROPY)
    op = B.FusedLinear(pu.desc_of(wl))
    t = torch.zeros(64 * 64, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(64, dtype=torch.float32, device="cuda")
    assert B.forge_fused_linear_run(op.h, t, t, t, None, None, o) == B.FORGE_ERR_INVALID_ARG
    op.close()


def test_decode_step_of_a_language_model_head_full_oracle():
    wl = wk.custom_workload("lse_decode", wk.BF16, 16, 32768, 4096, wk.ACT_IDENTITY, wk.RED_CROSS_ENTROPY, w_std=0.02, seed=12)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, plan = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op, repeats=3)
    op.close()
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_SKINNY and np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


def test_n2_sampled_rows_full_size():
    wl = wk.EXTRA_WORKLOADS["n2"]
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["cluster"] == 2 and np.isfinite(g).all()
    rows = wk.sample_rows(wl.M)[::2]
    pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
    assert abs(g.mean() - np.log(wl.N)) < 1.0                     # near-uniform predictions: loss close to log N
