"""GPU parity of the IEEE-half storage format (same kernels as bf16: tcgen05 pairs, LayerNorm,
skinny) against the CPU oracle."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]
REDS = [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX, wk.RED_LAYERNORM, wk.RED_MEAN_GELU_RESIDUAL, wk.RED_LOGSUMEXP, wk.RED_CROSS_ENTROPY]


def _case(M, N, K, act, red, seed=0, scale=1.0):
    return wk.custom_workload(f"f16_{M}x{N}x{K}_{red}", wk.F16, M, N, K, act, red, scale=scale, seed=seed, w_std=0.05)


def test_identity_weight_reproduces_x_in_half_precision():
    wl = _case(300, 64, 64, wk.ACT_IDENTITY, wk.RED_NONE)
    inp = wk.make_inputs(wl)
    inp["W"] = np.eye(64, dtype=np.float32)
    inp["b"][:] = 0.0
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05 and plan["cluster"] == 2
    assert np.array_equal(g, inp["X"].astype(np.float64))


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 520, 200), (1000, 776, 328), (16, 1192, 200), (5, 20000, 264),
                                   (29, 20000, 264), (32, 1192, 200)])
@pytest.mark.parametrize("red", REDS)
def test_shapes_and_reductions(M, N, K, red):
    act = ACTS[(M + N + K + red) % len(ACTS)]
    wl = _case(M, N, K, act, red, seed=M + K, scale=0.75)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"act={act} red={red}")


def test_half_is_more_exact_than_bf16_on_the_same_problem():
    errs = {}
    for dt in (wk.F16, wk.BF16):
        wl = wk.custom_workload("prec", dt, 512, 512, 256, wk.ACT_IDENTITY, wk.RED_NONE, seed=3, w_std=0.05)
        inp = wk.make_inputs(wl)
        g, _ = pu.run_gpu(wl, inp)
        errs[dt] = pu.rel_err(g, pu.run_oracle(wl, inp))
    assert errs[wk.F16] < errs[wk.BF16] / 4          # 11 mantissa bits against 8
