"""Seeded random shapes through every kernel family against the CPU oracle: ragged tails in M, N and
K, sizes around the tile, cluster, slice and split thresholds, every activation and reduction."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]
REDS = [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX, wk.RED_LAYERNORM, wk.RED_MEAN_GELU_RESIDUAL, wk.RED_LOGSUMEXP, wk.RED_CROSS_ENTROPY]


def _cases(dtype, n, seed, step, m_hi, n_hi, k_hi):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        M = int(rng.integers(1, m_hi + 1))
        N = int(rng.integers(1, n_hi // step + 1)) * step
        K = int(rng.integers(1, k_hi // step + 1)) * step
        if rng.random() < 0.3:                      # long K with few tiles: slices / K cuts
            K = int(rng.integers(k_hi // step, 4 * k_hi // step + 1)) * step
        act, red = ACTS[int(rng.integers(5))], REDS[int(rng.integers(7))]
        out.append((M, N, K, act, red, bool(rng.integers(2)), len(out)))
    return out


@pytest.mark.parametrize("M,N,K,act,red,bias,i", _cases(wk.F32, 24, 1, 1, 300, 700, 200))
def test_fp32(M, N, K, act, red, bias, i):
    _check(wk.F32, M, N, K, act, red, bias, i)


@pytest.mark.parametrize("M,N,K,act,red,bias,i", _cases(wk.F32_TF32X3, 24, 2, 4, 600, 1100, 600))
def test_fp32_on_tensor_cores(M, N, K, act, red, bias, i):
    _check(wk.F32_TF32X3, M, N, K, act, red, bias, i)


@pytest.mark.parametrize("M,N,K,act,red,bias,i", _cases(wk.BF16, 32, 3, 8, 600, 1100, 600))
def test_bf16(M, N, K, act, red, bias, i):
    _check(wk.BF16, M, N, K, act, red, bias, i)


@pytest.mark.parametrize("M,N,K,act,red,bias,i", _cases(wk.F16, 12, 4, 8, 300, 600, 300))
def test_f16(M, N, K, act, red, bias, i):
    _check(wk.F16, M, N, K, act, red, bias, i)


def _check(dtype, M, N, K, act, red, bias, i):
    w_std = None if dtype in (wk.F32, wk.F32_TF32X3) else 1.0 / max(K, 1) ** 0.5
    wl = wk.custom_workload(f"fuzz{dtype}_{i}", dtype, M, N, K, act, red, scale=0.5 + 0.25 * (i % 4), seed=100 + i,
                            w_std=w_std, has_bias=bias)
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp, repeats=2)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"M={M} N={N} K={K} act={act} red={red} kernel={plan['kernel']} grid={plan['grid']}")
