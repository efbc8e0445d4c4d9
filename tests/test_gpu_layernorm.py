"""GPU parity of the bf16 LayerNorm path (tcgen05 GEMM whose epilogue merges row statistics
across the N-tiles of a row strip and normalises out of TMEM) against the CPU oracle."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]


def _case(M, N, K, act, seed=0, scale=1.0, has_bias=True, eps=1e-5):
    return wk.custom_workload(f"ln_{M}x{N}x{K}", wk.BF16, M, N, K, act, wk.RED_LAYERNORM, scale=scale,
                              ln_eps=eps, seed=seed, has_bias=has_bias)


# one tile per strip, several, ragged last tile, M <= 16 (still this kernel), many strips per CTA
SHAPES = [(16, 8, 8), (128, 256, 64), (130, 264, 72), (300, 1000, 200), (1000, 1536, 128), (2500, 4096, 64),
          (128 * 40, 768, 64)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_shapes(M, N, K):
    act = ACTS[(M + N + K) % len(ACTS)]
    wl = _case(M, N, K, act, seed=M + N, scale=1.5)
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05_LN
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"act={act}")


@pytest.mark.parametrize("M,N,K", [(300, 32768, 64), (130, 256 * 75, 72), (16, 256 * 200 + 8, 16)])
def test_rows_with_more_tiles_than_the_grid_are_computed_twice(M, N, K):
    """A row strip of more 256-column tiles than there are CTA pairs cannot be held on chip at once: the kernel
    then makes a statistics pass and a normalising pass over every tile.  Same results, same tolerance; the
    strip counters carry over from run to run."""
    wl = _case(M, N, K, wk.ACT_GELU_TANH, seed=N % 97)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    g, plan = pu.run_gpu(wl, inp, op=op, repeats=3)
    op.close()
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05_LN
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_unit_affine_rows_have_zero_mean_and_unit_variance():
    wl = _case(256, 2048, 256, wk.ACT_GELU_ERF, seed=1, eps=1e-12)
    inp = wk.make_inputs(wl)
    inp["gamma"][:] = 1.0
    inp["beta"][:] = 0.0
    g, _ = pu.run_gpu(wl, inp)
    # bf16 output rounding (2^-9 relative per element) bounds how exactly this can hold
    assert np.abs(g.mean(1)).max() < 2e-3
    assert np.abs(g.var(1) - 1.0).max() < 1e-2
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_constant_rows_give_beta():
    wl = _case(64, 512, 64, wk.ACT_RELU, seed=2)
    inp = wk.make_inputs(wl)
    inp["X"] = -np.abs(inp["X"])
    inp["W"] = np.abs(inp["W"])
    inp["b"][:] = -0.5
    g, _ = pu.run_gpu(wl, inp)
    assert np.array_equal(g, np.tile(inp["beta"].astype(np.float64), (64, 1)))


def test_runs_back_to_back_on_one_handle():
    """The strip counters are never reset between runs; repeated runs must agree."""
    wl = _case(700, 1304, 256, wk.ACT_GELU_TANH, seed=3)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    outs = [pu.run_gpu(wl, inp, op=op, repeats=r)[0] for r in (1, 3, 1)]
    op.close()
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    pu.assert_parity(wl, outs[0], pu.run_oracle(wl, inp))


def test_c5_sampled_rows_full_size():
    wl = wk.WORKLOADS["c5"]
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_TCGEN05_LN
    assert np.isfinite(g).all()
    rows = wk.sample_rows(wl.M)
    pu.assert_parity(wl, g[rows], pu.run_oracle(wl, inp, rows))
