"""GPU parity of the skinny-M bf16 path (M <= 96: rows of W as the M dimension of tcgen05.mma, X as its
N dimension, a TMA ring, warp-shuffle row reductions) against the CPU oracle."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]


def _case(M, N, K, act, red, seed=0, scale=1.0, has_bias=True):
    return wk.custom_workload(f"skinny_{M}x{N}x{K}", wk.BF16, M, N, K, act, red, scale=scale, seed=seed,
                              has_bias=has_bias)


def test_identity_weight_reproduces_x():
    wl = _case(16, 64, 64, wk.ACT_IDENTITY, wk.RED_NONE, has_bias=False)
    inp = wk.make_inputs(wl)
    inp["W"] = np.eye(64, dtype=np.float32)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_SKINNY
    assert np.array_equal(g, inp["X"].astype(np.float64))


# N/8 below, at and far above the SM count (1, several and many strips per CTA); K with a
# ragged last block and fewer blocks than K-slices; M below 16
# ... and K long enough for many passes over the shared-memory ring
# ... and more than 16 rows of X (padded to a multiple of 16: the MMA's N dimension), full and ragged, up to
# the largest row count this kernel serves, with one or two TMA boxes per ring stage
SHAPES = [(16, 8, 8), (1, 64, 16), (5, 1184, 72), (16, 1192, 200), (16, 4096, 1024), (7, 20000, 264),
          (16, 148 * 8 * 17, 128), (16, 148 * 8 * 40 + 8, 64), (16, 2368, 4096), (3, 1184 * 13, 2048),
          (17, 8, 8), (32, 1192, 200), (27, 20000, 264), (24, 4096, 1024), (32, 148 * 8 * 17, 128),
          (19, 1184 * 13, 2048), (32, 2368, 4096),
          (33, 8, 8), (48, 1192, 200), (64, 4096, 1024), (80, 148 * 8 * 17, 128), (96, 20000, 264), (85, 2368, 4096),
          (96, 148 * 8 * 40 + 8, 64),
          # few rows of W per CTA: up to eight 64-k boxes per ring stage, full and ragged in K
          (16, 1184, 2048), (7, 2368, 1000), (40, 1184, 776), (16, 4096, 1536)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("red", [wk.RED_NONE, wk.RED_SUM, wk.RED_MAX])
def test_shapes_and_reductions(M, N, K, red):
    act = ACTS[(M + N + K + red) % len(ACTS)]
    wl = _case(M, N, K, act, red, seed=N + K, scale=0.75)
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp), f"act={act} red={red}")


def test_all_negative_rows_keep_their_maximum():
    wl = _case(16, 2048, 128, wk.ACT_IDENTITY, wk.RED_MAX, has_bias=False, seed=8)
    inp = wk.make_inputs(wl)
    inp["X"] = -np.abs(inp["X"])
    inp["W"] = np.abs(inp["W"])
    g, _ = pu.run_gpu(wl, inp)
    assert (g < 0).all()
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_repeatable_bits_and_back_to_back_runs():
    wl = _case(16, 8192, 512, wk.ACT_SILU, wk.RED_SUM, seed=3)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    a, _ = pu.run_gpu(wl, inp, op=op)
    b, _ = pu.run_gpu(wl, inp, op=op, repeats=4)      # four launches with no synchronisation between them
    op.close()
    assert np.array_equal(a, b)
    pu.assert_parity(wl, a, pu.run_oracle(wl, inp))


def test_row_tiles_follow_m():
    for M, rows in ((1, 16), (16, 16), (17, 32), (32, 32), (33, 48), (96, 96)):
        st, plan = B.forge_fused_linear_query_plan(pu.desc_of(_case(M, 4096, 256, wk.ACT_RELU, wk.RED_SUM)))
        assert st == B.FORGE_OK and plan.kernel == B.FORGE_KERNEL_BF16_SKINNY and plan.tile_m == rows
    st, plan = B.forge_fused_linear_query_plan(pu.desc_of(_case(97, 4096, 256, wk.ACT_RELU, wk.RED_SUM)))
    assert st == B.FORGE_OK and plan.kernel == B.FORGE_KERNEL_BF16_TCGEN05


def test_c4_full():
    wl = wk.WORKLOADS["c4"]
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == B.FORGE_KERNEL_BF16_SKINNY
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))
