"""The entry point that allocates nothing: forge_fused_linear_f32_reduce_static().

Some users of this library cannot allocate device memory at the moment they need a result
(they run inside another component's memory pool or under a fixed budget, or sit in a
latency-critical loop where cudaMalloc's device-wide synchronisation is unacceptable).  For
them the fp32 row sum / max is also offered with its scratch in a fixed array inside the
library.  This test drives that entry point through the C interface and checks it against
the ordinary handle-based path on the same inputs, twice in a row (the array is shared by
all calls and keeps the previous call's contents, so the second call is the one that shows
whether stale state is cleared), and checks that a problem beyond the array is refused.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu


def _both_paths(wl, inp):
    import torch
    dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items()}
    M = inp["X"].shape[0]
    want, _ = pu.run_gpu(wl, inp)                                   # handle-based path (allocates its workspace)
    got = []
    for _ in range(2):                                              # two calls in a row share the static array
        out = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
        st = B.forge_fused_linear_f32_reduce_static(M, wl.N, wl.K, wl.act, wl.red, wl.scale,
                                                    dev["X"], dev["W"], dev["b"], out)
        assert st == B.FORGE_OK, B.status_string(st)
        torch.cuda.synchronize()
        got.append(out.cpu().numpy().astype(np.float64))
    return want, got


@pytest.mark.parametrize("red", [wk.RED_SUM, wk.RED_MAX])
def test_static_scratch_matches_handle_path_twice(red):
    # 3 row strips x 6 column tiles with ragged edges: partials and arrival counters are in use
    wl = wk.custom_workload("noalloc", wk.F32, 300, 700, 96, wk.ACT_GELU_TANH, red, scale=0.5, seed=11)
    inp = wk.make_inputs(wl)
    want, got = _both_paths(wl, inp)
    ref = pu.run_oracle(wl, inp)
    for g in got:
        assert pu.rel_err(g, want) <= pu.TOL[wk.F32]                # same tolerance as the parity tests
        pu.assert_parity(wl, g, ref)
    assert np.array_equal(got[0], got[1])


def test_c1_through_static_scratch():
    wl = wk.WORKLOADS["c1"]
    inp = wk.make_inputs(wl)
    want, got = _both_paths(wl, inp)
    for g in got:
        assert pu.rel_err(g, want) <= pu.TOL[wk.F32]


def test_calls_allocate_no_device_memory_and_bias_is_optional():
    """What the entry point is for: after the first call on the device (which looks the array's address
    up) further calls leave the amount of free device memory exactly as it was.  Also: b = NULL means
    no bias."""
    import torch
    wl = wk.custom_workload("noalloc_nobias", wk.F32, 300, 700, 96, wk.ACT_SILU, wk.RED_SUM, seed=12, has_bias=False)
    inp = wk.make_inputs(wl)
    assert inp["b"] is None
    dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items()}
    out = torch.full((wl.M,), float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        st = B.forge_fused_linear_f32_reduce_static(wl.M, wl.N, wl.K, wl.act, wl.red, wl.scale, dev["X"], dev["W"], None, out, stream)
        assert st == B.FORGE_OK, B.status_string(st)
    call()                                                          # first call on this device: symbol lookup
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        call()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    pu.assert_parity(wl, out.cpu().numpy().astype(np.float64), pu.run_oracle(wl, inp))


def test_sizes_beyond_the_array_are_refused():
    import torch
    x = torch.zeros(16, device="cuda")
    # 4 * M * ceil(N/128) bytes of partials > 1 MiB
    M, N = 4096, 128 * 65
    assert 4 * M * 65 > B.FORGE_STATIC_SCRATCH_BYTES
    st = B.forge_fused_linear_f32_reduce_static(M, N, 8, wk.ACT_RELU, wk.RED_SUM, 1.0, x, x, None, x)
    assert st == B.FORGE_ERR_SCRATCH_LIMIT
    assert "scratch" in B.status_string(st)
    st = B.forge_fused_linear_f32_reduce_static(8, 8, 8, wk.ACT_RELU, wk.RED_NONE, 1.0, x, x, None, x)
    assert st == B.FORGE_ERR_INVALID_ARG                             # only row sum / max are offered here
