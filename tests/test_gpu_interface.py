"""GPU-side behaviour of the C interface itself: argument checks in run(), the host-buffer entry
point, unaligned fp32 operands, handles on a non-default stream, plan/launch bookkeeping."""
import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu


def test_run_rejects_missing_and_misaligned_pointers():
    import torch
    wl = wk.custom_workload("iface_bf16", wk.BF16, 64, 64, 64, wk.ACT_RELU, wk.RED_LAYERNORM)
    op = B.FusedLinear(pu.desc_of(wl))
    t = torch.zeros(64 * 64 + 8, dtype=torch.bfloat16, device="cuda")
    v = torch.zeros(64 + 8, dtype=torch.bfloat16, device="cuda")
    ok = (t, t, v, v, v, t)
    assert B.forge_fused_linear_run(op.h, *ok) == B.FORGE_OK
    for i in range(6):                                             # each pointer missing in turn
        args = list(ok)
        args[i] = None
        assert B.forge_fused_linear_run(op.h, *args) == B.FORGE_ERR_INVALID_ARG, i
    off = t[1:]                                                    # 2-byte offset: not 16-byte aligned
    assert B.forge_fused_linear_run(op.h, off, t, v, v, v, t) == B.FORGE_ERR_INVALID_ARG
    assert B.forge_fused_linear_run(op.h, t, t, v, v, v, off) == B.FORGE_ERR_INVALID_ARG
    torch.cuda.synchronize()
    op.check()
    op.close()
    assert B.forge_fused_linear_launches_per_run(None) == 0


def test_fp32_accepts_unaligned_operands_with_scalar_accesses():
    import torch
    wl = wk.custom_workload("iface_f32", wk.F32, 70, 50, 36, wk.ACT_SILU, wk.RED_NONE, seed=5)
    inp = wk.make_inputs(wl)
    op = B.FusedLinear(pu.desc_of(wl))
    assert B.forge_fused_linear_launches_per_run(op.h) == 1

    def shifted(a):                                                # same values, 4-byte-aligned only
        buf = torch.zeros(a.size + 1, dtype=torch.float32, device="cuda")
        buf[1:] = torch.from_numpy(a.ravel())
        return buf[1:]
    X, W, b = shifted(inp["X"]), shifted(inp["W"]), shifted(inp["b"])
    obuf = torch.full((70 * 50 + 1,), float("nan"), dtype=torch.float32, device="cuda")
    out = obuf[1:]
    assert X.data_ptr() % 16 != 0 and out.data_ptr() % 16 != 0
    assert B.forge_fused_linear_run(op.h, X, W, b, None, None, out) == B.FORGE_OK
    torch.cuda.synchronize()
    op.close()
    g = out.cpu().numpy().astype(np.float64).reshape(70, 50)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))
    assert np.isnan(obuf[0].item())                                # nothing written in front of the output


@pytest.mark.parametrize("name", ["c1", "skinny", "ln", "plain", "chain", "ce"])
def test_host_buffer_entry_point_matches_the_oracle(name):
    import torch
    wl = {"c1": wk.WORKLOADS["c1"],
          "skinny": wk.custom_workload("h_skinny", wk.BF16, 16, 1024, 256, wk.ACT_GELU_ERF, wk.RED_MAX, w_std=0.05),
          "ln": wk.custom_workload("h_ln", wk.BF16, 300, 520, 128, wk.ACT_GELU_TANH, wk.RED_LAYERNORM, w_std=0.05),
          "plain": wk.custom_workload("h_plain", wk.BF16, 300, 520, 128, wk.ACT_SILU, wk.RED_NONE, w_std=0.05),
          "chain": wk.custom_workload("h_chain", wk.F32, 150, 300, 40, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL),
          "ce": wk.custom_workload("h_ce", wk.BF16, 300, 1032, 128, wk.ACT_IDENTITY, wk.RED_CROSS_ENTROPY, w_std=0.05)}[name]
    inp = wk.make_inputs(wl)

    def host(a):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        return (t.to(torch.bfloat16) if wl.dtype == wk.BF16 else t).pin_memory()
    h = {k: host(v) for k, v in inp.items() if k != "target"}
    aux = h["sub"] if wl.red == wk.RED_MEAN_GELU_RESIDUAL else h["gamma"]
    if wl.red == wk.RED_CROSS_ENTROPY:
        aux = torch.from_numpy(np.ascontiguousarray(inp["target"], dtype=np.int32)).pin_memory()
    shape = (wl.M,) if wl.out_cols == 0 else (wl.M, wl.out_cols)
    out = torch.zeros(shape, dtype=torch.float32 if (wl.out_cols == 0 or wl.dtype == wk.F32) else torch.bfloat16).pin_memory()
    op = B.FusedLinear(pu.desc_of(wl))
    for _ in range(2):                                             # second call reuses the staging buffers
        op.run_host(h["X"], h["W"], h["b"], aux, h["beta"], out)
    op.check()
    op.close()
    pu.assert_parity(wl, out.float().numpy().astype(np.float64), pu.run_oracle(wl, inp))


@pytest.mark.parametrize("name", ["plain", "ln", "ce", "f32_sum", "f32_chain"])
def test_host_entry_point_in_row_blocks_matches_the_oracle(name):
    """Large X: the host entry point uploads, computes and downloads in blocks of rows on three
    streams (here 4 blocks of 512 rows and a last one of 252)."""
    import torch
    M = 2300
    wl = {"plain": wk.custom_workload("hp_plain", wk.BF16, M, 520, 2048, wk.ACT_SILU, wk.RED_NONE, w_std=0.03),
          "ln": wk.custom_workload("hp_ln", wk.BF16, M, 520, 2048, wk.ACT_GELU_TANH, wk.RED_LAYERNORM, w_std=0.03),
          "ce": wk.custom_workload("hp_ce", wk.BF16, M, 1032, 2048, wk.ACT_IDENTITY, wk.RED_CROSS_ENTROPY, w_std=0.03),
          "f32_sum": wk.custom_workload("hp_sum", wk.F32, M, 300, 1024, wk.ACT_RELU, wk.RED_SUM),
          "f32_chain": wk.custom_workload("hp_chain", wk.F32, M, 200, 1024, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL)}[name]
    inp = wk.make_inputs(wl)

    def host(a):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        return (t.to(torch.bfloat16) if wl.dtype == wk.BF16 else t).pin_memory()
    h = {k: host(v) for k, v in inp.items() if k != "target"}
    aux = h["sub"] if wl.red == wk.RED_MEAN_GELU_RESIDUAL else h["gamma"]
    if wl.red == wk.RED_CROSS_ENTROPY:
        aux = torch.from_numpy(np.ascontiguousarray(inp["target"], dtype=np.int32)).pin_memory()
    shape = (M,) if wl.out_cols == 0 else (M, wl.out_cols)
    out = torch.full(shape, float("nan"), dtype=torch.float32 if (wl.out_cols == 0 or wl.dtype == wk.F32) else torch.bfloat16).pin_memory()
    op = B.FusedLinear(pu.desc_of(wl))
    for _ in range(2):
        op.run_host(h["X"], h["W"], h["b"], aux, h["beta"], out)
    op.check()
    # the same handle's device entry point on the whole problem agrees far inside the tolerance (not to the
    # bit: a block of rows has fewer tiles than the whole problem, so its K range may be cut differently)
    dev = {k: (None if v is None else v.cuda()) for k, v in h.items()}
    dout = torch.empty(shape, dtype=out.dtype, device="cuda")
    op(dev["X"], dev["W"], dev["b"], None if aux is None else aux.cuda(), dev["beta"], dout)
    torch.cuda.synchronize()
    op.check()
    op.close()
    assert pu.rel_err(out.float().numpy().astype(np.float64), dout.float().cpu().numpy().astype(np.float64)) <= pu.TOL[wl.dtype] / 10
    rows = np.unique(np.concatenate([np.arange(0, M, 97), np.array([511, 512, 2047, 2048, M - 1])]))
    pu.assert_parity(wl, out.float().numpy().astype(np.float64)[rows], pu.run_oracle(wl, inp, rows=rows))


def test_runs_on_a_side_stream():
    import torch
    wl = wk.custom_workload("iface_stream", wk.BF16, 512, 512, 256, wk.ACT_SILU, wk.RED_SUM, w_std=0.05, seed=7)
    inp = wk.make_inputs(wl)
    dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items()}
    out = torch.zeros(512, dtype=torch.float32, device="cuda")
    op = B.FusedLinear(pu.desc_of(wl))
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        op(dev["X"], dev["W"], dev["b"], None, None, out, stream=s.cuda_stream)
    s.synchronize()
    op.check()
    op.close()
    pu.assert_parity(wl, out.cpu().numpy().astype(np.float64), pu.run_oracle(wl, inp))


def test_plans_report_the_kernel_families():
    for wl, kernel, cluster in [(wk.WORKLOADS["c2"], B.FORGE_KERNEL_F32_FFMA, 1),
                                (wk.WORKLOADS["c3"], B.FORGE_KERNEL_BF16_TCGEN05, 2),
                                (wk.WORKLOADS["c4"], B.FORGE_KERNEL_BF16_SKINNY, 1),
                                (wk.WORKLOADS["c5"], B.FORGE_KERNEL_BF16_TCGEN05_LN, 2)]:
        st, p = B.forge_fused_linear_query_plan(pu.desc_of(wl))
        assert st == B.FORGE_OK and p.kernel == kernel and p.cluster == cluster
        assert p.grid <= 148 or kernel == B.FORGE_KERNEL_F32_FFMA          # the bf16 kernels are persistent


def test_a_wait_that_nothing_satisfies_gives_up_and_reports():
    """The give-up path of the bounded waits, exercised the safe way: a barrier nobody signals and a
    50 ms budget.  The kernel must end by itself, report the time-out, and leave the GPU usable."""
    import time
    import torch
    t = time.perf_counter()
    st, detail = B.forge_selftest_bounded_wait(0, 50)
    dt = time.perf_counter() - t
    assert st == B.FORGE_ERR_TIMEOUT and detail == [1, 0x5A5A, 0, 32]
    assert 0.04 < dt < 2.0
    # the context is intact: an ordinary run right after it is correct
    wl = wk.WORKLOADS["c1"]
    inp = wk.make_inputs(wl)
    g, _ = pu.run_gpu(wl, inp)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))
    assert B.forge_selftest_bounded_wait(0, 0)[0] == B.FORGE_ERR_INVALID_ARG
    assert torch.cuda.is_available()


def test_two_handles_on_two_streams_do_not_disturb_each_other():
    """Every handle owns its workspace (partials, counters, hand-over areas), so launches of different
    handles may overlap on the GPU; the kernels whose CTAs wait on one another are launched
    cooperatively and simply take turns."""
    import torch
    cases = [wk.custom_workload("two_a", wk.BF16, 300, 520, 4096, wk.ACT_SILU, wk.RED_SUM, w_std=0.02, seed=1),      # K split, CTA pairs
             wk.custom_workload("two_b", wk.BF16, 700, 1032, 256, wk.ACT_GELU_TANH, wk.RED_LAYERNORM, w_std=0.05, seed=2),
             wk.custom_workload("two_c", wk.F32_TF32X3, 300, 520, 2048, wk.ACT_RELU, wk.RED_MAX, seed=3),
             wk.custom_workload("two_d", wk.F32, 200, 300, 96, wk.ACT_GELU_ERF, wk.RED_SUM, seed=4)]
    work = []
    for wl in cases:
        inp = wk.make_inputs(wl)
        dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items() if k != "target"}
        shape = (wl.M,) if wl.out_cols == 0 else (wl.M, wl.out_cols)
        odt = torch.float32 if (wl.out_cols == 0 or wl.dtype != wk.BF16) else torch.bfloat16
        work.append((wl, inp, dev, torch.full(shape, float("nan"), dtype=odt, device="cuda"), B.FusedLinear(pu.desc_of(wl)), torch.cuda.Stream()))
    torch.cuda.synchronize()
    for _ in range(5):
        for wl, inp, dev, out, op, st in work:
            op(dev["X"], dev["W"], dev["b"], dev["gamma"], dev["beta"], out, stream=st.cuda_stream)
    torch.cuda.synchronize()
    for wl, inp, dev, out, op, st in work:
        op.check()
        op.close()
        pu.assert_parity(wl, out.float().cpu().numpy().astype(np.float64), pu.run_oracle(wl, inp), wl.name)


def test_bound_call_is_the_same_call():
    import torch
    wl = wk.WORKLOADS["c1"]
    inp = wk.make_inputs(wl)
    dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items() if k != "target"}
    a = torch.zeros(wl.M, device="cuda")
    b = torch.zeros(wl.M, device="cuda")
    op = B.FusedLinear(pu.desc_of(wl))
    op(dev["X"], dev["W"], dev["b"], None, None, a)
    step = op.bind(dev["X"], dev["W"], dev["b"], None, None, b)
    step()
    step()
    torch.cuda.synchronize()
    op.check()
    op.close()
    assert torch.equal(a, b)
    pu.assert_parity(wl, b.cpu().numpy().astype(np.float64), pu.run_oracle(wl, inp))


@pytest.mark.parametrize("case", ["f32", "f32_sliced", "tf32x3", "tf32x3_ln", "bf16_pair", "bf16_ksplit", "bf16_ln", "skinny", "f16", "chain_bf16"])
def test_nothing_is_written_outside_the_output(case):
    """Every kernel family on a ragged shape, with the output in the middle of a larger buffer whose
    guard zones must keep their pattern (stores past a row end, a tile edge or the last row would
    land there)."""
    import torch
    M, N, K, dt, act, red = {
        "f32": (129, 257, 33, wk.F32, wk.ACT_GELU_ERF, wk.RED_NONE),
        "f32_sliced": (100, 204, 520, wk.F32, wk.ACT_RELU, wk.RED_NONE),
        "tf32x3": (300, 516, 132, wk.F32_TF32X3, wk.ACT_SILU, wk.RED_NONE),
        "tf32x3_ln": (300, 516, 132, wk.F32_TF32X3, wk.ACT_GELU_TANH, wk.RED_LAYERNORM),
        "bf16_pair": (300, 520, 136, wk.BF16, wk.ACT_SILU, wk.RED_NONE),
        "bf16_ksplit": (100, 520, 4096, wk.BF16, wk.ACT_GELU_TANH, wk.RED_NONE),
        "bf16_ln": (300, 520, 136, wk.BF16, wk.ACT_GELU_TANH, wk.RED_LAYERNORM),
        "skinny": (20, 1032, 520, wk.BF16, wk.ACT_GELU_ERF, wk.RED_NONE),
        "f16": (150, 264, 72, wk.F16, wk.ACT_RELU, wk.RED_NONE),
        "chain_bf16": (300, 520, 136, wk.BF16, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL),
    }[case]
    wl = wk.custom_workload("guard_" + case, dt, M, N, K, act, red, seed=len(case), w_std=0.05 if dt in (wk.BF16, wk.F16) else None)
    inp = wk.make_inputs(wl)
    dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items() if k != "target"}
    odt = {wk.F32: torch.float32, wk.F32_TF32X3: torch.float32, wk.BF16: torch.bfloat16, wk.F16: torch.float16}[dt]
    n_out, guard = M * wl.out_cols, 4096
    buf = torch.full((guard + n_out + guard,), 12345.0, dtype=odt, device="cuda")
    out = buf[guard:guard + n_out].view(M, wl.out_cols)
    aux = dev["sub"] if red == wk.RED_MEAN_GELU_RESIDUAL else dev["gamma"]
    op = B.FusedLinear(pu.desc_of(wl))
    op(dev["X"], dev["W"], dev["b"], aux, dev["beta"], out)
    torch.cuda.synchronize()
    op.check()
    op.close()
    assert bool((buf[:guard] == 12345.0).all()) and bool((buf[guard + n_out:] == 12345.0).all())
    pu.assert_parity(wl, out.float().cpu().numpy().astype(np.float64), pu.run_oracle(wl, inp))


@pytest.mark.parametrize("name", ["ln_bf16", "chain_bf16", "tailsplit_bf16", "ln_tf32x3", "rowsum_f32", "ln_f32", "ln_bf16_two_pass"])
def test_run_captured_in_a_graph_replays_correctly(name):
    """run() keeps no per-call state on the host: the counters that the CTAs of the LayerNorm, chain
    and K-cut launches wait on take their run index from device memory.  So a run captured into a
    CUDA graph and replayed (with other direct runs on the same handle in between) gives the same
    bits as a direct run."""
    import torch
    wl = {"ln_bf16": wk.custom_workload("g_ln", wk.BF16, 300, 1032, 128, wk.ACT_GELU_TANH, wk.RED_LAYERNORM, w_std=0.05),
          "chain_bf16": wk.custom_workload("g_chain", wk.BF16, 300, 520, 128, wk.ACT_IDENTITY, wk.RED_MEAN_GELU_RESIDUAL, w_std=0.05),
          "tailsplit_bf16": wk.custom_workload("g_tail", wk.BF16, 256, 512, 4096, wk.ACT_SILU, wk.RED_NONE, w_std=0.02),
          "ln_tf32x3": wk.custom_workload("g_ln5", wk.F32_TF32X3, 300, 520, 256, wk.ACT_GELU_TANH, wk.RED_LAYERNORM),
          "rowsum_f32": wk.custom_workload("g_sum", wk.F32, 300, 700, 96, wk.ACT_RELU, wk.RED_SUM),
          "ln_f32": wk.custom_workload("g_ln1", wk.F32, 300, 1300, 96, wk.ACT_GELU_TANH, wk.RED_LAYERNORM),
          "ln_bf16_two_pass": wk.custom_workload("g_ln2", wk.BF16, 130, 256 * 80, 64, wk.ACT_SILU, wk.RED_LAYERNORM, w_std=0.05)}[name]
    inp = wk.make_inputs(wl)
    dev = {k: pu.to_device(v, wl.dtype) for k, v in inp.items() if k != "target"}
    aux = dev["sub"] if wl.red == wk.RED_MEAN_GELU_RESIDUAL else dev["gamma"]
    dt = {wk.F32: torch.float32, wk.BF16: torch.bfloat16, wk.F32_TF32X3: torch.float32}[wl.dtype]
    shape = (wl.M,) if wl.out_cols == 0 else (wl.M, wl.out_cols)
    direct = torch.full(shape, float("nan"), dtype=torch.float32 if wl.out_cols == 0 else dt, device="cuda")
    replay = torch.full_like(direct, float("nan"))
    op = B.FusedLinear(pu.desc_of(wl))
    op(dev["X"], dev["W"], dev["b"], aux, dev["beta"], direct)            # first use outside any capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            op(dev["X"], dev["W"], dev["b"], aux, dev["beta"], replay, stream=side.cuda_stream)
    torch.cuda.synchronize()
    for i in range(3):
        replay.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(replay, direct), (name, i)
        op(dev["X"], dev["W"], dev["b"], aux, dev["beta"], direct)        # a direct run between the replays
        torch.cuda.synchronize()
    op.check()
    op.close()
    g = replay.float().cpu().numpy().astype(np.float64)
    pu.assert_parity(wl, g, pu.run_oracle(wl, inp))


def test_kernel_name_of_a_handle():
    wl = wk.custom_workload("kn", wk.BF16, 16, 1024, 256, wk.ACT_GELU_ERF, wk.RED_MAX, w_std=0.05)
    op = B.FusedLinear(pu.desc_of(wl))
    assert B.forge_fused_linear_kernel_name(op.h) == B.kernel_name(op.plan.kernel) == "bf16_skinny_swapab_tcgen05"
    op.close()


def test_measured_read_stream_is_plausible():
    st, b2b, single = B.forge_selftest_read_stream(0)
    assert st == B.FORGE_OK
    assert 4000.0 < b2b < 8000.0 and 3500.0 < single <= 1.02 * b2b, (b2b, single)      # GB/s; nominal HBM3e: 8000


def test_measured_ffma_rate_is_plausible():
    import torch
    st, tflops, mhz = B.forge_selftest_ffma_rate(0, 50)
    assert st == B.FORGE_OK
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nominal = sms * 128 * 2 * 1.965e9 / 1e12
    assert 0.5 * nominal < tflops < 1.05 * nominal, (tflops, nominal)
    assert 900.0 < mhz < 2100.0
