"""Helpers of the GPU parity tests: move a workload's host inputs to the device, call the
C interface, bring the result back, and compare with the CPU oracle under the pass rule

    |g - r| <= tol * (|r| + s),   s = sqrt(mean(r^2)) over the compared reference values,

with tol = 1e-4 for fp32 storage (the tolerance of the paper's correctness test, Section
2.2) and 2e-2 for bf16 storage with fp32 accumulation.  The rms term keeps the rule
meaningful where activation outputs cross zero."""
from __future__ import annotations

import numpy as np

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

# fp16 storage: output rounding is 2^-11, the approximate activations dominate
TOL = {wk.F32: 1e-4, wk.BF16: 2e-2, wk.F16: 5e-3, wk.F32_TF32X3: 1e-4}


def to_device(a, dtype):
    import torch
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    if dtype == wk.BF16:
        t = t.to(torch.bfloat16)          # exact: the values are already bf16-representable
    elif dtype == wk.F16:
        t = t.to(torch.float16)
    return t.cuda()


def desc_of(wl: wk.Workload, M=None, device=0):
    return B.make_desc(wl.M if M is None else M, wl.N, wl.K, wl.dtype, wl.act, wl.red, wl.scale, wl.ln_eps,
                       wl.bias.kind != "none", device)


def run_gpu(wl: wk.Workload, inp, check_status=True, op=None, repeats=1):
    """``repeats`` calls through the C interface (no synchronisation between them); returns
    (float64 numpy result of the last one, plan dict)."""
    import torch
    dev = {k: to_device(v, wl.dtype) for k, v in inp.items() if k != "target"}
    M = inp["X"].shape[0]
    own = op is None
    if own:
        op = B.FusedLinear(desc_of(wl, M))
    if wl.out_cols == 0:
        out = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
    else:
        out = torch.full((M, wl.out_cols), float("nan"), dtype={wk.F32: torch.float32, wk.BF16: torch.bfloat16, wk.F16: torch.float16, wk.F32_TF32X3: torch.float32}[wl.dtype],
                         device="cuda")
    # the mean-gelu-residual chain takes its subtract vector, and the cross-entropy its int32
    # class indices, in the gamma slot of the interface
    aux = dev["sub"] if wl.red == wk.RED_MEAN_GELU_RESIDUAL else dev["gamma"]
    if wl.red == wk.RED_CROSS_ENTROPY:
        aux = torch.from_numpy(np.ascontiguousarray(inp["target"], dtype=np.int32)).cuda()
    for _ in range(repeats):
        op(dev["X"], dev["W"], dev["b"], aux, dev["beta"], out)
    torch.cuda.synchronize()
    if check_status:
        op.check()
    plan = op.plan.as_dict()
    if own:
        op.close()
    return out.float().cpu().numpy().astype(np.float64), plan


def run_oracle(wl: wk.Workload, inp, rows=None):
    import oracle
    return oracle.fused_linear(inp["X"], inp["W"], inp["b"], inp["gamma"], inp["beta"], act=wl.act,
                               scale=wl.scale, red=wl.red, eps=wl.ln_eps, rows=rows, sub=inp.get("sub"),
                               target=inp.get("target"))


def rel_err(g: np.ndarray, r: np.ndarray) -> float:
    """max |g-r| / (|r| + rms(r)); inf if g holds a non-finite value."""
    if not np.isfinite(g).all():
        return float("inf")
    s = float(np.sqrt(np.mean(r * r)))
    if s == 0.0:
        s = 1.0
    return float(np.max(np.abs(g - r) / (np.abs(r) + s)))


def assert_parity(wl: wk.Workload, g: np.ndarray, r: np.ndarray, what=""):
    e = rel_err(g, r)
    assert e <= TOL[wl.dtype], f"{wl.name} {what}: max relative error {e:.3e} > {TOL[wl.dtype]:.0e}"
    return e
