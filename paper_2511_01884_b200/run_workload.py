"""Run one of the five synthetic workloads a few times on cuda:0 and print the device time.

    python -m paper_2511_01884_b200.run_workload c3 --launches 5

A small, fixed launch sequence for use under a profiler (``ncu -k regex:... -s 3 -c 1``) or
for a quick timing; inputs come from the seeded generators, nothing else is computed.
"""
from __future__ import annotations

import argparse

import numpy as np

from . import binding as B
from . import workloads as wk


def main() -> int:
    ap = argparse.ArgumentParser()
    every = {**wk.WORKLOADS, **wk.EXTRA_WORKLOADS}
    ap.add_argument("workload", choices=sorted(every))
    ap.add_argument("--launches", type=int, default=5)
    ap.add_argument("--rows", type=int, default=0, help="use only the first ROWS rows of X (smaller case)")
    args = ap.parse_args()
    import torch
    wl = every[args.workload]
    M = args.rows or wl.M
    inp = wk.make_inputs(wl, M=M)

    def dev(a):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        return (t.to(torch.bfloat16) if wl.dtype == wk.BF16 else t).cuda()
    d = {k: dev(v) for k, v in inp.items() if k != "target"}
    if wl.red == wk.RED_CROSS_ENTROPY:     # int32 class indices travel in the gamma slot
        d["gamma"] = torch.from_numpy(np.ascontiguousarray(inp["target"], dtype=np.int32)).cuda()
    reduce = wl.out_cols == 0
    out = torch.empty((M,) if reduce else (M, wl.out_cols), device="cuda",
                      dtype=torch.float32 if (reduce or wl.dtype != wk.BF16) else torch.bfloat16)
    if wl.red == wk.RED_MEAN_GELU_RESIDUAL:
        d["gamma"] = d["sub"]          # the chain's subtract vector travels in the gamma slot
    op = B.FusedLinear(B.make_desc(M, wl.N, wl.K, wl.dtype, wl.act, wl.red, wl.scale, wl.ln_eps,
                                   wl.bias.kind != "none", 0))
    torch.cuda.synchronize()
    times = []
    for _ in range(args.launches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        op(d["X"], d["W"], d["b"], d["gamma"], d["beta"], out)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    op.check()
    print(f"{wl.name} M={M} N={wl.N} K={wl.K} kernel={B.kernel_name(op.plan.kernel)} "
          f"us per launch: {', '.join(f'{t:.1f}' for t in times)}")
    op.close()
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
