#!/usr/bin/env python
"""Benchmark of the fused linear operator on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl reference]

One "step" is one pass of the whole hot path (operand fetch, contraction, bias, activation,
scale, row reduction, store: a single kernel launch) over one batch of seeded synthetic
input.  The headline workload is C3 (bf16, M=N=K=8192, SiLU); at N=1 the line also carries
short measurements of the other four workloads under "workloads".  With N>1 (launched by
torch.distributed.run, one rank per GPU) every rank runs the workload on its own block of
rows of a global X (rows are independent: no collective on the data path) and the value is
the aggregate over ranks of work / max-over-ranks time.

Timing: CUDA events on the stream the kernels are launched on, after >= 3 warm-up steps,
barrier + synchronize on both sides.  L2: the operands of C2, C3, C5 exceed the 126 MB L2 and
those kernels are compute-bound; C4 (HBM-bound: the whole cost is streaming W once) rotates
through three distinct copies of W (768 MiB) so that no byte of a W can still be in L2 when it
is read again; C1 fits in L2 and is timed with an L2 flush (a 256 MiB write) before every call.

    python bench.py --workload c5 --kernel-only --steps 4 [--rows R]

launches the workload's kernel a few times (each launch timed alone) and nothing else: the
fixed launch sequence to put under a profiler, R rows of X for a small case.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2511_01884_b200 import multigpu  # noqa: E402
from paper_2511_01884_b200 import workloads as wk  # noqa: E402

HEADLINE = "c3"
ALL_WORKLOADS = {**wk.WORKLOADS, **wk.EXTRA_WORKLOADS}
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}
TF32_OVER_BF16 = 1.1 / 2.25          # nominal dense tensor peaks, TF32 : bf16
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# Per-launch DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel
# from the ncu captures summarised under profiles/, keyed by workload, with the sha256 of the
# kernel source the capture was taken from.  A changed source invalidates the figure (-> null).
NCU_TRAFFIC = {
    "c2": {"bytes": 556_733_184, "sha": "a8edcb07ff7a7bdb"},
    "c3": {"bytes": 1_001_968_384, "sha": "ab482763f83be5c8"},
    "c4": {"bytes": 273_245_696, "sha": "7f82c84d18aa5daf"},
    "c5": {"bytes": 326_729_728, "sha": "ab482763f83be5c8"},
    "c2t": {"bytes": 304_342_528, "sha": "29bae20a963fe65f"},
    "n2": {"bytes": 876_474_368, "sha": "ab482763f83be5c8"},
    "m64": {"bytes": 554_519_552, "sha": "7f82c84d18aa5daf"},
    "n1b": {"bytes": 1_025_926_656, "sha": "ab482763f83be5c8"},
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def source_digest(text: str) -> str:
    """Hash of a source text with comments and blank space removed: a reworded comment does not
    make the traffic counters stale, a changed statement does."""
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    return hashlib.sha256("".join(text.split()).encode()).hexdigest()[:16]


def kernel_source_hash(kernel: int) -> str:
    name = {1: "k1_f32_ffma.cu", 2: "k2_bf16_tcgen05.cu", 3: "k3_bf16_skinny.cu", 4: "k2_bf16_tcgen05.cu",
            5: "k5_f32_tf32x3.cu"}[kernel]
    with open(os.path.join(ROOT, "paper_2511_01884_b200", "csrc", name), "r") as f:
        return source_digest(f.read())


# ---- clocks during the timed region (NVML; nvidia-smi as a fallback) -------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if self._nv is None or not self.samples:
            return self._smi_once()
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples), "how": "nvml during the timed region"}

    def _smi_once(self):
        import subprocess
        try:
            out = subprocess.run(["nvidia-smi", f"--id={self.index}", "--query-gpu=clocks.sm,clocks.max.sm",
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
            a, b = [float(t) for t in out.strip().split(",")]
            return {"sm_mhz": a, "sm_max_mhz": b, "reasons": [], "samples": 1, "how": "nvidia-smi after the timed region"}
        except Exception:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "how": "unavailable"}


# ---- device-side measurement ---------------------------------------------------------------------
def device_tensors(wl, inp, torch):
    def dev(a):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
        return (t.to(torch.bfloat16) if wl.dtype == wk.BF16 else t).cuda()
    d = {k: dev(v) for k, v in inp.items() if k != "target"}
    M = inp["X"].shape[0]
    if wl.red == wk.RED_CROSS_ENTROPY:     # the int32 class indices travel in the gamma slot of the interface
        d["gamma"] = torch.from_numpy(np.ascontiguousarray(inp["target"], dtype=np.int32)).cuda()
    if wl.out_cols == 0:
        d["out"] = torch.empty((M,), dtype=torch.float32, device="cuda")
    else:
        d["out"] = torch.empty((M, wl.out_cols), dtype=torch.bfloat16 if wl.dtype == wk.BF16 else torch.float32, device="cuda")
    if wl.red == wk.RED_MEAN_GELU_RESIDUAL:
        d["gamma"] = d["sub"]          # the chain's subtract vector travels in the gamma slot of the interface
    return d


def make_op(wl, M, device):
    from paper_2511_01884_b200 import binding as B
    return B.FusedLinear(B.make_desc(M, wl.N, wl.K, wl.dtype, wl.act, wl.red, wl.scale, wl.ln_eps,
                                     wl.bias.kind != "none", device))


class Rotation:
    """The step callables of one workload.  Normally one handle bound to one set of buffers.  For the
    HBM-bound workload: `copies` handles, each bound to its own copy of W (its tensor map is encoded
    once), called in turn, so that a W is read again only after the other copies -- several times the
    L2 -- have streamed through."""

    def __init__(self, wl, d, device, torch, copies=1):
        self.ops, self.steps, self.keep = [], [], []
        for i in range(copies):
            W = d["W"] if i == 0 else d["W"].clone()
            op = make_op(wl, d["X"].shape[0], device)
            self.ops.append(op)
            self.keep.append(W)
            self.steps.append(op.bind(d["X"], W, d["b"], d["gamma"], d["beta"], d["out"]))
        self.w_bytes = sum(w.numel() * w.element_size() for w in self.keep)
        self.i = 0

    def step(self):
        self.steps[self.i]()
        self.i = (self.i + 1) % len(self.steps)

    def check(self):
        for op in self.ops:
            op.check()

    def close(self):
        for op in self.ops:
            op.close()
        self.keep = []

    @property
    def plan(self):
        return self.ops[0].plan


def w_copies(wl):
    """Distinct copies of W the timed loop rotates through (only the HBM-bound workload needs more than one)."""
    return 3 if wl.hbm_bound else 1


def time_steps(rot, steps, warmup, torch, flush_buf=None, barrier=None):
    """Average device milliseconds per step over exactly `steps` steps (CUDA events on the
    launching stream).  With flush_buf every step is bracketed by its own events and L2 is
    overwritten before it.  The calls go through a pre-bound forge_fused_linear_run (pointers
    marshalled once), so the host side of a step is one foreign-function call."""
    for _ in range(warmup):
        rot.step()
    torch.cuda.synchronize()
    rot.check()
    if barrier:
        barrier()
    torch.cuda.synchronize()
    if flush_buf is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            rot.step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
    else:
        tot = 0.0
        for _ in range(steps):
            flush_buf.fill_(1.0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            rot.step()
            e1.record()
            torch.cuda.synchronize()
            tot += e0.elapsed_time(e1)
        ms = tot / steps
    if barrier:
        barrier()
    torch.cuda.synchronize()
    rot.check()
    return ms


def isolated_us(rot, torch, calls=30):
    """Microseconds of one call with nothing before or after it on the device (a synchronise after every
    call): no overlap with a neighbour's start-up or tail.  Median and minimum over `calls` calls."""
    ts = []
    for _ in range(calls):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rot.step()
        e1.record()
        torch.cuda.synchronize()
        ts.append(1e3 * e0.elapsed_time(e1))
    rot.check()
    return statistics.median(ts), min(ts)


def sustained_block(rot, wl, peaks, local, torch, seconds=2.5):
    """Back-to-back launches for `seconds` of device time: what the kernel holds once the GPU has settled
    at the clock its power limit allows, with the clocks sampled meanwhile."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        rot.step()
    e1.record()
    torch.cuda.synchronize()
    n = max(50, int(seconds * 1e3 / max(e0.elapsed_time(e1) / 20, 1e-3)))
    with ClockSampler(local, period_s=0.02) as cs:
        e0.record()
        for _ in range(n):
            rot.step()
        e1.record()
        torch.cuda.synchronize()
    rot.check()
    ms = e0.elapsed_time(e1) / n
    v, u = unit_value(wl, ms)
    key = "hbm_gbs" if wl.hbm_bound else "bf16_tflops_sustained"
    blk = {"steps": n, "seconds": round(ms * n / 1e3, 3), "ms_per_step": round(ms, 5), "value": round(v, 2), "unit": u,
           "clocks": cs.summary()}
    if wl.dtype == wk.BF16 and peaks.get(key):
        blk["frac_of_sustained_peak"] = round(v / peaks[key], 4)
        blk["peak"] = peaks[key]
        blk["note"] = f"peak = {key} of {peaks['_source']}"
    return blk, n


def back_to_back_us(rot, torch, calls=1000):
    """Microseconds per call of `calls` calls issued without anything in between (operands stay in
    L2): what a latency-bound problem costs inside a stream of work."""
    for _ in range(20):
        rot.step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(calls):
        rot.step()
    e1.record()
    torch.cuda.synchronize()
    rot.check()
    return 1e3 * e0.elapsed_time(e1) / calls


def eager_context_us(wl, d, torch, steps=10):
    """PyTorch eager on the same GPU, the unfused operator chain in the workload's dtype: context
    only (a library path, never part of this package's hot path).  Microseconds per call."""
    import torch.nn.functional as F

    def chain():
        z = F.linear(d["X"], d["W"], d["b"])
        if wl.act == wk.ACT_RELU:
            z = F.relu(z)
        elif wl.act == wk.ACT_GELU_ERF:
            z = F.gelu(z)
        elif wl.act == wk.ACT_GELU_TANH:
            z = F.gelu(z, approximate="tanh")
        elif wl.act == wk.ACT_SILU:
            z = F.silu(z)
        if wl.scale != 1.0:
            z = z * wl.scale
        if wl.red == wk.RED_SUM:
            return z.sum(1, dtype=torch.float32)
        if wl.red == wk.RED_MAX:
            return z.amax(1).float()
        if wl.red == wk.RED_LAYERNORM:
            return F.layer_norm(z, (wl.N,), d["gamma"], d["beta"], wl.ln_eps)
        if wl.red == wk.RED_MEAN_GELU_RESIDUAL:
            return d["X"] + F.gelu((z - d["gamma"]).mean(1, keepdim=True))
        if wl.red == wk.RED_LOGSUMEXP:
            return torch.logsumexp(z.float(), 1)
        if wl.red == wk.RED_CROSS_ENTROPY:
            return F.cross_entropy(z.float(), d["gamma"].long(), reduction="none")
        return z
    for _ in range(3):
        chain()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        chain()
    e1.record()
    torch.cuda.synchronize()
    return 1e3 * e0.elapsed_time(e1) / steps


def roofline_of(wl, ms, peaks, kernel, sm_max_mhz, sm_count, alu_peak=None):
    """Roofline of the (single) kernel of a step: achieved = algorithmic work / measured time."""
    src = peaks["_source"]
    if wl.hbm_bound:
        ach = wl.algorithmic_bytes / ms / 1e6
        peak, unit, bound = peaks["hbm_gbs"], "GB/s", "hbm"
        note = f"{wl.algorithmic_bytes} algorithmic bytes per launch; peak = copy bandwidth, of {src}"
    elif wl.dtype == wk.BF16:
        ach = wl.flops / ms / 1e9
        peak, unit, bound = peaks["bf16_tflops"], "TFLOP/s", "tensor"
        note = f"2MNK = {wl.flops} flops per launch; peak = cuBLAS bf16 burst, of {src}"
    elif wl.dtype == wk.F32_TF32X3:
        ach = wl.flops / ms / 1e9
        peak, unit, bound = peaks["bf16_tflops"] * TF32_OVER_BF16, "TFLOP/s", "tensor"
        note = (f"2MNK = {wl.flops} algorithmic flops per launch, each product computed as three TF32 MMAs (ceiling of the "
                f"scheme: a third of the peak); peak = cuBLAS bf16 burst, of {src}, x the nominal TF32/bf16 ratio 1.1/2.25")
    else:
        ach = wl.flops / ms / 1e9
        derived = sm_count * 128 * 2 * (sm_max_mhz or 1965.0) * 1e6 / 1e12
        unit, bound = "TFLOP/s", "alu"
        if alu_peak:
            peak = alu_peak
            note = (f"fp32 FFMA peak measured on this GPU with a register-only FMA loop (forge_selftest_ffma_rate); "
                    f"SMs x 128 lanes x 2 flop x max SM clock would be {derived:.2f}")
        else:
            peak = derived
            note = "fp32 FFMA peak = SMs x 128 lanes x 2 flop x max SM clock (derived, not measured)"
    key = NCU_TRAFFIC.get(wl.name)
    traffic = key["bytes"] if key and key["sha"] == kernel_source_hash(kernel) else None
    return {"bound": bound, "achieved": round(ach, 2), "peak": round(peak, 2), "unit": unit,
            "frac": round(ach / peak, 4), "traffic": traffic, "note": note}


def unit_value(wl, ms, n_units=1):
    """Whole-job rate: the units (bytes or flops of one workload) all ranks processed / the slowest rank's time."""
    if wl.hbm_bound:
        return multigpu.aggregate_rate(wl.algorithmic_bytes, n_units, ms) / 1e9, "GB/s"
    return multigpu.aggregate_rate(wl.flops, n_units, ms) / 1e12, "TFLOP/s"


# ---- CPU oracle leg -------------------------------------------------------------------------------
def oracle_sample(wl, inp, target_s=12.0, max_rows=None):
    """Time the oracle, as it stands, on a bounded sample of rows of the workload."""
    import oracle
    M = inp["X"].shape[0]
    rows_all = wk.sample_rows(M)
    probe = rows_all[: min(len(rows_all), max(4, 2 * oracle.threads()))]      # enough rows to occupy every thread
    extra = {"sub": inp.get("sub"), "target": inp.get("target")}
    per_row = 0.0
    for _ in range(2):          # the first call pays for thread start-up and first touches; estimate from the second
        t = time.perf_counter()
        oracle.fused_linear(inp["X"], inp["W"], inp["b"], inp["gamma"], inp["beta"], act=wl.act, scale=wl.scale,
                            red=wl.red, eps=wl.ln_eps, rows=probe, **extra)
        per_row = (time.perf_counter() - t) / len(probe)
    n = int(max(len(probe), min(M, target_s / max(per_row, 1e-9))))
    if max_rows:
        n = min(n, max_rows)
    rows = np.arange(n, dtype=np.int64) * (M // n) if n < M else np.arange(M, dtype=np.int64)
    t = time.perf_counter()
    oracle.fused_linear(inp["X"], inp["W"], inp["b"], inp["gamma"], inp["beta"], act=wl.act, scale=wl.scale,
                        red=wl.red, eps=wl.ln_eps, rows=rows, **extra)
    dt = time.perf_counter() - t
    flops = 2.0 * len(rows) * wl.N * wl.K
    if wl.hbm_bound:
        value, unit = (len(rows) / M) * wl.algorithmic_bytes / dt / 1e9, "GB/s"
    else:
        value, unit = flops / dt / 1e12, "TFLOP/s"
    return {"value": value, "unit": unit, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{len(rows)} of {M} rows of {wl.name} (all N, all K), fp64 loops, {dt:.2f} s",
            "seconds": dt, "rows": len(rows)}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, same metric and workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    wl = ALL_WORKLOADS[args.workload]
    inp = wk.make_inputs(wl)
    per_step_target = max(1.0, min(10.0, 60.0 / max(1, args.steps + args.warmup)))
    first = oracle_sample(wl, inp, target_s=per_step_target)
    rows = first["rows"]
    import oracle
    sel = np.arange(rows, dtype=np.int64) * (wl.M // rows)
    times = []
    for i in range(args.warmup + args.steps):
        t = time.perf_counter()
        oracle.fused_linear(inp["X"], inp["W"], inp["b"], inp["gamma"], inp["beta"], act=wl.act, scale=wl.scale,
                            red=wl.red, eps=wl.ln_eps, rows=sel, sub=inp.get("sub"), target=inp.get("target"))
        if i >= args.warmup:
            times.append(time.perf_counter() - t)
    ms = 1e3 * sum(times) / len(times)
    if wl.hbm_bound:
        value, unit = (rows / wl.M) * wl.algorithmic_bytes / ms / 1e6, "GB/s"
    else:
        value, unit = 2.0 * rows * wl.N * wl.K / ms / 1e9, "TFLOP/s"
    line = {"impl": "reference", "metric": f"fused-op {unit} ({wl.name})", "value": value, "unit": unit,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, args.gpus, extra={"step": f"{rows} sampled rows of the workload per step"}),
            "cpu_baseline": {"value": value, "unit": unit, "cores": first["cores"], "kind": "oracle",
                             "sample": f"{rows} of {wl.M} rows of {wl.name} per step, fp64 loops"},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


def run_column_sharded(args, wl, torch, dist, rank, world, local, peaks, props):
    """--shard cols: the rows of W (and the slice of b) are split over the ranks, X is replicated, every
    rank runs the fused kernel on its slice and the partial out[M] are combined by one all-reduce of M
    floats per step (inside the timed region).  Strong scaling of one skinny-M problem."""
    import dataclasses
    if wl.red not in multigpu.COLUMN_SHARDABLE:
        raise SystemExit("--shard cols needs a row-sum or row-max workload (c4)")
    lo, hi = multigpu.rank_cols(wl, rank, world)
    inp = wk.make_inputs(wl)
    inp["W"] = np.ascontiguousarray(inp["W"][lo:hi])
    if inp["b"] is not None:
        inp["b"] = np.ascontiguousarray(inp["b"][lo:hi])
    wl_r = dataclasses.replace(wl, N=hi - lo)
    d = device_tensors(wl_r, inp, torch)
    op = make_op(wl_r, wl.M, local)
    step = op.bind(d["X"], d["W"], d["b"], d["gamma"], d["beta"], d["out"])
    grp = dist if world > 1 else None

    def one():
        step()
        multigpu.combine_column_partials(d["out"], wl.red, grp)
    for _ in range(args.warmup):
        one()
    torch.cuda.synchronize()
    op.check()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as cs:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            one()
        e1.record()
        torch.cuda.synchronize()
    ms = multigpu.max_over_ranks(e0.elapsed_time(e1) / args.steps, grp, device="cuda")
    op.check()
    value = wl.algorithmic_bytes / ms / 1e6            # the one global problem's bytes: strong scaling
    # end to end: this rank's slice from pinned host memory, the combined result back
    host = {k: (None if d[k] is None else d[k].cpu().pin_memory()) for k in ("X", "W", "b")}
    host_out = torch.empty_like(d["out"], device="cpu").pin_memory()
    op.run_host(host["X"], host["W"], host["b"], None, None, host_out)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    n = max(1, min(args.steps, 10))
    for _ in range(n):
        op.run_host(host["X"], host["W"], host["b"], None, None, host_out)
        if world > 1:
            t = host_out.cuda()
            multigpu.combine_column_partials(t, wl.red, grp)
            host_out.copy_(t)
    torch.cuda.synchronize()
    e2e_ms = multigpu.max_over_ranks(1e3 * (time.perf_counter() - t0) / n, grp, device="cuda")
    line = {"metric": f"fused-op GB/s ({wl.name})", "value": round(value, 2), "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 5), "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16" if wl.dtype == wk.BF16 else "f32", "data": "synthetic",
            "config": config_of(wl, world, {"kernel": op.plan.as_dict(),
                                            "parallelism": f"rows of W sharded over {world} gpu(s), X replicated, one all-reduce of M floats per step"}),
            "clocks": cs.summary(),
            "e2e": {"value": round(wl.algorithmic_bytes / e2e_ms / 1e6, 3), "unit": "GB/s",
                    "h2d_bytes_per_step": sum(v.numel() * v.element_size() for v in host.values() if v is not None),
                    "d2h_bytes_per_step": host_out.numel() * host_out.element_size(), "steps": n, "ms_per_step": round(e2e_ms, 3)},
            "gpu_launches": args.steps,
            "roofline": {"bound": "hbm", "achieved": round(value / world, 2), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": round(value / world / peaks["hbm_gbs"], 4), "traffic": None,
                         "note": f"per GPU: the global problem's {wl.algorithmic_bytes} bytes / {world} ranks; peak = copy bandwidth, of {peaks['_source']}"}}
    op.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def config_of(wl, n_gpus, extra=None):
    names = {wk.ACT_IDENTITY: "identity", wk.ACT_RELU: "relu", wk.ACT_GELU_ERF: "gelu_erf",
             wk.ACT_GELU_TANH: "gelu_tanh", wk.ACT_SILU: "silu"}
    reds = {wk.RED_NONE: "none", wk.RED_SUM: "row_sum", wk.RED_MAX: "row_max", wk.RED_LAYERNORM: "layernorm",
            wk.RED_MEAN_GELU_RESIDUAL: "subtract_rowmean_gelu_residual", wk.RED_LOGSUMEXP: "row_logsumexp",
            wk.RED_CROSS_ENTROPY: "row_cross_entropy"}
    c = {"workload": f"{wl.name}: {wl.note}", "M_per_gpu": wl.M, "N": wl.N, "K": wl.K,
         "dtype": "bf16" if wl.dtype == wk.BF16 else "f32", "act": names[wl.act], "scale": wl.scale,
         "reduction": reds[wl.red], "seed": wl.seed, "parallelism": f"rows sharded over {n_gpus} gpu(s), no collective",
         "l2": l2_policy(wl)}
    if extra:
        c.update(extra)
    return c


EXTRA_STEPS = {"c1": 200, "c2": 20, "c4": 300, "c5": 50, "c3": 50, "n1": 20, "n2": 10, "c2t": 50, "n1t": 50, "n1b": 50, "m64": 150}


def measure_extra(w2, local, torch, peaks, props, alu_peak):
    """One of the other workloads, measured the same way as the headline (shorter), with its own clock
    record.  Returns (entry, launches)."""
    i2 = wk.make_inputs(w2)
    d2 = device_tensors(w2, i2, torch)
    rot = Rotation(w2, d2, local, torch, copies=w_copies(w2))
    fl = torch.empty(64 * 1024 * 1024, dtype=torch.float32, device="cuda") if w2.algorithmic_bytes < 130e6 else None
    steps2 = EXTRA_STEPS[w2.name]
    with ClockSampler(local, period_s=0.001) as cs:
        ms2 = time_steps(rot, steps2, 3, torch, flush_buf=fl)
    clocks2 = cs.summary()
    v2, u2 = unit_value(w2, ms2)
    launches = steps2 + 3
    entry = {"us_per_call": round(ms2 * 1e3, 2), "value": round(v2, 2), "unit": u2, "steps": steps2,
             "l2": l2_policy(w2), "clocks": clocks2, "kernel": rot.plan.as_dict()["kernel"]}
    if fl is not None:            # latency-bound workload: also the figure without the flush
        entry["us_per_call_back_to_back_warm_l2"] = round(back_to_back_us(rot, torch), 2)
        launches += 1020
    if w2.hbm_bound:           # HBM-bound: one call alone on the device, beside the back-to-back figure
        med, best = isolated_us(rot, torch)
        entry["us_per_call_isolated"] = {"median": round(med, 2), "min": round(best, 2), "calls": 30,
                                         "how": "a synchronise after every call; W copies rotated as in the timed loop"}
        entry["w_copies"] = {"count": len(rot.steps), "bytes": rot.w_bytes}
        launches += 30
    entry["roofline"] = roofline_of(w2, ms2, peaks, rot.plan.kernel, clocks2.get("sm_max_mhz"), props.multi_processor_count, alu_peak)
    time.sleep(1.0)
    entry["torch_eager_context_us"] = round(eager_context_us(w2, d2, torch, steps=5 if w2.flops > 1e11 else 50), 1)
    rot.close()
    return entry, launches


def run_kernel_only(args, wl, torch, local):
    """--kernel-only: `steps` launches of the workload's kernel on (the first --rows rows of) its seeded
    input, each timed alone, nothing else on the device: the launch sequence to profile."""
    from paper_2511_01884_b200 import binding as B
    M = args.rows or wl.M
    inp = wk.make_inputs(wl, M=M)
    d = device_tensors(wl, inp, torch)
    rot = Rotation(wl, d, local, torch, copies=1)
    torch.cuda.synchronize()
    times = []
    for _ in range(args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rot.step()
        e1.record()
        torch.cuda.synchronize()
        times.append(round(1e3 * e0.elapsed_time(e1), 1))
    rot.check()
    print(json.dumps({"kernel_only": True, "workload": wl.name, "M": M, "N": wl.N, "K": wl.K,
                      "kernel": B.kernel_name(rot.plan.kernel), "plan": rot.plan.as_dict(), "us_per_launch": times}), flush=True)
    rot.close()
    return 0


def l2_policy(wl):
    if wl.hbm_bound:
        return (f"HBM-bound: three distinct copies of W ({3 * wl.N * wl.K * wl.elem_bytes >> 20} MiB) rotated, "
                "no byte of a W is in L2 when it is read again")
    if wl.algorithmic_bytes > 130e6:
        return "operands larger than L2 (126 MB), compute-bound: no flush"
    return "L2 flushed (256 MiB write) before every call"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=HEADLINE, choices=sorted(ALL_WORKLOADS))
    ap.add_argument("--impl", default="forge", choices=["forge", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the sustained block and the short runs of the other workloads")
    ap.add_argument("--kernel-only", action="store_true",
                    help="only launch the workload's kernel --steps times, each timed alone (for use under a profiler)")
    ap.add_argument("--rows", type=int, default=0, help="with --kernel-only: use only the first ROWS rows of X (a smaller case)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="with --shard rows and N > 1: weak = every rank runs the whole workload on its own rows of a global X; "
                         "strong = the workload's M rows are split over the ranks")
    ap.add_argument("--shard", default="rows", choices=["rows", "cols"],
                    help="rows: every rank its own rows of X (weak scaling, no collective); cols: the rows of W of one "
                         "skinny-M problem over the ranks, partial out[M] combined by an all-reduce (strong scaling)")
    args = ap.parse_args()
    if not args.kernel_only:
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    n_gpus = world

    def barrier():
        if world > 1:
            dist.barrier()

    peaks = load_peaks()
    props = torch.cuda.get_device_properties(local)
    wl = ALL_WORKLOADS[args.workload]

    if args.shard == "cols":
        return run_column_sharded(args, wl, torch, dist, rank, world, local, peaks, props)

    if args.kernel_only:
        return run_kernel_only(args, wl, torch, local)

    # this rank's block of rows of the global [world * M, K] input; W, b, gamma, beta replicated
    strong = args.scaling == "strong"       # one workload's rows split over the ranks instead of one workload per rank
    rows, row_offset = multigpu.rank_rows_strong(wl, rank, world) if strong else multigpu.rank_rows_weak(wl, rank)
    n_units = 1 if strong else world
    inp = wk.make_inputs(wl, M=rows, row_offset=row_offset)
    d = device_tensors(wl, inp, torch)
    rot = Rotation(wl, d, local, torch, copies=w_copies(wl))
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.float32, device="cuda") if wl.algorithmic_bytes < 130e6 else None

    with ClockSampler(local, period_s=0.001) as cs:
        ms = time_steps(rot, args.steps, args.warmup, torch, flush_buf=flush, barrier=barrier)
    clocks = cs.summary()
    ms_max = multigpu.max_over_ranks(ms, dist if world > 1 else None, device="cuda")
    value, unit = unit_value(wl, ms_max, n_units=n_units)
    launches = args.steps * 1
    op = rot.ops[0]

    # ---- end to end: pinned host buffers in, result out, through the host entry point ----
    e2e_steps = max(1, min(args.steps, 10))
    host = {}
    for k in ("X", "W", "b", "gamma", "beta"):      # (gamma holds the subtract vector for the chain workload)
        host[k] = None if d[k] is None else d[k].cpu().pin_memory()
    host_out = torch.empty_like(d["out"], device="cpu").pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values() if v is not None)
    d2h = host_out.numel() * host_out.element_size()
    op.run_host(host["X"], host["W"], host["b"], host["gamma"], host["beta"], host_out)   # warm-up, allocates staging
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        op.run_host(host["X"], host["W"], host["b"], host["gamma"], host["beta"], host_out)
    torch.cuda.synchronize()
    e2e_ms = 1e3 * (time.perf_counter() - t0) / e2e_steps
    e2e_ms = multigpu.max_over_ranks(e2e_ms, dist if world > 1 else None, device="cuda")
    e2e_val, _ = unit_value(wl, e2e_ms, n_units=n_units)
    # run_host() plans its blocks of rows for their own row count, so a block may walk K in another order than the
    # whole problem does: the two results agree to the last place of the storage type (where the pre-activation is
    # near zero: to the rounding of the fp32 accumulation over K, bounded here by 1e-4), not always bit for bit
    e2e_out, dev_out = host_out.cuda().float(), d["out"].float()
    ulp = 2.0 ** -7 if wl.dtype != wk.F32 else 2.0 ** -22
    same = bool(((e2e_out - dev_out).abs() <= ulp * torch.maximum(e2e_out.abs(), dev_out.abs()) + 1e-4).all())
    differing = int((e2e_out != dev_out).sum())
    max_abs_diff = float((e2e_out - dev_out).abs().max())
    del e2e_out, dev_out
    op.check()

    # the measured fp32 ceiling: a register-only FMA loop on every SM
    alu_peak = None
    if rank == 0 and world == 1:
        from paper_2511_01884_b200 import binding as B
        time.sleep(1.0)
        st, tf, mhz = B.forge_selftest_ffma_rate(local, 200)
        if st == B.FORGE_OK:
            alu_peak = tf
        time.sleep(0.5)
        st, rs_b2b, rs_single = B.forge_selftest_read_stream(local)
        read_stream = {"back_to_back_gbs": round(rs_b2b, 1), "single_launch_gbs": round(rs_single, 1),
                       "how": "forge_selftest_read_stream: load-only kernel (four 32-KiB bulk copies in flight per SM) over three "
                              "rotating 256-MiB buffers, CUDA events"} if st == B.FORGE_OK else None
    line = {"metric": f"fused-op {unit} ({wl.name})", "value": round(value, 2), "unit": unit, "n_gpus": n_gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_max, 5), "higher_is_better": True,
            "scaling": args.scaling, "vs_baseline": None, "dtype": "bf16" if wl.dtype == wk.BF16 else "f32",
            "data": "synthetic", "config": config_of(wl, n_gpus, {"kernel": op.plan.as_dict(), "M_per_gpu": rows}),
            "clocks": clocks,
            "e2e": {"value": round(e2e_val, 3), "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "ms_per_step": round(e2e_ms, 3),
                    "matches_device_run": same, "elements_differing_in_the_last_place": differing, "max_abs_difference": max_abs_diff, "how": "forge_fused_linear_run_host, pinned host buffers, wall clock"},
            "gpu_launches": launches,
            "roofline": roofline_of(wl, ms * wl.M / rows, peaks, op.plan.kernel, clocks.get("sm_max_mhz"), props.multi_processor_count, alu_peak),
            "nominal_frac": round((value / world) / (NOMINAL["hbm_gbs"] if wl.hbm_bound else NOMINAL["bf16_tflops"]), 4)
            if wl.dtype == wk.BF16 else None}
    if rank == 0 and world == 1 and read_stream:
        line["hbm_read_measured"] = read_stream          # what a kernel that only reads gets: the ceiling of the HBM-bound workloads
    if alu_peak:
        line["alu_peak_measured"] = {"value": round(alu_peak, 2), "unit": "TFLOP/s", "effective_sm_mhz": round(mhz, 1),
                                     "how": "forge_selftest_ffma_rate: 200 ms of independent register-to-register fma.rn.f32x2 on every SM, CUDA events"}
    # the static half of the paper's hardware feedback (Section 2.3): what the device is
    line["gpu_spec"] = {"name": props.name, "compute_capability": f"{props.major}.{props.minor}",
                        "sms": props.multi_processor_count, "l2_bytes": getattr(props, "L2_cache_size", None),
                        "hbm_bytes": props.total_memory,
                        "shared_memory_per_sm": getattr(props, "shared_memory_per_multiprocessor", None),
                        "registers_per_sm": getattr(props, "regs_per_multiprocessor", None),
                        "measured_peaks": {k: peaks.get(k) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained")},
                        "peaks_source": peaks["_source"]}
    if rank == 0 and world == 1:
        time.sleep(2.0)
        eager_us = eager_context_us(wl, d, torch, steps=args.steps)      # same number of back-to-back calls as the timed region
        line["torch_eager_context"] = {"us_per_call": round(eager_us, 1), "value": round(unit_value(wl, eager_us / 1e3)[0], 2),
                                       "unit": unit, "what": "unfused F.linear + activation (+ reduction) in the same dtype, same GPU"}
        if not args.no_extras:
            # seconds of back-to-back launches: the clock the power limit allows, not the burst clock
            time.sleep(1.0)
            line["sustained"], n_sus = sustained_block(rot, wl, peaks, local, torch)
            launches += n_sus + 20
    rot.close()
    del d, host

    if rank == 0 and world == 1:
        line["cpu_baseline"] = {k: v for k, v in oracle_sample(wl, inp).items() if k not in ("seconds", "rows")}
        if not args.no_extras:
            line["workloads"] = {}
            for name in sorted(ALL_WORKLOADS):
                if name == wl.name:
                    continue
                torch.cuda.empty_cache()
                time.sleep(2.0)      # each workload is measured from the same (burst) power state, not in the wake of the previous one
                line["workloads"][name], n2 = measure_extra(ALL_WORKLOADS[name], local, torch, peaks, props, alu_peak)
                launches += n2
            line["gpu_launches_all_workloads"] = launches
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
