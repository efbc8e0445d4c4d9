"""Seeded synthetic inputs for the fused linear operator.

This module only *draws numbers and rounds them to the storage type*; it holds none of
the operator's arithmetic (no contraction, activation, reduction).  Both the CPU oracle's
tests and the CUDA path's tests / benchmark take their inputs from here so that the two
sides see the same bytes.

Generator: a counter-based stream.  Element ``i`` of stream ``s`` under seed ``seed`` is a
64-bit integer obtained by running the SplitMix64 output function (Steele, Lea & Flood,
"Fast splittable pseudorandom number generators", OOPSLA 2014) over a key built from
``(seed, s, i)``; its top 53 bits give a uniform in [0, 1).  Normal variates use the
Box-Muller transform on the pair of uniforms at counters ``2i`` and ``2i+1``.  The float64
value is then rounded once to float32 and, for the bf16 workloads, once more to bfloat16
(round to nearest, ties to even).

The five workloads (C1..C5) are the five synthetic stand-ins for fused-operator-chain
benchmark tasks: same shapes, value distributions and epilogues on every run.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np

# Enumerations of the public C interface, restated as plain integers so that this module
# depends on neither side.
F32, BF16, F16, F32_TF32X3 = 0, 1, 2, 3      # F32_TF32X3: fp32 storage, tensor-core arithmetic
ACT_IDENTITY, ACT_RELU, ACT_GELU_ERF, ACT_GELU_TANH, ACT_SILU = 0, 1, 2, 3, 4
RED_NONE, RED_SUM, RED_MAX, RED_LAYERNORM, RED_MEAN_GELU_RESIDUAL, RED_LOGSUMEXP, RED_CROSS_ENTROPY = 0, 1, 2, 3, 4, 5, 6
VECTOR_OUT = (RED_SUM, RED_MAX, RED_LOGSUMEXP, RED_CROSS_ENTROPY)      # reductions whose output is fp32 [M]

STREAM_X, STREAM_W, STREAM_B, STREAM_GAMMA, STREAM_BETA, STREAM_SUB, STREAM_TARGET = 0, 1, 2, 3, 4, 5, 6

_MASK64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on an array of uint64 states (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)) & _MASK64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK64
        return z ^ (z >> np.uint64(31))


def uniform01(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """``count`` uniforms in [0,1) for counters ``start .. start+count-1`` (float64)."""
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(seed * 0x100000001B3 + stream) & 0xFFFFFFFFFFFFFFFF],
                                   dtype=np.uint64))[0]
        ctr = np.arange(start, start + count, dtype=np.uint64)
        bits = _splitmix64(ctr ^ key)
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def _chunks(n: int, step: int = 1 << 20):
    return [(lo, min(n, lo + step)) for lo in range(0, n, step)]


def _for_chunks(n: int, fill) -> None:
    """Run ``fill(a, b)`` over the chunks of range(n); chunks are independent (the stream is
    counter-based), so they are filled by a few host threads."""
    ch = _chunks(n)
    if len(ch) <= 1:
        for a, b in ch:
            fill(a, b)
        return
    with ThreadPoolExecutor(max_workers=min(len(ch), os.cpu_count() or 1)) as ex:
        list(ex.map(lambda ab: fill(*ab), ch))


def draw_uniform(seed: int, stream: int, n: int, lo: float, hi: float) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)

    def fill(a, b):
        out[a:b] = (lo + (hi - lo) * uniform01(seed, stream, a, b - a)).astype(np.float32)
    _for_chunks(n, fill)
    return out


def draw_normal(seed: int, stream: int, n: int, std: float, start: int = 0) -> np.ndarray:
    """``n`` normals N(0, std) for element indices ``start .. start+n-1`` of the stream."""
    out = np.empty(n, dtype=np.float32)

    def fill(a, b):
        u = uniform01(seed, stream, 2 * (start + a), 2 * (b - a))
        u1 = 1.0 - u[0::2]                      # (0, 1]: log is finite
        u2 = u[1::2]
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        out[a:b] = (std * z).astype(np.float32)
    _for_chunks(n, fill)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest, ties to even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> the float32 holding the same value (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_storage(x: np.ndarray, dtype: int) -> np.ndarray:
    """Return float32 values that are exactly representable in the storage dtype."""
    if dtype in (F32, F32_TF32X3):
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == F16:          # IEEE half: numpy rounds to nearest even
        return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).astype(np.float32)
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


@dataclasses.dataclass(frozen=True)
class Dist:
    kind: str                     # "normal" | "uniform" | "zero" | "none"
    a: float = 0.0                # std (normal) or low (uniform)
    b: float = 0.0                # high (uniform)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: int
    M: int
    N: int
    K: int
    act: int
    red: int
    scale: float
    ln_eps: float
    x: Dist
    w: Dist
    bias: Dist
    gamma: Dist = Dist("none")
    beta: Dist = Dist("none")
    seed: int = 0
    note: str = ""
    sub: Dist = Dist("none")      # vector subtracted before the row mean (mean-gelu-residual only)

    @property
    def flops(self) -> int:
        return 2 * self.M * self.N * self.K

    @property
    def hbm_bound(self) -> bool:
        """Few rows of X on 16-bit storage: streaming W once is the whole cost (below 128 flop per byte the
        tensor cores wait for the memory), so the rate that means something is bytes per second."""
        return self.dtype in (BF16, F16) and self.M < 128

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype in (F32, F32_TF32X3) else 2

    @property
    def out_cols(self) -> int:
        """Columns of the output matrix (0: the output is a vector of M floats)."""
        if self.red in VECTOR_OUT:
            return 0
        return self.K if self.red == RED_MEAN_GELU_RESIDUAL else self.N

    @property
    def out_bytes(self) -> int:
        return self.M * 4 if self.out_cols == 0 else self.M * self.out_cols * self.elem_bytes

    @property
    def algorithmic_bytes(self) -> int:
        """Every input read once plus the output written once."""
        e = self.elem_bytes
        n = self.M * self.K + self.N * self.K
        if self.bias.kind != "none":
            n += self.N
        if self.red == RED_LAYERNORM:
            n += 2 * self.N
        if self.sub.kind != "none":
            n += self.N
        return n * e + self.out_bytes + (4 * self.M if self.red == RED_CROSS_ENTROPY else 0)


WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", F32, 128, 512, 256, ACT_RELU, RED_SUM, 1.0, 0.0,
                   Dist("normal", 1.0), Dist("uniform", -1 / 16, 1 / 16), Dist("uniform", -0.1, 0.1),
                   note="fp32, ReLU, row sum"),
    "c2": Workload("c2", F32, 4096, 4096, 4096, ACT_GELU_TANH, RED_NONE, 0.5, 0.0,
                   Dist("normal", 1.0), Dist("uniform", -1 / 64, 1 / 64), Dist("uniform", -0.1, 0.1),
                   note="fp32, GELU-tanh, scale 0.5"),
    "c3": Workload("c3", BF16, 8192, 8192, 8192, ACT_SILU, RED_NONE, 1.0, 0.0,
                   Dist("normal", 1.0), Dist("normal", 0.02), Dist("normal", 0.02),
                   note="bf16, SiLU"),
    "c4": Workload("c4", BF16, 16, 16384, 8192, ACT_GELU_ERF, RED_MAX, 1.0, 0.0,
                   Dist("normal", 1.0), Dist("normal", 0.02), Dist("zero"),
                   note="bf16 skinny-M, GELU-erf, row max"),
    "c5": Workload("c5", BF16, 16384, 4096, 4096, ACT_GELU_TANH, RED_LAYERNORM, 1.0, 1e-5,
                   Dist("normal", 1.0), Dist("normal", 0.02), Dist("normal", 0.02),
                   Dist("uniform", 0.9, 1.1), Dist("normal", 0.01),
                   note="bf16, GELU-tanh, LayerNorm over N"),
}


# Workloads beyond the five configurations: the paper's own case-study chain (Appendix B.1), the
# loss of a classifier head, and C2 / the chain again with the contraction on the tensor cores.
EXTRA_WORKLOADS: Dict[str, Workload] = {
    "n1": Workload("n1", F32, 4096, 4096, 4096, ACT_IDENTITY, RED_MEAN_GELU_RESIDUAL, 1.0, 0.0,
                   Dist("normal", 1.0), Dist("uniform", -1 / 64, 1 / 64), Dist("uniform", -0.1, 0.1),
                   note="fp32, subtract, row mean, GELU-erf, residual add", sub=Dist("uniform", -0.5, 0.5)),
    # the loss of a language-model head: logits never materialised (Section 4's CrossEntropyLoss case)
    "n2": Workload("n2", BF16, 8192, 32768, 4096, ACT_IDENTITY, RED_CROSS_ENTROPY, 1.0, 0.0,
                   Dist("normal", 1.0), Dist("normal", 0.02), Dist("normal", 0.02),
                   note="bf16, per-row cross-entropy over 32768 classes"),
    "n1b": Workload("n1b", BF16, 8192, 8192, 8192, ACT_IDENTITY, RED_MEAN_GELU_RESIDUAL, 1.0, 0.0,
                    Dist("normal", 1.0), Dist("normal", 0.02), Dist("normal", 0.02),
                    note="bf16, subtract, row mean, GELU-erf, residual add", sub=Dist("uniform", -0.5, 0.5)),
    # between the skinny kernel's 32 rows and a full 128-row tile: still bound by the stream of W
    "m64": Workload("m64", BF16, 64, 32768, 8192, ACT_GELU_TANH, RED_NONE, 1.0, 0.0,
                    Dist("normal", 1.0), Dist("normal", 0.02), Dist("normal", 0.02),
                    note="bf16, 64 rows against a 32768 x 8192 weight, GELU-tanh"),
    "c2t": dataclasses.replace(WORKLOADS["c2"], name="c2t", dtype=F32_TF32X3,
                               note="C2's tensors, contraction as three TF32 tensor-core products"),
}
EXTRA_WORKLOADS["n1t"] = dataclasses.replace(EXTRA_WORKLOADS["n1"], name="n1t", dtype=F32_TF32X3,
                                             note="n1's tensors, contraction as three TF32 tensor-core products")


def _draw(d: Dist, seed: int, stream: int, n: int) -> Optional[np.ndarray]:
    if d.kind == "none":
        return None
    if d.kind == "zero":
        return np.zeros(n, dtype=np.float32)
    if d.kind == "normal":
        return draw_normal(seed, stream, n, d.a)
    if d.kind == "uniform":
        return draw_uniform(seed, stream, n, d.a, d.b)
    raise ValueError(d.kind)


def make_inputs(wl: Workload, M: Optional[int] = None, row_offset: int = 0) -> Dict[str, Optional[np.ndarray]]:
    """Host inputs of a workload as float32 arrays holding storage-exact values.

    ``M``/``row_offset`` select a contiguous block of rows of X (used when the rows are
    sharded over ranks: rank r draws rows ``row_offset .. row_offset+M-1`` of the same
    global X, so the shards tile the single-process input exactly).
    """
    rows = wl.M if M is None else M
    if wl.x.kind != "normal":
        raise ValueError("X distribution must be normal")
    x = draw_normal(wl.seed, STREAM_X, rows * wl.K, wl.x.a, start=row_offset * wl.K)
    w = _draw(wl.w, wl.seed, STREAM_W, wl.N * wl.K)
    b = _draw(wl.bias, wl.seed, STREAM_B, wl.N)
    g = _draw(wl.gamma, wl.seed, STREAM_GAMMA, wl.N)
    be = _draw(wl.beta, wl.seed, STREAM_BETA, wl.N)
    sb = _draw(wl.sub, wl.seed, STREAM_SUB, wl.N)
    r = lambda t: None if t is None else round_to_storage(t, wl.dtype)
    tg = None
    if wl.red == RED_CROSS_ENTROPY:      # class index of every row: uniform over the N columns
        u = uniform01(wl.seed, STREAM_TARGET, row_offset, rows)
        tg = np.minimum((u * wl.N).astype(np.int32), wl.N - 1)
    return {"X": r(x).reshape(rows, wl.K), "W": r(w).reshape(wl.N, wl.K),
            "b": r(b), "gamma": r(g), "beta": r(be), "sub": r(sb), "target": tg}


def custom_workload(name: str, dtype: int, M: int, N: int, K: int, act: int, red: int,
                    scale: float = 1.0, ln_eps: float = 1e-5, seed: int = 0,
                    w_std: Optional[float] = None, has_bias: bool = True) -> Workload:
    """A workload of arbitrary shape with the same kind of distributions as C1..C5."""
    w = Dist("normal", w_std) if w_std is not None else Dist("uniform", -1.0 / max(K, 1) ** 0.5,
                                                              1.0 / max(K, 1) ** 0.5)
    ln = red == RED_LAYERNORM
    return Workload(name, dtype, M, N, K, act, red, scale, ln_eps,
                    Dist("normal", 1.0), w, Dist("uniform", -0.1, 0.1) if has_bias else Dist("none"),
                    Dist("uniform", 0.9, 1.1) if ln else Dist("none"),
                    Dist("normal", 0.01) if ln else Dist("none"), seed,
                    sub=Dist("uniform", -0.5, 0.5) if red == RED_MEAN_GELU_RESIDUAL else Dist("none"))


def sample_rows(M: int, tile: int = 128) -> np.ndarray:
    """Rows used for row-sampled comparison on large shapes: one row per ``tile``-row block
    at an offset that walks through every position inside a block, plus rows 0 and M-1."""
    rows = {0, M - 1}
    for t in range((M + tile - 1) // tile):
        r = tile * t + (37 * t) % tile
        if r < M:
            rows.add(r)
    return np.array(sorted(rows), dtype=np.int64)


def shard_rows(M: int, rank: int, world: int):
    """Contiguous row block [lo, hi) of rank ``rank`` when M rows are split over ``world``
    ranks (rows are independent: every reduction of the operator runs along N)."""
    base, rem = divmod(M, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
