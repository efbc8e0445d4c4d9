"""ctypes front end of the C oracle in ``fused_linear_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  It shares nothing with the CUDA library and holds no arithmetic of its
own: it compiles the C file with gcc, marshals numpy arrays, and calls it.

The operator it evaluates is the chain the paper's agents fuse (Appendix A.1: matmul then
relu; Appendix B.1: a Linear layer, an element-wise epilogue and a per-row statistic),
checked the way Section 2.2 checks a kernel: same inputs, compare outputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fused_linear_oracle.c")
_LIB = os.path.join(_HERE, "libforge_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over rows) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-D_GNU_SOURCE", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        fp = ctypes.POINTER(ctypes.c_float)
        lib.forge_oracle_fused_linear.restype = ctypes.c_int
        lib.forge_oracle_fused_linear.argtypes = [
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, fp, fp, fp, fp, fp, fp,
            ctypes.POINTER(ctypes.c_int32), ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_double,
            ctypes.POINTER(ctypes.c_int64), ctypes.c_int64, ctypes.POINTER(ctypes.c_double)]
        lib.forge_oracle_act.restype = ctypes.c_double
        lib.forge_oracle_act.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.forge_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a: Optional[np.ndarray]):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def threads() -> int:
    return int(_load().forge_oracle_threads())


def act(kind: int, z: float) -> float:
    return float(_load().forge_oracle_act(int(kind), float(z)))


def fused_linear(X: np.ndarray, W: np.ndarray, b: Optional[np.ndarray] = None,
                 gamma: Optional[np.ndarray] = None, beta: Optional[np.ndarray] = None,
                 act: int = 0, scale: float = 1.0, red: int = 0, eps: float = 1e-5,
                 rows: Optional[Sequence[int]] = None, sub: Optional[np.ndarray] = None,
                 target: Optional[np.ndarray] = None) -> np.ndarray:
    """float64 result for all rows of X, or for the listed ``rows`` only.  ``sub`` is the
    vector subtracted before the row mean of reduction 4 (mean-gelu-residual); ``target`` [M]
    holds the class index of each row for reduction 6 (cross-entropy)."""
    lib = _load()
    M, K = X.shape
    N, K2 = W.shape
    if K2 != K:
        raise ValueError("X and W disagree on K")
    Xa, Xp = _f32(X)
    Wa, Wp = _f32(W)
    ba, bp = _f32(b)
    ga, gp = _f32(gamma)
    bea, bep = _f32(beta)
    sa, sp = _f32(sub)
    ta = None if target is None else np.ascontiguousarray(target, dtype=np.int32)
    tp = None if ta is None else ta.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    if rows is None:
        ra, rp, nrows = None, None, M
    else:
        ra = np.ascontiguousarray(rows, dtype=np.int64)
        rp, nrows = ra.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), int(ra.size)
    out = np.empty((nrows,) if red in (1, 2, 5, 6) else (nrows, K if red == 4 else N), dtype=np.float64)
    rc = lib.forge_oracle_fused_linear(M, N, K, Xp, Wp, bp, gp, bep, sp, tp, int(act), float(scale),
                                       int(red), float(eps), rp, nrows,
                                       out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc != 0:
        raise ValueError("oracle rejected its arguments")
    return out
