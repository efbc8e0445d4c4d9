"""ctypes binding of ``libforge.so``: same names as ``include/forge.h``, argument
marshalling only.  There is no fallback: if the library is missing, loading raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
# FORGE_LIBRARY names another build of the same library to load instead (the bounds-checked one, say)
LIB_PATH = os.environ.get("FORGE_LIBRARY") or os.path.join(_HERE, "libforge.so")

# enums of forge.h
(FORGE_OK, FORGE_ERR_INVALID_ARG, FORGE_ERR_UNSUPPORTED, FORGE_ERR_CUDA, FORGE_ERR_ALLOC, FORGE_ERR_TIMEOUT,
 FORGE_ERR_SCRATCH_LIMIT, FORGE_ERR_BOUNDS) = range(8)
FORGE_STATIC_SCRATCH_BYTES = 1 << 20
FORGE_F32, FORGE_BF16, FORGE_F16, FORGE_F32_TF32X3 = 0, 1, 2, 3
FORGE_ACT_IDENTITY, FORGE_ACT_RELU, FORGE_ACT_GELU_ERF, FORGE_ACT_GELU_TANH, FORGE_ACT_SILU = range(5)
(FORGE_RED_NONE, FORGE_RED_SUM, FORGE_RED_MAX, FORGE_RED_LAYERNORM, FORGE_RED_MEAN_GELU_RESIDUAL,
 FORGE_RED_LOGSUMEXP, FORGE_RED_CROSS_ENTROPY) = range(7)
FORGE_KERNEL_F32_FFMA, FORGE_KERNEL_BF16_TCGEN05, FORGE_KERNEL_BF16_SKINNY, FORGE_KERNEL_BF16_TCGEN05_LN = 1, 2, 3, 4
FORGE_KERNEL_F32_TF32X3 = 5

EXPORTS = [
    "forge_fused_linear_query_plan", "forge_fused_linear_create", "forge_fused_linear_run",
    "forge_fused_linear_run_host", "forge_fused_linear_last_status", "forge_fused_linear_get_plan",
    "forge_fused_linear_launches_per_run", "forge_fused_linear_destroy", "forge_fused_linear_last_wait_detail",
    "forge_fused_linear_f32_reduce_static", "forge_selftest_bounded_wait", "forge_selftest_ffma_rate",
    "forge_selftest_read_stream", "forge_status_string", "forge_kernel_name", "forge_fused_linear_kernel_name",
]


class Desc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("dtype", ctypes.c_int), ("act", ctypes.c_int), ("red", ctypes.c_int),
                ("scale", ctypes.c_float), ("ln_eps", ctypes.c_float),
                ("has_bias", ctypes.c_int), ("device", ctypes.c_int)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int), ("tile_m", ctypes.c_int), ("tile_n", ctypes.c_int),
                ("tile_k", ctypes.c_int), ("stages", ctypes.c_int), ("cluster", ctypes.c_int),
                ("threads", ctypes.c_int), ("grid", ctypes.c_int64), ("smem_bytes", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class ForgeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libforge.so`` (built in-tree by ``paper_2511_01884_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_01884_b200.build` "
                               "(there is no non-CUDA fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i = ctypes.c_void_p, ctypes.c_int
        L.forge_fused_linear_query_plan.argtypes = [ctypes.POINTER(Desc), i, ctypes.POINTER(PlanInfo)]
        L.forge_fused_linear_create.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(vp)]
        L.forge_fused_linear_run.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
        L.forge_fused_linear_run_host.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.forge_fused_linear_last_status.argtypes = [vp]
        L.forge_fused_linear_get_plan.argtypes = [vp, ctypes.POINTER(PlanInfo)]
        L.forge_fused_linear_launches_per_run.argtypes = [vp]
        L.forge_fused_linear_destroy.argtypes = [vp]
        L.forge_fused_linear_last_wait_detail.argtypes = [vp, ctypes.POINTER(ctypes.c_int * 4)]
        L.forge_status_string.argtypes = [i]
        L.forge_status_string.restype = ctypes.c_char_p
        L.forge_kernel_name.argtypes = [i]
        L.forge_kernel_name.restype = ctypes.c_char_p
        L.forge_fused_linear_f32_reduce_static.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, i, i,
                                                           ctypes.c_float, vp, vp, vp, vp, vp]
        L.forge_selftest_bounded_wait.argtypes = [i, i, ctypes.POINTER(ctypes.c_int * 4)]
        L.forge_selftest_ffma_rate.argtypes = [i, i, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.forge_fused_linear_kernel_name.argtypes = [vp]
        L.forge_fused_linear_kernel_name.restype = ctypes.c_char_p
        L.forge_selftest_read_stream.argtypes = [i, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        for n in EXPORTS[:13]:
            getattr(L, n).restype = i
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().forge_status_string(int(status)).decode()


def kernel_name(kernel: int) -> str:
    return lib().forge_kernel_name(int(kernel)).decode()


def make_desc(M, N, K, dtype, act, red, scale=1.0, ln_eps=1e-5, has_bias=True, device=0) -> Desc:
    return Desc(int(M), int(N), int(K), int(dtype), int(act), int(red), float(scale), float(ln_eps),
                1 if has_bias else 0, int(device))


def forge_fused_linear_query_plan(desc: Desc, sm_count: int = 148):
    """(status, PlanInfo) -- host only, touches no device."""
    info = PlanInfo()
    st = lib().forge_fused_linear_query_plan(ctypes.byref(desc), int(sm_count), ctypes.byref(info))
    return st, info


def forge_fused_linear_create(desc: Desc):
    """(status, handle)"""
    h = ctypes.c_void_p()
    st = lib().forge_fused_linear_create(ctypes.byref(desc), ctypes.byref(h))
    return st, h


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()           # torch tensor (device or pinned host)


def forge_fused_linear_run(h, X, W, b, gamma, beta, out, stream=None) -> int:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    return lib().forge_fused_linear_run(h, _ptr(X), _ptr(W), _ptr(b), _ptr(gamma), _ptr(beta), _ptr(out), stream)


def forge_fused_linear_run_host(h, X, W, b, gamma, beta, out) -> int:
    return lib().forge_fused_linear_run_host(h, _ptr(X), _ptr(W), _ptr(b), _ptr(gamma), _ptr(beta), _ptr(out))


def forge_fused_linear_last_status(h) -> int:
    return lib().forge_fused_linear_last_status(h)


def forge_fused_linear_last_wait_detail(h):
    """[wait site, detail word, CTA, thread] of the give-up the last last_status() call saw."""
    d = (ctypes.c_int * 4)()
    st = lib().forge_fused_linear_last_wait_detail(h, ctypes.byref(d))
    if st != FORGE_OK:
        raise ForgeError(st, "last_wait_detail")
    return list(d)


def forge_selftest_bounded_wait(device: int = 0, budget_ms: int = 50):
    """(status, [site, detail, CTA, thread]) of the bounded-wait self-test (expects FORGE_ERR_TIMEOUT)."""
    d = (ctypes.c_int * 4)()
    st = lib().forge_selftest_bounded_wait(int(device), int(budget_ms), ctypes.byref(d))
    return st, list(d)


def forge_selftest_ffma_rate(device: int = 0, milliseconds: int = 200):
    """(status, TFLOP/s, effective SM MHz) of the register-only FMA loop: the measured fp32 ceiling."""
    t, f = ctypes.c_double(0.0), ctypes.c_double(0.0)
    st = lib().forge_selftest_ffma_rate(int(device), int(milliseconds), ctypes.byref(t), ctypes.byref(f))
    return st, t.value, f.value


def forge_selftest_read_stream(device: int = 0):
    """(status, GB/s back to back, GB/s of a single launch) of the load-only stream: the measured HBM read ceiling."""
    a, b = ctypes.c_double(0.0), ctypes.c_double(0.0)
    st = lib().forge_selftest_read_stream(int(device), ctypes.byref(a), ctypes.byref(b))
    return st, a.value, b.value


def forge_fused_linear_kernel_name(h) -> str:
    return lib().forge_fused_linear_kernel_name(h).decode()


def forge_fused_linear_get_plan(h) -> PlanInfo:
    info = PlanInfo()
    st = lib().forge_fused_linear_get_plan(h, ctypes.byref(info))
    if st != FORGE_OK:
        raise ForgeError(st, "get_plan")
    return info


def forge_fused_linear_launches_per_run(h) -> int:
    return lib().forge_fused_linear_launches_per_run(h)


def forge_fused_linear_f32_reduce_static(M, N, K, act, red, scale, X, W, b, out, stream=None) -> int:
    """fp32 row sum / max on the current device using the library's fixed scratch array: no
    handle, no allocation (see forge.h for who needs this and for the size limit)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    return lib().forge_fused_linear_f32_reduce_static(int(M), int(N), int(K), int(act), int(red), float(scale),
                                                      _ptr(X), _ptr(W), _ptr(b), _ptr(out), stream)


def forge_fused_linear_destroy(h) -> int:
    return lib().forge_fused_linear_destroy(h)


class FusedLinear:
    """Small convenience owner of a handle: ``FusedLinear(desc)(X, W, b, gamma, beta, out)``.
    Raises ForgeError on any non-OK status; computes nothing itself."""

    def __init__(self, desc: Desc):
        st, h = forge_fused_linear_create(desc)
        if st != FORGE_OK:
            raise ForgeError(st, "forge_fused_linear_create")
        self.desc, self.h = desc, h
        self.plan = forge_fused_linear_get_plan(h)

    def __call__(self, X, W, b=None, gamma=None, beta=None, out=None, stream=None):
        st = forge_fused_linear_run(self.h, X, W, b, gamma, beta, out, stream)
        if st != FORGE_OK:
            raise ForgeError(st, "forge_fused_linear_run")
        return out

    def bind(self, X, W, b=None, gamma=None, beta=None, out=None, stream=None):
        """A zero-argument callable that issues ``forge_fused_linear_run`` on these buffers: the
        pointers and the stream are marshalled once, so a call costs one foreign-function call (for
        launch-latency-bound problems the per-call argument handling of ``__call__`` is a visible
        share of the time).  The buffers must stay alive and in place while the callable is used."""
        if stream is None:
            import torch
            stream = torch.cuda.current_stream().cuda_stream
        vp = ctypes.c_void_p
        args = (self.h, vp(_ptr(X)), vp(_ptr(W)), vp(_ptr(b)), vp(_ptr(gamma)), vp(_ptr(beta)), vp(_ptr(out)), vp(stream))
        fn = lib().forge_fused_linear_run

        def call():
            st = fn(*args)
            if st != FORGE_OK:
                raise ForgeError(st, "forge_fused_linear_run")
        return call

    def run_host(self, X, W, b=None, gamma=None, beta=None, out=None):
        st = forge_fused_linear_run_host(self.h, X, W, b, gamma, beta, out)
        if st != FORGE_OK:
            raise ForgeError(st, "forge_fused_linear_run_host")
        return out

    def check(self):
        st = forge_fused_linear_last_status(self.h)
        if st != FORGE_OK:
            raise ForgeError(st, f"forge_fused_linear_last_status (wait detail {forge_fused_linear_last_wait_detail(self.h)})")

    def close(self):
        if self.h:
            forge_fused_linear_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
