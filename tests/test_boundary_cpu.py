"""Host-side checks of the C interface that need no GPU: the library loads, exports every
symbol the header declares, validates descriptors, and plans kernels as documented."""
import ctypes
import os
import re
import subprocess

import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import build as forge_build
from paper_2511_01884_b200 import workloads as wk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    forge_build.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "forge.h")).read()
    declared = set(re.findall(r"\b(forge_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    L = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), f"{name} is declared in forge.h but not exported"
    assert declared == set(B.EXPORTS)


def test_header_compiles_and_links_as_c99(tmp_path):
    """include/forge.h is a C interface: a strict C99 translation unit includes it, links the library and
    calls the host-only entry points and every NULL-argument path."""
    exe = str(tmp_path / "header_c99")
    pkg = os.path.dirname(B.LIB_PATH)
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "c", "header_c99.c"), "-o", exe, "-L", pkg, "-lforge", f"-Wl,-rpath,{pkg}"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "ok" in r.stdout


def test_kernel_name_of_a_handle_needs_a_handle():
    assert B.forge_fused_linear_kernel_name(None) == "no handle"


def test_no_vendor_gemm_library_is_linked():
    out = subprocess.run(["ldd", B.LIB_PATH], capture_output=True, text=True).stdout
    for lib in ("cublas", "cudnn", "cutlass", "nccl"):
        assert lib not in out.lower()


def test_enums_match_the_workload_module():
    assert (B.FORGE_F32, B.FORGE_BF16, B.FORGE_F16, B.FORGE_F32_TF32X3) == (wk.F32, wk.BF16, wk.F16, wk.F32_TF32X3)
    assert (B.FORGE_ACT_IDENTITY, B.FORGE_ACT_RELU, B.FORGE_ACT_GELU_ERF, B.FORGE_ACT_GELU_TANH, B.FORGE_ACT_SILU) == \
           (wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU)
    assert (B.FORGE_RED_NONE, B.FORGE_RED_SUM, B.FORGE_RED_MAX, B.FORGE_RED_LAYERNORM) == \
           (wk.RED_NONE, wk.RED_SUM, wk.RED_MAX, wk.RED_LAYERNORM)


def test_invalid_descriptors():
    ok = dict(M=8, N=8, K=8, dtype=0, act=0, red=0)
    for bad in (dict(M=0), dict(N=-1), dict(K=0), dict(dtype=4), dict(dtype=-1), dict(act=5), dict(act=-1), dict(red=7), dict(red=-1)):
        st, _ = B.forge_fused_linear_query_plan(B.make_desc(**{**ok, **bad}))
        assert st == B.FORGE_ERR_INVALID_ARG, bad
        st, h = B.forge_fused_linear_create(B.make_desc(**{**ok, **bad}))
        assert st == B.FORGE_ERR_INVALID_ARG and not h
    st, _ = B.forge_fused_linear_query_plan(B.make_desc(8, 8, 8, 0, 0, 0, scale=float("nan")))
    assert st == B.FORGE_ERR_INVALID_ARG
    st, _ = B.forge_fused_linear_query_plan(B.make_desc(8, 8, 8, 0, 0, 3, ln_eps=-1.0))
    assert st == B.FORGE_ERR_INVALID_ARG
    assert B.lib().forge_fused_linear_query_plan(None, 148, None) == B.FORGE_ERR_INVALID_ARG
    assert B.lib().forge_fused_linear_create(None, None) == B.FORGE_ERR_INVALID_ARG
    assert B.forge_fused_linear_destroy(None) == B.FORGE_ERR_INVALID_ARG
    assert B.forge_fused_linear_last_status(None) == B.FORGE_ERR_INVALID_ARG
    assert B.lib().forge_fused_linear_run(None, None, None, None, None, None, None, None) == B.FORGE_ERR_INVALID_ARG


def test_unsupported_is_reported_not_rerouted():
    # bf16 rows must have a 16-byte pitch
    for M, N, K in ((64, 8, 12), (64, 12, 8)):
        st, _ = B.forge_fused_linear_query_plan(B.make_desc(M, N, K, wk.BF16, 0, 0))
        assert st == B.FORGE_ERR_UNSUPPORTED
    # LayerNorm: the tiles of a row strip wait for one another, so a row may not have more tiles than resident CTAs
    st, p = B.forge_fused_linear_query_plan(B.make_desc(64, 4096, 8, wk.F32, 0, wk.RED_LAYERNORM))
    assert st == B.FORGE_OK and p.kernel == B.FORGE_KERNEL_F32_FFMA and p.cluster == 1 and p.grid == 32
    st, p = B.forge_fused_linear_query_plan(B.make_desc(64, 128 * 296 + 1, 8, wk.F32, 0, wk.RED_LAYERNORM))
    assert st == B.FORGE_OK and p.grid == 296          # more tiles per strip than CTAs: every tile is computed twice
    # fp32 on the tensor cores: 16-byte pitch of X, W and Y rows; LayerNorm rows of at most 74 tiles
    for M, N, K, red in ((64, 64, 66, wk.RED_NONE), (64, 66, 64, wk.RED_NONE)):
        st, _ = B.forge_fused_linear_query_plan(B.make_desc(M, N, K, wk.F32_TF32X3, 0, red))
        assert st == B.FORGE_ERR_UNSUPPORTED
    st, _ = B.forge_fused_linear_query_plan(B.make_desc(64, 256 * 74 + 4, 64, wk.F32_TF32X3, 0, wk.RED_LAYERNORM))
    assert st == B.FORGE_OK


def test_tf32x3_plan():
    wl = wk.EXTRA_WORKLOADS["c2t"]
    st, p = B.forge_fused_linear_query_plan(B.make_desc(wl.M, wl.N, wl.K, wl.dtype, wl.act, wl.red, wl.scale))
    assert st == B.FORGE_OK and p.kernel == B.FORGE_KERNEL_F32_TF32X3
    assert (p.tile_m, p.tile_n, p.tile_k, p.cluster, p.grid, p.threads) == (256, 256, 32, 2, 148, 512)
    assert p.smem_bytes <= 227 * 1024
    assert "tf32" in B.kernel_name(B.FORGE_KERNEL_F32_TF32X3)
    # 256 pair tiles on 74 clusters leave 34 for the last wave: each is cut in two along K, and the
    # workspace holds one 256x256 fp32 hand-over area per cut tile
    assert p.workspace_bytes >= 34 * 256 * 256 * 4
    # a problem of 4 tiles and 128 k-blocks is cut into 8 parts per tile: 32 clusters
    st, p = B.forge_fused_linear_query_plan(B.make_desc(512, 512, 4096, wl.dtype, 0, 0))
    assert st == B.FORGE_OK and p.grid == 2 * 4 * 8
    # short K: no cut
    st, p = B.forge_fused_linear_query_plan(B.make_desc(512, 512, 256, wl.dtype, 0, 0))
    assert st == B.FORGE_OK and p.grid == 2 * 4


def test_status_and_kernel_strings():
    seen = {B.status_string(s) for s in range(8)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert B.status_string(99) == "unknown status"
    assert "f32" in B.kernel_name(B.FORGE_KERNEL_F32_FFMA)


def test_fp32_plan():
    st, p = B.forge_fused_linear_query_plan(pu_desc("c1"))
    assert st == B.FORGE_OK and p.kernel == B.FORGE_KERNEL_F32_FFMA
    # few tiles: the small tile, and K = 256 cut into 4 slices of 64 so that 64 CTAs take part
    assert (p.tile_m, p.tile_n, p.grid) == (64, 64, 16 * 4) and p.workspace_bytes >= 8 * 128 * 4 + 16 * 4 * 64 * 64 * 4
    st, p = B.forge_fused_linear_query_plan(pu_desc("c2"))
    assert st == B.FORGE_OK and p.grid == 32 * 32 and p.cluster == 1 and p.tile_m == 128


def test_skinny_plan():
    """The skinny kernel's plan: C4 on 148 SMs streams 104 or 112 rows of W per CTA in stages of two 64-k boxes; a strip of
    few rows takes more boxes per stage; M beyond 96, and a long K against 16 rows of W per SM or fewer, go to the tile
    kernel."""
    st, p = B.forge_fused_linear_query_plan(pu_desc("c4"))
    assert st == B.FORGE_OK and p.kernel == B.FORGE_KERNEL_BF16_SKINNY
    assert (p.tile_m, p.tile_n, p.tile_k, p.stages, p.grid, p.threads, p.cluster) == (16, 112, 128, 6, 148, 192, 1)
    assert p.smem_bytes <= 227 * 1024 and p.workspace_bytes >= 148 * 16 * 4
    st, p = B.forge_fused_linear_query_plan(B.make_desc(16, 1184, 8192, wk.BF16, wk.ACT_RELU, wk.RED_SUM))
    assert st == B.FORGE_OK and p.kernel == B.FORGE_KERNEL_BF16_SKINNY and (p.tile_n, p.tile_k) == (8, 512)
    for M, N, K, kernel in ((96, 16384, 8192, B.FORGE_KERNEL_BF16_SKINNY), (97, 16384, 8192, B.FORGE_KERNEL_BF16_TCGEN05),
                            (16, 1024, 65536, B.FORGE_KERNEL_BF16_TCGEN05), (16, 2368, 24576, B.FORGE_KERNEL_BF16_TCGEN05),
                            (16, 2368, 16384, B.FORGE_KERNEL_BF16_SKINNY), (16, 4096, 65536, B.FORGE_KERNEL_BF16_SKINNY)):
        st, p = B.forge_fused_linear_query_plan(B.make_desc(M, N, K, wk.BF16, wk.ACT_RELU, wk.RED_MAX))
        assert st == B.FORGE_OK and p.kernel == kernel, (M, N, K)
        assert p.smem_bytes <= 227 * 1024


def pu_desc(name):
    wl = wk.WORKLOADS[name]
    return B.make_desc(wl.M, wl.N, wl.K, wl.dtype, wl.act, wl.red, wl.scale, wl.ln_eps, wl.bias.kind != "none")


def test_create_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    st, h = B.forge_fused_linear_create(pu_desc("c1"))
    assert st == B.FORGE_ERR_CUDA and not h
    with pytest.raises(B.ForgeError):
        B.FusedLinear(pu_desc("c1"))
