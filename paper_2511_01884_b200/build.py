"""Build the CUDA library in-tree: ``python -m paper_2511_01884_b200.build [-v] [-f] [-DNAME[=VALUE] ...]``
(``--debug-bounds``: the bounds-checked build as a second library, ``libforge_debug_bounds.so``).

One shared object, ``libforge.so``, next to this file, from every ``csrc/*.cu``; compiled
for sm_100a only (the kernels use tcgen05 / TMEM / TMA and have no other target).

``-D`` options make a special-purpose build in place of the normal one (they force a full
rebuild, and so does the next build without them):
  -DFORGE_PROFILING_NO_COOPERATIVE   launch the kernels whose CTAs wait on one another without the
                                     cooperative attribute (profilers refuse cooperative launches of
                                     clusters); not for production use
  -DFORGE_DEBUG_BOUNDS               check shared-memory ring offsets, TMEM columns and workspace indices
                                     against their allocations and report the first violation through the
                                     handle's status word instead of making the access
  -DFORGE_K2_GROUP_M=.. -DFORGE_K2_PAIR=0 -DFORGE_K2_TAIL_SPLIT=0 -DFORGE_K2_K_SERPENTINE=0 -DFORGE_K5_K_SERPENTINE=0
  -DFORGE_K5_GROUP_M=.. -DFORGE_K5_CHUNK_KB=..
  -DFORGE_K5_TAIL_SPLIT=0 -DFORGE_TMA_L2_PROMOTION=0|64|128|256 -DFORGE_SKINNY_MAX_M=0..128 -DFORGE_K3_KB=1..8   tuning variants
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libforge.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
         "-Xcompiler", "-fPIC"]


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


DEBUG_LIB = os.path.join(HERE, "libforge_debug_bounds.so")


def build_debug_bounds(verbose: bool = False) -> str:
    """The bounds-checked build, beside the normal one (load it with FORGE_LIBRARY=<path>)."""
    return build(verbose=verbose, defines=["-DFORGE_DEBUG_BOUNDS"], out=DEBUG_LIB)


def build(verbose: bool = False, force: bool = False, defines=(), out: str = LIB) -> str:
    global OBJ
    LIB_OUT = out
    OBJ = os.path.join(HERE, "_build" if out == LIB else "_build_" + os.path.splitext(os.path.basename(out))[0])
    # a build with -D options, and the first build after one, recompile everything
    stamp = os.path.join(OBJ, "defines.txt")
    os.makedirs(OBJ, exist_ok=True)
    want = " ".join(sorted(defines))
    have = open(stamp).read() if os.path.exists(stamp) else ""
    if want != have:
        force = True
        with open(stamp, "w") as f:
            f.write(want)
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    hdrs = sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) +
                  glob.glob(os.path.join(HERE, "..", "include", "*.h")))
    os.makedirs(OBJ, exist_ok=True)
    objs, jobs = [], []
    for s in srcs:
        o = os.path.join(OBJ, os.path.basename(s)[:-3] + ".o")
        objs.append(o)
        if force or _stale(o, [s] + hdrs):
            cmd = [NVCC] + FLAGS + list(defines) + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, r

    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as ex:
        for cmd, r in ex.map(run, jobs):
            if verbose or r.returncode != 0:
                sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError("nvcc failed: " + " ".join(cmd))
    # drop objects of deleted sources
    for o in glob.glob(os.path.join(OBJ, "*.o")):
        if o not in objs:
            os.remove(o)
    if force or jobs or _stale(LIB_OUT, objs):
        tmp = LIB_OUT + f".tmp{os.getpid()}"
        subprocess.check_call([NVCC, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, LIB_OUT)
    return LIB_OUT


if __name__ == "__main__":
    if "--debug-bounds" in sys.argv:
        print(build_debug_bounds(verbose="-v" in sys.argv))
    else:
        print(build(verbose="-v" in sys.argv, force="-f" in sys.argv, defines=[a for a in sys.argv[1:] if a.startswith("-D")]))
