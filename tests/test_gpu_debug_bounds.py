"""The bounds-checked build (-DFORGE_DEBUG_BOUNDS) on the small-shape fuzz of every kernel family.

No memory checker can be run on these GPUs, so the library can be built to check itself: every offset into
the shared-memory ring, every tensor-memory column range and every workspace index is compared with the extent
of its allocation before use; a violation is recorded in the handle's status word (FORGE_ERR_BOUNDS) and the
access skipped, which the fuzz tests would see as a failed status check.  The checked library is loaded in a
child process (FORGE_LIBRARY) so that this process keeps the normal one.
"""
import os
import subprocess
import sys

import pytest

from paper_2511_01884_b200 import build as forge_build

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_fuzz_of_every_kernel_family_passes_with_all_indices_checked():
    lib = forge_build.build_debug_bounds()
    env = dict(os.environ, FORGE_LIBRARY=lib)
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2511_01884_b200 import binding as B; B.lib(); print(B.LIB_PATH); print(B.status_string(7))"],
                           capture_output=True, text=True, cwd=ROOT, env=env, timeout=300)
    assert probe.returncode == 0 and "libforge_debug_bounds.so" in probe.stdout and "bounds-checked" in probe.stdout, probe.stdout + probe.stderr
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                        "tests/test_gpu_fuzz.py", "tests/test_gpu_skinny.py", "tests/test_gpu_layernorm.py"],
                       capture_output=True, text=True, cwd=ROOT, env=env, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
