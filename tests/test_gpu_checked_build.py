"""The bounds-checked build of the library (``-DDX_CHECKED``) under the small-shape parity tests.

A memory checker is not available for these kernels, so the library can be built with explicit bounds checks on the
indices its kernels compute (expert id, table entry, work-list position, permutation index, ring slot, output row):
a violated bound records DX_DEV_BOUNDS in the device status word and skips the access.  Here the parity tests of the
small ragged shapes, the cache path and the give-up path run once against that build in a child process (the binding
picks the library up from DX_LIB_PATH); every one of them also asserts that the status word stayed clean."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_shape_parity_under_the_checked_build():
    from paper_2607_24434_b200 import build as dx_build
    lib = dx_build.build(checked=True)
    env = dict(os.environ, DX_LIB_PATH=lib)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_parity.py"), os.path.join(ROOT, "tests", "test_gpu_cache.py"),
           os.path.join(ROOT, "tests", "test_gpu_giveup.py"), os.path.join(ROOT, "tests", "test_gpu_draft_stack.py"),
           "-k", "tiny or small or duplicate or detached or top_r or residual_forms or cached or giveup or expires "
                 "or single_layer or ties or ring or gives_up"]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "failed" not in res.stdout, tail
