"""The -DDART_DEBUG build of the library run over the small-shape suites.

No memory sanitizer is available for these kernels, so the debug build puts an index check in front of the stores whose
indices come from the caller's lengths, counts and plans (cache appends, projection outputs, tree nodes): a check that
fails skips the store and records an error in the device status word -- nothing traps or faults.  The small-shape tests
assert a clean status word after every call; here they run once more, in a child process that loads the debug library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_suites_are_clean_under_the_debug_build():
    from paper_2601_19278_b200 import build
    lib = build.build_debug()
    env = dict(os.environ, DART_LIB=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_small.py", "tests/test_gpu_tree.py", "-x", "-q", "-m", "gpu",
                        "-p", "no:cacheprovider"], cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    assert r.returncode == 0, r.stdout[-3000:]
