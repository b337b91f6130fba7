"""The GPU tests once more on the development build of the library (-DZC_DEBUG_CHECKS=1).

That build checks every shared-memory and global-memory access the kernels make through their load/store helpers
against the block's shared window and the buffers of the launch, counts what it refuses and skips it: nothing traps.
`conftest.py` reads the counters after every test when such a build is loaded and fails the test on any count, so
running the parity, batch and failure-path tests on it shows that no kernel leaves its buffers on edge sizes
(empty, one element, ragged ends, every chunk size), on damaged containers or while a wait runs out.
"""
import os
import subprocess
import sys

import pytest

from paper_2508_19263_b200 import build as zbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_no_kernel_leaves_its_buffers_in_the_checked_build():
    lib = zbuild.build_debug_library()
    env = dict(os.environ, ZC_LIBRARY=lib)
    files = ["tests/test_gpu_parity.py", "tests/test_gpu_failure_paths.py", "tests/test_gpu_batch.py", "tests/test_gpu_kv_dictionary.py"]
    r = subprocess.run([sys.executable, "-m", "pytest", *files, "-m", "gpu", "-x", "-q", "-k", "not bench_size and not large_tensor"],
                       cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    assert r.returncode == 0, r.stdout[-4000:]
    assert " passed" in r.stdout and "debug build: checked" in r.stdout, r.stdout[-2000:]
