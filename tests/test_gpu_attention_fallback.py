"""The mma.sync attention kernel is the fallback of the tcgen05 kernel (head_dim 128) when the driver offers no tensor
maps.  The head_dim-128 parity cases are run again in a child process that switches the tcgen05 kernel off
(the CATS_TEST_ATTENTION_KERNEL variable is read by tests/conftest.py, which calls the library's
cats_debug_attention_kernel hook; the library itself reads no environment variable); they compare against the oracle
exactly as in the parent."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_head_dim_128_cases_on_the_mma_sync_kernel():
    env = dict(os.environ, CATS_TEST_ATTENTION_KERNEL="0")
    sel = "test_tree_attention_matches_oracle and (heap64_P256 or rand128_P1024 or rand128_P2048_h40 or rand77_P300_h32 or heap64_P4096)"
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-q", "-x", "-k", sel],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


def test_cases_on_the_two_threads_per_row_instances():
    """By default every tree runs the instances with four softmax threads per query row; the instances with two are run
    on the same cases here."""
    env = dict(os.environ, CATS_TEST_ATTENTION_KERNEL="2")
    sel = "test_tree_attention_matches_oracle and (heap64_P256 or heap64_P4096 or chain16 or chain5_P0 or single_P1 or rand40 or rand49_P200_h32 or rand33 or rand17_P700_h40 or rand128_P256 or rand128_P1024 or rand90_P5000_h32 or rand100_P63)"
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-q", "-x", "-k", sel],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout
