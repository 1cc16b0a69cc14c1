"""The mma.sync attention kernel is the fallback of the tcgen05 kernel (head_dim 128) when the driver offers no tensor
maps.  The choice is made once per process, so the head_dim-128 parity cases are run again in a child process with the
tcgen05 kernel switched off (CATS_ATTN_TC=0); they compare against the oracle exactly as in the parent."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_head_dim_128_cases_on_the_mma_sync_kernel():
    env = dict(os.environ, CATS_ATTN_TC="0")
    sel = "test_tree_attention_matches_oracle and (heap64_P256 or rand128_P1024 or rand128_P2048_h40 or rand77_P300_h32 or heap64_P4096)"
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-q", "-x", "-k", sel],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout
