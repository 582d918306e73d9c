"""The CTA-pair dense kernel behind both dense entry points.

sparsed_attn_full_stats always runs the kernel whose MMAs span CTA pairs; sparsed_attn_full runs the single-CTA
kernel unless SPARSED_DENSE_KERNEL=pair (read once per process). The oracle parity tests of the dense pass are
re-run in a child process with that setting, so that the pair kernel is also checked on what the statistics
path never gives it: lengths that are no multiple of 32, strided layouts, a softmax scale, the rescaling path."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_dense_parity_suite_on_the_pair_kernel():
    env = dict(os.environ, SPARSED_DENSE_KERNEL="pair")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity_small.py", "tests/test_gpu_more_cases.py", "-k", "attn_full or entry_point"]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "failed" not in res.stdout, tail
