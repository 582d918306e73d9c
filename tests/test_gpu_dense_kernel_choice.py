"""Both dense kernels behind sparsed_attn_full.

sparsed_attn_full_stats always runs the kernel whose MMAs span CTA pairs; sparsed_attn_full runs it from 16384
tokens on and the single-CTA kernel below that, unless SPARSED_DENSE_KERNEL=pair|single (read once per process)
names one. The oracle parity tests of the dense pass are re-run in child processes with each setting, so that the
pair kernel is also checked on what the statistics path never gives it (lengths that are no multiple of 32, strided
layouts, a softmax scale, the rescaling path) and the single-CTA kernel on the long workloads."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("kernel,files,keyword", [
    ("pair", ["tests/test_gpu_parity_small.py", "tests/test_gpu_more_cases.py"], "attn_full or entry_point"),
    ("single", ["tests/test_gpu_parity_configs.py"], "config3"),
])
def test_dense_parity_suite_with_one_kernel_forced(kernel, files, keyword):
    env = dict(os.environ, SPARSED_DENSE_KERNEL=kernel)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + files + ["-k", keyword]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "failed" not in res.stdout, tail
