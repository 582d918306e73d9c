"""Both dense kernels behind both dense entry points.

By default sparsed_attn_full runs the single-CTA kernel and sparsed_attn_full_stats the kernel whose MMAs span
CTA pairs; SPARSED_DENSE_KERNEL (read once per process) forces one kernel for both. The oracle parity tests of
the dense pass and of the statistics path are re-run in child processes with each kernel forced, so that every
kernel is checked against the oracle through every entry point (ragged lengths, GQA, strided layouts, the
rescaling path, statistics per 32 / 64 / 128 keys)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("kernel", ["pair", "single"])
def test_parity_suites_with_forced_dense_kernel(kernel):
    env = dict(os.environ, SPARSED_DENSE_KERNEL=kernel)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity_small.py", "tests/test_gpu_switch_step_stats.py", "tests/test_gpu_block32.py",
           "-k", "attn_full or from_stats or stats or block32_select"]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "failed" not in res.stdout, tail
