"""The two alternative forward kernels against the fp64 oracle: `pair` (pairs of SMs, two-CTA
tensor-core mode) and `solo` (one query tile per CTA with double-buffered scores).

Both are opt-in through the environment variable HILBERTA_FORWARD_KERNEL, which the library reads
once per process.  So this test runs the bf16 forward and log-sum-exp parity tests again in a child
process with that variable set: the same cases, the same tolerances (max-abs <= 1e-2, relative L2
<= 5e-3, same launch twice bit-identical), the other kernel."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("kernel", ["pair", "solo"])
def test_alternative_kernel_passes_the_bf16_parity_tests(kernel):
    env = dict(os.environ, HILBERTA_FORWARD_KERNEL=kernel)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_attn_bf16_gpu.py"), os.path.join(ROOT, "tests", "test_lse_gpu.py"),
           "-k", "not largest_grid and not flux4096"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout or "")[-3000:] + (r.stderr or "")[-1000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout, tail
