"""The GEMM kernel on CTA pairs (tiles of 256 rows shared by the two CTAs of a cluster) at every shape.

By default pairs are used only where a launch has at least one 256-row tile per pair of SMs, so the small and
ragged shapes of tests/test_block_gpu.py run on single CTAs.  MOA_GEMM_PAIR=2 forces pairs wherever the kernel is
launched (the variable is read once per process, hence the child process): the same tests, the same tolerances,
now with second halves that lie partly or wholly past the last row, one-tile problems and every operand layout."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_block_tests_pass_with_pairs_forced():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    env = dict(os.environ, MOA_GEMM_PAIR="2")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_block_gpu.py"), "-x", "-q", "-m", "gpu",
                        "-k", "gemm or mlp or block", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (r.stdout or "")[-1500:] + (r.stderr or "")[-500:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and " failed" not in r.stdout, tail
