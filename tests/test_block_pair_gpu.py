"""The GEMM kernel's two tilings at every shape: CTA pairs (tiles of 256 rows shared by the two CTAs of a cluster)
and single CTAs (tiles of 128 rows).

By default a launch runs on pairs unless it has only a few tiles or its M is so small that pairs would need more
waves, so each shape of tests/test_block_gpu.py exercises one of the two.  MOA_GEMM_PAIR=2 forces pairs wherever the
kernel is launched and MOA_GEMM_PAIR=0 forces single CTAs (the variable is read once per process, hence the child
processes): the same tests, the same tolerances, now with second halves that lie partly or wholly past the last row,
one-tile problems and every operand layout on pairs, and the large shapes on single CTAs."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("mode", ["2", "0"])
def test_block_tests_pass_with_the_tiling_forced(mode):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    env = dict(os.environ, MOA_GEMM_PAIR=mode)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_block_gpu.py"), "-x", "-q", "-m", "gpu",
                        "-k", "gemm or mlp or block", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = (r.stdout or "")[-1500:] + (r.stderr or "")[-500:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and " failed" not in r.stdout, tail
