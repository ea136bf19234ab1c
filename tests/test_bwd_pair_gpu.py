"""The tensor-core backward's two forms for head dimensions up to 128 in the 128-column kernel: pairs of CTAs
(two adjacent key tiles per cluster, UMMAs of 256 keys issued by one CTA, dS^T halves exchanged through the
cluster's shared-memory window) and single CTAs.

dK and dV have one writer per element in both forms and add up over the query tiles in the same order, so they
must agree bit for bit; dQ is accumulated from per-key-tile (single) or per-pair partial sums in fp32, so it
agrees to rounding (bit for bit in the atomic-free mode, whose dQ comes from the query-parallel kernel).  Every
case is also held to the oracle.  The remaining parity tests run in the default form (single CTAs, the faster
one); a child process re-runs a selection of them with pairs forced."""
import math
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2609_33916_b200 import inputs as mi

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    return gpu_harness


def _both_forms(H, inp, causal, scale, **kw):
    from paper_2609_33916_b200 import binding as mb
    before = mb.moa_bwd_pair_mode(1)
    assert mb.moa_bwd_pair_mode(-1) == 1
    try:
        pair = H.run_library(inp, "bf16", causal, scale, **kw)
        mb.moa_bwd_pair_mode(0)
        single = H.run_library(inp, "bf16", causal, scale, **kw)
    finally:
        mb.moa_bwd_pair_mode(before)
    return pair, single


CASES = [
    # B, Hq, Hkv, n, d, causal
    (1, 2, 2, 128, 128, False),      # one key tile: the pair's second CTA lies past the last key
    (2, 2, 2, 256, 128, True),       # one full pair, causal: the second CTA's first query tile is wholly masked
    (1, 3, 3, 384, 128, False),      # odd number of key tiles
    (1, 2, 2, 333, 128, True),       # ragged n
    (1, 1, 1, 1000, 128, False),
    (1, 2, 2, 1111, 128, True),
    (2, 4, 2, 640, 128, True),       # shared K/V heads
    (1, 6, 1, 300, 96, False),       # multi-query, zero-filled columns
    (1, 2, 2, 520, 72, True),
    (1, 1, 1, 2048, 128, True),
]


@pytest.mark.parametrize("B,Hq,Hkv,n,d,causal", CASES)
@pytest.mark.parametrize("dq_mode", [1, 2, 3])
@pytest.mark.parametrize("layout", [0, 1])
def test_pairs_and_single_ctas_agree(H, B, Hq, Hkv, n, d, causal, dq_mode, layout):
    if layout == 1 and n > 700:
        pytest.skip("token-major layout: covered at the smaller shapes")
    q = mi.make_inputs(B, Hq, n, d, 900 + n, "bf16")
    kv = mi.make_inputs(B, Hkv, n, d, 1900 + n, "bf16")
    inp = {"Q": q["Q"], "dO": q["dO"], "K": kv["K"], "V": kv["V"]}
    scale = 1.0 / math.sqrt(d)
    pair, single = _both_forms(H, inp, causal, scale, dq_mode=dq_mode, layout=layout, path=2)
    for k in ("O", "L", "dK", "dV"):
        np.testing.assert_array_equal(pair[k], single[k], err_msg=k)
    if dq_mode == 3:
        np.testing.assert_array_equal(pair["dQ"], single["dQ"])
    f = H.f64_inputs(inp, "bf16")
    ref = oracle.attn_fwd_bwd_gqa(f["Q"], f["K"], f["V"], f["dO"], causal, scale)
    H.assert_close(pair, ref, H.TOL_BF16, tag=f"pairs n{n} d{d} dq{dq_mode}")
    H.assert_close(single, ref, H.TOL_BF16, tag=f"single n{n} d{d} dq{dq_mode}")


def test_split_call_on_pairs(H):
    """moa_attn_fwd then moa_attn_bwd (D from the preprocess kernel) in both forms."""
    inp = mi.make_inputs(2, 2, 777, 128, seed=55, dtype="bf16")
    pair, single = _both_forms(H, inp, True, 0.09, op="split", dq_mode=2)
    for k in ("O", "L", "dK", "dV"):
        np.testing.assert_array_equal(pair[k], single[k], err_msg=k)
    assert mi.rel_err(pair["dQ"], single["dQ"]) <= 8e-3


def test_many_calls_in_a_row_give_the_same_bits(H):
    """The pair protocol has no state that survives a launch: twenty calls, identical dK and dV."""
    from paper_2609_33916_b200 import binding as mb
    inp = mi.make_inputs(1, 5, 900, 128, seed=56, dtype="bf16")
    before = mb.moa_bwd_pair_mode(1)
    try:
        first = H.run_library(inp, "bf16", True, 0.088, dq_mode=3)
        for _ in range(19):
            again = H.run_library(inp, "bf16", True, 0.088, dq_mode=3)
            for k in ("O", "L", "dQ", "dK", "dV"):
                np.testing.assert_array_equal(first[k], again[k], err_msg=k)
    finally:
        mb.moa_bwd_pair_mode(before)


def test_parity_tests_pass_on_pairs():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    env = dict(os.environ, MOA_BWD_PAIR="1")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_parity_gpu.py"), "-x", "-q", "-m", "gpu",
                        "-k", "bf16_shapes or gqa_matches or other_head_dimensions or bnhd_layout_matches or c3_causal",
                        "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout or "")[-1500:] + (r.stderr or "")[-500:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and " failed" not in r.stdout, tail
