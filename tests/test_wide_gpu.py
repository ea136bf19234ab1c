"""Head dimensions above 128 (136 ... 256) on the tensor cores: the forward accumulates the scores over two 128-column
chunks and runs two passes over the output halves; the backward uses tiles of 128 keys x 64 queries and two passes over
the halves of d.  Every element against the fp64 oracle: ragged n, causal or not, shared K/V heads, token-major and
strided tensors, fused and separate calls, forward alone."""
import math

import numpy as np
import pytest

import oracle
from paper_2609_33916_b200 import inputs as mi

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    return gpu_harness


def _inputs(B, Hq, Hkv, n, d, seed):
    q = mi.make_inputs(B, Hq, n, d, seed, "bf16")
    kv = mi.make_inputs(B, Hkv, n, d, seed + 1000, "bf16")
    return {"Q": q["Q"], "dO": q["dO"], "K": kv["K"], "V": kv["V"]}


@pytest.mark.parametrize("d", [136, 192, 256])
@pytest.mark.parametrize("n", [1, 64, 129, 300, 640])
@pytest.mark.parametrize("causal", [False, True])
def test_wide_forward_matches_oracle(H, d, n, causal):
    inp = _inputs(1, 3, 3, n, d, seed=40 + n + d)
    scale = 1.0 / math.sqrt(d)
    f = H.f64_inputs(inp, "bf16")
    ref = oracle.attn_fwd_bwd(f["Q"], f["K"], f["V"], f["dO"], causal, scale)
    got = H.run_library(inp, "bf16", causal, scale, op="fwd")
    H.assert_close(got, ref, H.TOL_BF16, keys=("O",), tag=f"wide fwd d{d} n{n}")
    assert mi.rel_err(got["L"], ref["L"]) <= 1e-3


@pytest.mark.parametrize("d", [136, 192, 256])
@pytest.mark.parametrize("B,Hq,Hkv,n,causal", [(1, 2, 2, 128, False), (2, 2, 2, 200, True), (1, 3, 3, 333, True),
                                               (1, 4, 2, 520, False), (1, 6, 1, 257, True), (1, 1, 1, 1000, True)])
@pytest.mark.parametrize("op", ["fused", "split"])
def test_wide_forward_backward_matches_oracle(H, d, B, Hq, Hkv, n, causal, op):
    inp = _inputs(B, Hq, Hkv, n, d, seed=60 + n + d)
    scale = 1.0 / math.sqrt(d)
    f = H.f64_inputs(inp, "bf16")
    ref = oracle.attn_fwd_bwd_gqa(f["Q"], f["K"], f["V"], f["dO"], causal, scale)
    got = H.run_library(inp, "bf16", causal, scale, op=op)
    errs = H.assert_close(got, ref, H.TOL_BF16, tag=f"wide d{d} B{B} H{Hq}/{Hkv} n{n} causal{causal} {op}")
    assert mi.rel_err(got["L"], ref["L"]) <= 1e-3
    print(f"wide d{d} n{n} causal{causal} {op}", {k: f"{v:.2e}" for k, v in errs.items()})


@pytest.mark.parametrize("layout", [0, 1])
def test_wide_layouts_and_explicit_mode(H, layout):
    inp = _inputs(2, 4, 2, 300, 192, seed=77)
    scale = 1.0 / math.sqrt(192)
    f = H.f64_inputs(inp, "bf16")
    ref = oracle.attn_fwd_bwd_gqa(f["Q"], f["K"], f["V"], f["dO"], True, scale)
    got = H.run_library(inp, "bf16", True, scale, dq_mode=1, layout=layout)
    H.assert_close(got, ref, H.TOL_BF16, tag=f"wide layout{layout}")


def test_wide_equals_zero_padded_problem_and_is_rejected_where_unsupported(H):
    """d = 192 is the d = 256 problem with 64 zero columns: O, L, dK, dV are the same bits (one writer per element, zero
    columns add nothing); dQ goes through fp32 atomics and agrees to rounding.  The bulk-reduce and separate-pass dQ
    strategies do not exist above 128: MOA_ERR_UNSUPPORTED, before anything is enqueued."""
    from paper_2609_33916_b200 import binding as mb
    B, Hh, n, d = 1, 2, 384, 192
    inp = _inputs(B, Hh, Hh, n, d, seed=81)
    pad = {k: np.concatenate([v, np.zeros((B, Hh, n, 256 - d), dtype=v.dtype)], axis=3) for k, v in inp.items()}
    a = H.run_library(inp, "bf16", True, 0.07)
    b = H.run_library(pad, "bf16", True, 0.07)
    np.testing.assert_array_equal(a["L"], b["L"])
    for k in ("O", "dK", "dV"):
        np.testing.assert_array_equal(a[k], b[k][..., :d], err_msg=k)
        assert not b[k][..., d:].any(), k
    assert mi.rel_err(a["dQ"], b["dQ"][..., :d]) <= 8e-3
    assert not b["dQ"][..., d:].any()
    for mode in (mb.MOA_DQ_BULK_REDUCE, mb.MOA_DQ_SEPARATE_PASS):
        desc = mb.make_desc(B, Hh, n, d, True, 0.07, dq_mode=mode)
        assert mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_FUSED) == 0
        assert mb.moa_attn_fwd(desc, 4096, 4096, 4096, 4096, 4096, check=False) == mb.MOA_ERR_UNSUPPORTED


def test_wide_long_sequence_sampled(H):
    """B1 H4 n4096 d256 causal: sampled rows and columns of the first and last head, invariants on all heads."""
    import test_parity_gpu as tp
    w = mi.Workload("d256_n4096", 1, 4, 4096, 256, True, "bf16", 91)
    tp._sampled_check(H, w, heads=[(0, 0), (0, 3)], nrows=12, ncols=12)
