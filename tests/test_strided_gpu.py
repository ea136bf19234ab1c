"""MOA_LAYOUT_STRIDED: every tensor addressed through explicit (row, head, batch) strides -- the thirds of a packed
[B,n,3,H,d] projection output as Q, K, V (and a packed gradient buffer for dQ, dK, dV), packed grouped-query layouts
[B,n,H+2H_kv,d], and rows padded to a wider pitch.  Same results as the oracle, element by element, and the same bits
as the contiguous call in the deterministic mode."""
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


def _run_strided(H, inp, causal, scale, kind, dq_mode, op):
    """inp: Q, dO [B,Hq,n,d]; K, V [B,Hkv,n,d] as bf16 bit patterns.  Builds the chosen memory layout on the device,
    calls the library with MOA_LAYOUT_STRIDED and returns [B,H,n,d]-shaped float64 results."""
    import torch
    from paper_2609_33916_b200 import binding as mb
    B, Hq, n, d = inp["Q"].shape
    Hkv = inp["K"].shape[1]
    dev = {k: H.to_device(v, "bf16") for k, v in inp.items()}
    nan = float("nan")
    if kind == "packed":                 # [B, n, Hq + 2 Hkv, d]: Q heads, then K heads, then V heads, per token
        T = Hq + 2 * Hkv
        buf = torch.empty((B, n, T, d), dtype=torch.bfloat16, device="cuda")
        gbuf = torch.full((B, n, T, d), nan, dtype=torch.bfloat16, device="cuda")
        view = lambda b, lo, hi: b[:, :, lo:hi].permute(0, 2, 1, 3)          # [B, heads, n, d] view, no copy
        Q, K, V = view(buf, 0, Hq), view(buf, Hq, Hq + Hkv), view(buf, Hq + Hkv, T)
        Q.copy_(dev["Q"]); K.copy_(dev["K"]); V.copy_(dev["V"])
        dQ, dK, dV = view(gbuf, 0, Hq), view(gbuf, Hq, Hq + Hkv), view(gbuf, Hq + Hkv, T)
        dO = dev["dO"].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)   # [B,n,H,d] in memory
        O = torch.full((B, n, Hq, d), nan, dtype=torch.bfloat16, device="cuda").permute(0, 2, 1, 3)
    elif kind == "pitched":              # [B, heads, n, d + 8]: rows padded to a wider pitch
        def pitched(src, heads):
            b = torch.full((B, heads, n, d + 8), nan, dtype=torch.bfloat16, device="cuda")
            v = b[..., :d]
            if src is not None:
                v.copy_(src)
            return v
        Q, K, V, dO = pitched(dev["Q"], Hq), pitched(dev["K"], Hkv), pitched(dev["V"], Hkv), pitched(dev["dO"], Hq)
        O, dQ, dK, dV = pitched(None, Hq), pitched(None, Hq), pitched(None, Hkv), pitched(None, Hkv)
    else:
        raise ValueError(kind)
    assert mb.strides_of(Q) == mb.strides_of(dQ) and mb.strides_of(K) == mb.strides_of(V) == mb.strides_of(dK) == mb.strides_of(dV)
    assert mb.strides_of(O) == mb.strides_of(dO)
    desc = mb.make_desc(B, Hq, n, d, causal, scale, mb.MOA_BF16, dq_mode, H_kv=0 if Hkv == Hq else Hkv,
                        layout=mb.MOA_LAYOUT_STRIDED, strides=(mb.strides_of(Q), mb.strides_of(K), mb.strides_of(O)))
    L = torch.full((B, Hq, n), nan, dtype=torch.float32, device="cuda")
    ws = torch.full((max(16, mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_FUSED)),), 0xFF, dtype=torch.uint8, device="cuda")
    if op == "fused":
        mb.moa_attn_fused_fwd_bwd(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws)
    else:
        mb.moa_attn_fwd(desc, Q, K, V, O, L, ws)
        mb.moa_attn_bwd(desc, Q, K, V, O, L, dO, dQ, dK, dV, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    return {k: H.to_host_f64(t) for k, t in (("O", O), ("L", L), ("dQ", dQ), ("dK", dK), ("dV", dV))}


def _inputs(B, Hq, Hkv, n, d, seed):
    q = mi.make_inputs(B, Hq, n, d, seed, "bf16")
    kv = mi.make_inputs(B, Hkv, n, d, seed + 1000, "bf16")
    return {"Q": q["Q"], "dO": q["dO"], "K": kv["K"], "V": kv["V"]}


@pytest.mark.parametrize("kind", ["packed", "pitched"])
@pytest.mark.parametrize("B,Hq,Hkv,n,d,causal", [(2, 3, 3, 300, 128, True), (1, 4, 2, 257, 64, False), (2, 6, 1, 333, 96, True)])
@pytest.mark.parametrize("dq_mode", [0, 1, 3])
@pytest.mark.parametrize("op", ["fused", "split"])
def test_strided_tensors_match_oracle(H, kind, B, Hq, Hkv, n, d, causal, dq_mode, op):
    inp = _inputs(B, Hq, Hkv, n, d, seed=700 + n)
    scale = 1.0 / math.sqrt(d)
    got = _run_strided(H, inp, causal, scale, kind, dq_mode, op)
    f = H.f64_inputs(inp, "bf16")
    ref = oracle.attn_fwd_bwd_gqa(f["Q"], f["K"], f["V"], f["dO"], causal, scale)
    H.assert_close(got, ref, H.TOL_BF16, tag=f"{kind} B{B} H{Hq}/{Hkv} n{n} d{d} dq{dq_mode} {op}")
    assert mi.rel_err(got["L"], ref["L"]) <= 1e-3


@pytest.mark.parametrize("kind", ["packed", "pitched"])
def test_strided_call_is_bitwise_the_contiguous_call(H, kind):
    """Strides change addresses only: in the deterministic mode the results are the same bits."""
    inp = _inputs(2, 4, 2, 384, 128, seed=808)
    for op in ("fused", "split"):
        a = H.run_library(inp, "bf16", True, 0.09, dq_mode=3, op=op)
        b = _run_strided(H, inp, True, 0.09, kind, 3, op)
        for k in ("O", "L", "dQ", "dK", "dV"):
            np.testing.assert_array_equal(a[k], b[k], err_msg=f"{k} {op}")


def test_strided_long_sequence_sampled(H):
    """B1 H8/2 n8192 d128 causal in the packed layout: the whole result against the contiguous call (same bits in the
    deterministic mode), which the other tests hold to the oracle at this size."""
    inp = _inputs(1, 8, 2, 8192, 128, seed=909)
    a = H.run_library(inp, "bf16", True, 0.088, dq_mode=3)
    b = _run_strided(H, inp, True, 0.088, "packed", 3, "fused")
    for k in ("O", "L", "dQ", "dK", "dV"):
        np.testing.assert_array_equal(a[k], b[k], err_msg=k)
    c = _run_strided(H, inp, True, 0.088, "packed", 0, "fused")
    assert mi.rel_err(c["dQ"], a["dQ"]) <= 1e-2
