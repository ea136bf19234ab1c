"""Decode attention (one query per head over a K/V cache) against the fp64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2609_33916_b200 import inputs as mi


@pytest.fixture(scope="module")
def rt():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build
    build.build()
    mb.lib()
    return torch, mb


def _run(rt, q, K, V, scale, dtype):
    torch, mb = rt
    B, H, d = q.shape
    Hkv, n = K.shape[1], K.shape[2]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32

    def dev(x):
        t = torch.from_numpy(np.ascontiguousarray(x))
        return (t.view(torch.bfloat16) if dtype == "bf16" else t).cuda()

    dq, dK, dV = dev(q), dev(K), dev(V)
    desc = mb.make_decode_desc(B, H, n, d, scale, mb.MOA_BF16 if dtype == "bf16" else mb.MOA_F32, H_kv=0 if Hkv == H else Hkv)
    out = torch.full((B, H, d), float("nan"), dtype=tdt, device="cuda")
    lse = torch.full((B, H), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.full((max(mb.moa_decode_workspace_bytes(desc), 16),), 0xFF, dtype=torch.uint8, device="cuda")
    mb.moa_decode_attn(desc, dq, dK, dV, out, lse, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def _inputs(B, H, Hkv, n, d, seed, dtype, gain=1.0):
    rng = np.random.default_rng(seed)
    q = (gain * rng.standard_normal((B, H, d))).astype(np.float32)
    K = rng.standard_normal((B, Hkv, n, d), dtype=np.float32)
    V = rng.standard_normal((B, Hkv, n, d), dtype=np.float32)
    if dtype == "bf16":
        return tuple(mi.f32_to_bf16_bits(x) for x in (q, K, V))
    return q, K, V


@pytest.mark.parametrize("dtype,tol", [("bf16", 1e-2), ("f32", 1e-5)])
@pytest.mark.parametrize("B,H,Hkv,n,d", [
    (1, 1, 1, 1, 64), (2, 4, 4, 7, 128), (3, 8, 2, 1000, 128), (2, 6, 1, 4097, 64), (1, 16, 1, 513, 128),
    (1, 3, 3, 20000, 128), (2, 12, 4, 300, 64),
])
def test_decode_matches_oracle(rt, dtype, tol, B, H, Hkv, n, d):
    """Every output element and the logsumexp against the oracle: cache lengths from 1 to 20000 (one
    to many segments, ragged tails), group sizes 1, 2, 3, 4, 6, 16 (a group of 16 takes two passes)."""
    q, K, V = _inputs(B, H, Hkv, n, d, seed=n + H, dtype=dtype)
    scale = 1.0 / math.sqrt(d)
    got, lse = _run(rt, q, K, V, scale, dtype)
    ref = oracle.decode_attn(mi.to_f64(q, dtype), mi.to_f64(K, dtype), mi.to_f64(V, dtype), scale)
    assert np.all(np.isfinite(got))
    assert mi.rel_err(got, ref["o"]) <= tol, (mi.rel_err(got, ref["o"]),)
    assert np.max(np.abs(lse - ref["lse"])) <= (1e-3 if dtype == "bf16" else 1e-4)


def test_decode_large_scores_need_the_running_max(rt):
    """Queries scaled x30: scores of order +-300 in the exponent; without the running maximum the
    sums overflow."""
    q, K, V = _inputs(2, 4, 2, 3000, 128, seed=3, dtype="bf16", gain=30.0)
    got, lse = _run(rt, q, K, V, 1.0 / math.sqrt(128), "bf16")
    ref = oracle.decode_attn(mi.to_f64(q, "bf16"), mi.to_f64(K, "bf16"), mi.to_f64(V, "bf16"), 1.0 / math.sqrt(128))
    assert np.all(np.isfinite(got)) and np.all(np.isfinite(lse))
    assert mi.rel_err(got, ref["o"]) <= 1e-2
    assert np.max(np.abs(lse - ref["lse"]) / np.abs(ref["lse"])) <= 1e-3


def test_decode_is_the_last_row_of_the_causal_forward(rt):
    """The library's own two paths agree: decode of the last token equals row n-1 of the causal forward."""
    torch, mb = rt
    B, H, n, d = 1, 4, 640, 128
    inp = mi.make_inputs(B, H, n, d, seed=12, dtype="bf16")
    scale = 1.0 / math.sqrt(d)
    got, lse = _run(rt, inp["Q"][:, :, n - 1], inp["K"], inp["V"], scale, "bf16")
    Q, K, V = (torch.from_numpy(inp[k]).view(torch.bfloat16).cuda() for k in ("Q", "K", "V"))
    O = torch.empty_like(Q); L = torch.empty((B, H, n), dtype=torch.float32, device="cuda")
    mb.moa_attn_fwd(mb.make_desc(B, H, n, d, True, scale), Q, K, V, O, L)
    torch.cuda.synchronize()
    last = O[:, :, n - 1].float().cpu().numpy().astype(np.float64)
    assert mi.rel_err(got, last) <= 1e-2
    assert np.max(np.abs(lse - L[:, :, n - 1].cpu().numpy())) <= 2e-3


@pytest.mark.parametrize("B,H,Hkv,n,d", [(3, 24, 3, 65536, 128), (2, 16, 4, 40000, 128), (2, 16, 2, 65536, 64)])
def test_decode_long_cache_groups_every_launch(rt, B, H, Hkv, n, d):
    """Long caches with query groups of 4 and 8 (the tensor-core route, hundreds of CTAs of many tiles each,
    keys arriving at memory pace), four launches on the same inputs, each compared with the oracle and with
    one another bit for bit.  A CTA that reads its output accumulator before its last products have
    completed shows here as one head's output off by tens of percent in some launches only."""
    torch, mb = rt
    q, K, V = _inputs(B, H, Hkv, n, d, seed=n + H + d, dtype="bf16")
    scale = 1.0 / math.sqrt(d)
    ref = oracle.decode_attn(mi.to_f64(q, "bf16"), mi.to_f64(K, "bf16"), mi.to_f64(V, "bf16"), scale)
    first = None
    for launch in range(4):
        got, lse = _run(rt, q, K, V, scale, "bf16")
        per_head = np.max(np.abs(got - ref["o"]), axis=-1) / np.max(np.abs(ref["o"]))
        assert np.max(per_head) <= 1e-2, (launch, np.argwhere(per_head > 1e-2)[:4].tolist(), float(np.max(per_head)))
        assert np.max(np.abs(lse - ref["lse"])) <= 1e-3
        if first is None:
            first = got
        else:
            assert np.array_equal(got, first), ("launch differs from the first", launch)
