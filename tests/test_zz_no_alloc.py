"""moa_attn_bwd_static_scratch: the backward for callers that cannot allocate device
memory (no workspace argument; scratch lives in an array inside the library image).

Checked through the C ABI against moa_attn_bwd on the same inputs, on two calls in a
row -- the second call finds the previous call's leftovers in the shared array, so it
also checks that what must start at zero is cleared.  This file is collected last so a
run that stops at the first failure has already run every other test."""
import math

import numpy as np
import pytest

from paper_2609_33916_b200 import inputs as mi

pytestmark = pytest.mark.gpu


def _run(mb, torch, desc, dev, O, L, static: bool):
    dQ = torch.full_like(dev["Q"], float("nan"))
    dK, dV = torch.full_like(dev["K"], float("nan")), torch.full_like(dev["K"], float("nan"))
    if static:
        mb.moa_attn_bwd_static_scratch(desc, dev["Q"], dev["K"], dev["V"], O, L, dev["dO"], dQ, dK, dV)
    else:
        ws = torch.empty(max(16, mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_BWD)), dtype=torch.uint8, device="cuda")
        mb.moa_attn_bwd(desc, dev["Q"], dev["K"], dev["V"], O, L, dev["dO"], dQ, dK, dV, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    return {k: t.to(torch.float64).cpu().numpy() for k, t in (("dQ", dQ), ("dK", dK), ("dV", dV))}


# dtype, B, H, H_kv, n, d, causal, dq_mode, layout
CASES = [
    ("bf16", 1, 3, 3, 640, 128, True, 0, 0),      # tensor cores, default dQ strategy
    ("bf16", 1, 3, 3, 300, 64, False, 0, 0),
    ("f32", 1, 2, 2, 300, 64, True, 1, 0),        # fp32 CUDA-core path: only D lives in the scratch, dQ accumulates in place
    ("f32", 2, 1, 1, 129, 128, False, 3, 0),
    ("bf16", 1, 2, 2, 333, 128, True, 3, 0),      # atomic-free mode: no accumulator in the scratch
    ("bf16", 2, 4, 2, 257, 128, True, 0, 1),      # shared K/V heads, token-major tensors
    ("bf16", 1, 2, 2, 200, 40, False, 1, 0),      # accumulator rows of the kernel's width (64), not of d
    ("bf16", 1, 2, 2, 16128, 128, False, 2, 0),   # workspace just under the limit (16,773,120 of 16,777,216 bytes)
]


@pytest.mark.parametrize("dtype,B,H,Hkv,n,d,causal,dq_mode,layout", CASES)
def test_static_scratch_backward_matches_workspace_backward(dtype, B, H, Hkv, n, d, causal, dq_mode, layout):
    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    scale = 1.0 / math.sqrt(d)
    q = mi.make_inputs(B, H, n, d, seed=77, dtype=dtype)
    kv = mi.make_inputs(B, Hkv, n, d, seed=78, dtype=dtype)
    inp = {"Q": q["Q"], "dO": q["dO"], "K": kv["K"], "V": kv["V"]}
    if dtype == "bf16":
        dev = {k: torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16) for k, v in inp.items()}
    else:
        dev = {k: torch.from_numpy(v).cuda() for k, v in inp.items()}
    if layout:
        dev = {k: t.permute(0, 2, 1, 3).contiguous() for k, t in dev.items()}
    desc = mb.make_desc(B, H, n, d, causal, scale, mb.MOA_BF16 if dtype == "bf16" else mb.MOA_F32, dq_mode,
                        H_kv=0 if Hkv == H else Hkv, layout=layout)
    need = mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_BWD)
    assert need <= mb.MOA_STATIC_SCRATCH_BYTES
    if n > 10000:
        assert need > mb.MOA_STATIC_SCRATCH_BYTES - (1 << 17)      # this case is meant to sit just under the limit
    O = torch.empty_like(dev["Q"])
    L = torch.empty((B, H, n), dtype=torch.float32, device="cuda")
    mb.moa_attn_fwd(desc, dev["Q"], dev["K"], dev["V"], O, L)
    ref = _run(mb, torch, desc, dev, O, L, static=False)
    tol = 1e-2 if dtype == "bf16" else 1e-5
    for call in range(2):   # the second call starts from the first call's leftovers
        got = _run(mb, torch, desc, dev, O, L, static=True)
        for k in ("dQ", "dK", "dV"):
            assert np.all(np.isfinite(got[k])), (k, call)
            e = mi.rel_err(got[k], ref[k])
            assert e <= tol, (k, call, e)
        # dK and dV have one writer per element: identical bits either way
        np.testing.assert_array_equal(got["dK"], ref["dK"])
        np.testing.assert_array_equal(got["dV"], ref["dV"])


def test_static_scratch_rejects_oversized_problem():
    import torch
    from paper_2609_33916_b200 import binding as mb
    desc = mb.make_desc(1, 16, 16384, 128, False, 0.1, mb.MOA_BF16)
    assert mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_BWD) > mb.MOA_STATIC_SCRATCH_BYTES
    a = torch.empty(16, dtype=torch.uint8, device="cuda")   # never dereferenced: the size check comes first
    s = mb.moa_attn_bwd_static_scratch(desc, a, a, a, a, a, a, a, a, a, check=False)
    assert s == mb.MOA_ERR_SCRATCH_LIMIT
    assert "scratch" in mb.status_string(s)
