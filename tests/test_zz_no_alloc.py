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
    B, H, n, d = desc.B, desc.H, desc.n, desc.d
    dQ, dK, dV = (torch.full((B, H, n, d), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(3))
    if static:
        mb.moa_attn_bwd_static_scratch(desc, dev["Q"], dev["K"], dev["V"], O, L, dev["dO"], dQ, dK, dV)
    else:
        ws = torch.empty(mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_BWD), dtype=torch.uint8, device="cuda")
        mb.moa_attn_bwd(desc, dev["Q"], dev["K"], dev["V"], O, L, dev["dO"], dQ, dK, dV, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    return {k: t.to(torch.float64).cpu().numpy() for k, t in (("dQ", dQ), ("dK", dK), ("dV", dV))}


@pytest.mark.parametrize("n,d,causal", [(640, 128, True), (300, 64, False)])
def test_static_scratch_backward_matches_workspace_backward(n, d, causal):
    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    B, H = 1, 3
    scale = 1.0 / math.sqrt(d)
    inp = mi.make_inputs(B, H, n, d, seed=77, dtype="bf16")
    dev = {k: torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16) for k, v in inp.items()}
    desc = mb.make_desc(B, H, n, d, causal, scale, mb.MOA_BF16)
    assert mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_BWD) <= mb.MOA_STATIC_SCRATCH_BYTES
    O = torch.empty((B, H, n, d), dtype=torch.bfloat16, device="cuda")
    L = torch.empty((B, H, n), dtype=torch.float32, device="cuda")
    mb.moa_attn_fwd(desc, dev["Q"], dev["K"], dev["V"], O, L)
    ref = _run(mb, torch, desc, dev, O, L, static=False)
    for call in range(2):   # the second call starts from the first call's leftovers
        got = _run(mb, torch, desc, dev, O, L, static=True)
        for k in ("dQ", "dK", "dV"):
            assert np.all(np.isfinite(got[k])), (k, call)
            e = mi.rel_err(got[k], ref[k])
            assert e <= 1e-2, (k, call, e)
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
