"""Helpers for the GPU parity tests: move seeded inputs to the device, call the
library through its C ABI (via the ctypes binding) and bring results back as
float64 numpy arrays.  torch is used for device memory only."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_33916_b200 import binding as mb
from paper_2609_33916_b200 import inputs as mi

TOL_BF16 = 1e-2   # max|err|/max|ref| per output, bf16 storage with fp32 accumulation
TOL_F32 = 1e-5    # the fp32 path


def to_device(arr: np.ndarray, dtype: str) -> torch.Tensor:
    if dtype == "bf16":
        return torch.from_numpy(arr.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(arr).cuda()


def to_host_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def run_library(inp: dict, dtype: str, causal: bool, scale: float, *, op: str = "fused",
                dq_mode: int = mb.MOA_DQ_AUTO, path: int = mb.MOA_PATH_AUTO, materialize: int = 0,
                poison: bool = True, layout: int = 0) -> dict:
    """op: 'fused' (one call) or 'split' (moa_attn_fwd then moa_attn_bwd) or 'fwd'.
    layout = 1: the library sees every tensor as [B,n,H,d] in memory (inputs are permuted on the way
    in, results permuted back), so the returned arrays are [B,H,n,d] either way."""
    B, H, n, d = inp["Q"].shape
    Hkv = inp["K"].shape[1]          # fewer K/V heads than query heads: grouped-query attention
    Q, K, V, dO = (to_device(inp[k], dtype) for k in ("Q", "K", "V", "dO"))
    if layout:
        Q, K, V, dO = (t.permute(0, 2, 1, 3).contiguous() for t in (Q, K, V, dO))
    desc = mb.make_desc(B, H, n, d, causal, scale, mb.MOA_BF16 if dtype == "bf16" else mb.MOA_F32,
                        dq_mode, materialize, path, H_kv=0 if Hkv == H else Hkv, layout=layout)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    fill = float("nan") if poison else 0.0   # unwritten elements must show up
    q_shape, kv_shape = ((B, n, H, d), (B, n, Hkv, d)) if layout else ((B, H, n, d), (B, Hkv, n, d))
    O, dQ = (torch.full(q_shape, fill, dtype=tdt, device="cuda") for _ in range(2))
    dK, dV = (torch.full(kv_shape, fill, dtype=tdt, device="cuda") for _ in range(2))
    L = torch.full((B, H, n), fill, dtype=torch.float32, device="cuda")
    ws_bytes = mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_FUSED if op != "fwd" else mb.MOA_OP_FWD)
    if materialize and op == "split":
        raise ValueError("the materialising variant has no separate backward call")
    ws = torch.full((max(ws_bytes, 16),), 0xFF, dtype=torch.uint8, device="cuda")
    if op in ("rowpar1", "rowpar2"):      # the row-parallel single-kernel comparison variant, 1 or 2 atomic sites
        ws_bytes = mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_ROWPARALLEL)
        ws = torch.full((max(ws_bytes, 16),), 0xFF, dtype=torch.uint8, device="cuda")
        mb.moa_attn_fused_rowparallel(desc, Q, K, V, dO, O, L, dQ, dK, dV, int(op[-1]), ws)
    elif op == "fused":
        mb.moa_attn_fused_fwd_bwd(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws)
    elif op == "split":
        mb.moa_attn_fwd(desc, Q, K, V, O, L, ws)
        mb.moa_attn_bwd(desc, Q, K, V, O, L, dO, dQ, dK, dV, ws)
    elif op == "fwd":
        mb.moa_attn_fwd(desc, Q, K, V, O, L, ws)
    else:
        raise ValueError(op)
    st = mb.moa_last_device_status()
    assert st == mb.MOA_OK, mb.status_string(st)
    if layout:
        O, dQ, dK, dV = (t.permute(0, 2, 1, 3) for t in (O, dQ, dK, dV))
    out = dict(O=to_host_f64(O), L=to_host_f64(L))
    if op != "fwd":
        out.update(dQ=to_host_f64(dQ), dK=to_host_f64(dK), dV=to_host_f64(dV))
    out["ws_bytes"] = ws_bytes
    return out


def f64_inputs(inp: dict, dtype: str) -> dict:
    return {k: mi.to_f64(v, dtype) for k, v in inp.items()}


def assert_close(got: dict, ref: dict, tol: float, keys=("O", "dQ", "dK", "dV"), tag=""):
    errs = {k: mi.rel_err(got[k], ref[k]) for k in keys}
    bad = {k: e for k, e in errs.items() if not (e <= tol)}
    assert not bad, f"{tag} max|err|/max|ref| over tolerance {tol}: {errs}"
    return errs
