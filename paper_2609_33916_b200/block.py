"""A pre-norm transformer block as a fixed sequence of calls into the C-ABI library.

Argument marshalling only: every step below is one library call (RMSNorm, GEMM, attention, gated MLP);
this module owns the buffers and passes pointers.

    h1 = RMSNorm(x; g1)      q, k, v = h1 Wq^T, h1 Wk^T, h1 Wv^T       o = attention(q, k, v)   (token-major)
    x2 = x + o Wo^T          h2 = RMSNorm(x2; g2)                       y = x2 + gated_mlp(h2)

With `packed_qkv` (the default) the three projections are one GEMM against the stacked weight Wqkv = [Wq; Wk; Wv]
([3 H d, H d]): its [T, 3 H d] output is a packed [B, n, 3, H, d] array whose thirds go to the attention as Q, K, V through
explicit strides (MOA_LAYOUT_STRIDED, no copy), dQ, dK, dV come back into one such array, and the backward of the
projection is one GEMM for dh1 and one for dWqkv.  Forward: 6 calls; backward: 8 calls.  Without it: 8 and 12 calls."""
from __future__ import annotations

import math

from . import binding as mb

WEIGHTS = ("g1", "g2", "Wq", "Wk", "Wv", "Wo", "W1", "W3", "W2")


class TransformerBlock:
    def __init__(self, torch, B: int, n: int, H: int, d: int, d_ff: int, causal: bool, eps: float = 1e-5,
                 packed_qkv: bool = True):
        self.torch, self.B, self.n, self.H, self.d, self.d_ff, self.causal, self.eps = torch, B, n, H, d, d_ff, causal, eps
        self.packed = bool(packed_qkv)
        T, dm = B * n, H * d
        self.T, self.dm = T, dm
        bf = torch.bfloat16
        E = lambda *s: torch.empty(s, dtype=bf, device="cuda")
        u8 = lambda nbytes: torch.empty(max(16, nbytes), dtype=torch.uint8, device="cuda")
        self.nd = mb.make_rmsnorm_desc(T, dm, eps)
        if self.packed:
            # Q, K, V (and dQ, dK, dV) are thirds of a [B, n, 3, H, d] array; O and dO are [B, n, H, d]
            third = (3 * dm, d, n * 3 * dm)
            self.ad = mb.make_desc(B, H, n, d, causal, 1.0 / math.sqrt(d), layout=mb.MOA_LAYOUT_STRIDED,
                                   strides=(third, third, (dm, d, n * dm)))
        else:
            self.ad = mb.make_desc(B, H, n, d, causal, 1.0 / math.sqrt(d), layout=mb.MOA_LAYOUT_BNHD)
        self.md = mb.make_mlp_desc(T, dm, d_ff)
        self.proj = mb.make_gemm_desc(T, dm, dm)              # y = x W^T
        self.back = mb.make_gemm_desc(T, dm, dm, 0, 1)        # dx = dy W
        self.wgrad = mb.make_gemm_desc(dm, dm, T, 1, 1)       # dW = dy^T x
        self.proj3 = mb.make_gemm_desc(T, 3 * dm, dm)         # qkv = h1 Wqkv^T
        self.back3 = mb.make_gemm_desc(T, dm, 3 * dm, 0, 1)   # dh1 = dqkv Wqkv
        self.wgrad3 = mb.make_gemm_desc(3 * dm, dm, T, 1, 1)  # dWqkv = dqkv^T h1
        self.nws = u8(mb.moa_rmsnorm_workspace_bytes(self.nd))
        self.aws = u8(mb.moa_attn_workspace_bytes(self.ad, mb.MOA_OP_BWD))
        self.mws = u8(mb.moa_gated_mlp_workspace_bytes(self.md))
        # activations kept by the forward
        self.h1, self.o, self.x2, self.h2, self.y = (E(T, dm) for _ in range(5))
        self.qkv, self.dqkv = E(T, 3 * dm), E(T, 3 * dm)
        if self.packed:
            third_of = lambda t, i: t.view(B, n, 3, H, d)[:, :, i]
            self.q, self.k, self.v = (third_of(self.qkv, i) for i in range(3))
            self.dq, self.dk, self.dv = (third_of(self.dqkv, i) for i in range(3))
        else:
            carve = lambda t, i: t.view(-1)[i * T * dm:(i + 1) * T * dm].view(T, dm)     # three separate [T, dm] arrays
            self.q, self.k, self.v = (carve(self.qkv, i) for i in range(3))
            self.dq, self.dk, self.dv = (carve(self.dqkv, i) for i in range(3))
        self.a, self.u, self.h = (E(T, d_ff) for _ in range(3))
        self.r1, self.r2 = (torch.empty((T,), dtype=torch.float32, device="cuda") for _ in range(2))
        self.L = torch.empty((B, H, n), dtype=torch.float32, device="cuda")
        # gradients and backward scratch
        self.dh2, self.dx2, self.do, self.dh1, self.dx = (E(T, dm) for _ in range(5))
        gqkv = E(3 * dm, dm)          # dWq, dWk, dWv are its row blocks
        self.grads = dict(g1=E(dm), g2=E(dm), Wq=gqkv[:dm], Wk=gqkv[dm:2 * dm], Wv=gqkv[2 * dm:], Wo=E(dm, dm),
                          W1=E(d_ff, dm), W3=E(d_ff, dm), W2=E(dm, d_ff))
        self.gqkv = gqkv

    def prepare_weights(self, w: dict) -> dict:
        """The weights as the block reads them: with packed_qkv, adds Wqkv = [Wq; Wk; Wv] (a choice of parameter
        layout made once, outside the step; a caller that stores the stacked weight passes it as w["Wqkv"])."""
        if self.packed and "Wqkv" not in w:
            w = dict(w)
            w["Wqkv"] = self.torch.cat([w["Wq"], w["Wk"], w["Wv"]], dim=0).contiguous()
        return w

    def model_flops(self) -> float:
        """Forward+backward model FLOPs: 4 projections (2 T dm^2 forward, twice that backward), attention
        (14 n^2 d per head and sequence, halved when causal), gated MLP (18 T dm d_ff)."""
        T, dm = self.T, self.dm
        att = 14.0 * self.B * self.H * float(self.n) ** 2 * self.d * (0.5 if self.causal else 1.0)
        return 4 * 6.0 * T * dm * dm + att + 18.0 * T * dm * self.d_ff

    def forward(self, x, w, stream=None):
        s = stream
        mb.moa_rmsnorm_fwd(self.nd, x, w["g1"], self.h1, self.r1, s)
        if self.packed:
            mb.moa_gemm(self.proj3, self.h1, w["Wqkv"], self.qkv, stream=s)
        else:
            mb.moa_gemm(self.proj, self.h1, w["Wq"], self.q, stream=s)
            mb.moa_gemm(self.proj, self.h1, w["Wk"], self.k, stream=s)
            mb.moa_gemm(self.proj, self.h1, w["Wv"], self.v, stream=s)
        mb.moa_attn_fwd(self.ad, self.q, self.k, self.v, self.o, self.L, self.aws, s)
        mb.moa_gemm(self.proj, self.o, w["Wo"], self.x2, R=x, stream=s)
        mb.moa_rmsnorm_fwd(self.nd, self.x2, w["g2"], self.h2, self.r2, s)
        mb.moa_gated_mlp_fwd(self.md, self.h2, w["W1"], w["W3"], w["W2"], self.a, self.u, self.h, self.y, s, res=self.x2)
        return self.y

    def backward(self, x, w, dy, stream=None):
        s, g = stream, self.grads
        mb.moa_gated_mlp_bwd(self.md, self.h2, w["W1"], w["W3"], w["W2"], self.a, self.u, self.h, dy, self.dh2,
                             g["W1"], g["W3"], g["W2"], self.mws, s)
        mb.moa_rmsnorm_bwd(self.nd, self.x2, w["g2"], self.r2, self.dh2, self.dx2, g["g2"], self.nws, s, dx_add=dy)
        mb.moa_gemm(self.wgrad, self.dx2, self.o, g["Wo"], stream=s)
        mb.moa_gemm(self.back, self.dx2, w["Wo"], self.do, stream=s)
        mb.moa_attn_bwd(self.ad, self.q, self.k, self.v, self.o, self.L, self.do, self.dq, self.dk, self.dv, self.aws, s)
        if self.packed:
            mb.moa_gemm(self.back3, self.dqkv, w["Wqkv"], self.dh1, stream=s)
            mb.moa_gemm(self.wgrad3, self.dqkv, self.h1, self.gqkv, stream=s)
        else:
            mb.moa_gemm(self.back, self.dq, w["Wq"], self.dh1, stream=s)
            mb.moa_gemm(self.back, self.dk, w["Wk"], self.dh1, R=self.dh1, stream=s)
            mb.moa_gemm(self.back, self.dv, w["Wv"], self.dh1, R=self.dh1, stream=s)
            mb.moa_gemm(self.wgrad, self.dq, self.h1, g["Wq"], stream=s)
            mb.moa_gemm(self.wgrad, self.dk, self.h1, g["Wk"], stream=s)
            mb.moa_gemm(self.wgrad, self.dv, self.h1, g["Wv"], stream=s)
        mb.moa_rmsnorm_bwd(self.nd, x, w["g1"], self.r1, self.dh1, self.dx, g["g1"], self.nws, s, dx_add=self.dx2)
        return self.dx, g
