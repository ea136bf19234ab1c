"""fp64 oracle of the two token-wise pieces of the transformer block: RMSNorm and the gated MLP,
each forward with its backward.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Plain numpy, the definitions written out.
The paper's block section names the pieces (RMSNorm, gated MLP, their backward passes, hidden
width d_ff) and gives the block's traffic count, but prints no formula for either piece; the
readings taken here are the usual ones:

RMSNorm over the last axis, with a gain g and a constant eps inside the root:
    r_i   = 1 / sqrt( (1/d) sum_k x_ik^2 + eps )
    y_ik  = x_ik * r_i * g_k
  backward, for an upstream dy:
    dg_k  = sum_i dy_ik * x_ik * r_i
    dx_ik = r_i * g_k * dy_ik  -  x_ik * r_i^3 * (1/d) * sum_m x_im g_m dy_im

Gated MLP with a SiLU gate (weights stored [out, in], no biases):
    a = x W1^T      u = x W3^T          [n, d_ff]
    h = silu(a) * u                     silu(a) = a * sigmoid(a)
    y = h W2^T                          [n, d]
  backward, for an upstream dy:
    dh  = dy W2                     dW2 = dy^T h
    da  = dh * u * sigmoid(a) * (1 + a * (1 - sigmoid(a)))
    du  = dh * silu(a)
    dW1 = da^T x    dW3 = du^T x    dx  = da W1 + du W3
"""
from __future__ import annotations

import numpy as np


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def rmsnorm_fwd_bwd(x, g, dy, eps: float):
    """x, dy [n,d]; g [d].  Returns dict(y [n,d], r [n], dx [n,d], dg [d]), float64."""
    x, g, dy = _f64(x), _f64(g), _f64(dy)
    n, d = x.shape
    if g.shape != (d,) or dy.shape != (n, d):
        raise ValueError("expected x, dy [n,d] and g [d]")
    r = 1.0 / np.sqrt((x * x).sum(axis=1) / d + eps)           # [n]
    y = x * r[:, None] * g[None, :]
    dg = (dy * x * r[:, None]).sum(axis=0)
    s = (x * g[None, :] * dy).sum(axis=1)                       # [n]
    dx = r[:, None] * g[None, :] * dy - x * (r ** 3 * s / d)[:, None]
    return dict(y=y, r=r, dx=dx, dg=dg)


def _sigmoid(a):
    # 1/(1+exp(-a)) evaluated without overflow for large |a|
    out = np.empty_like(a)
    pos = a >= 0
    out[pos] = 1.0 / (1.0 + np.exp(-a[pos]))
    e = np.exp(a[~pos])
    out[~pos] = e / (1.0 + e)
    return out


def gated_mlp_fwd_bwd(x, W1, W3, W2, dy):
    """x, dy [n,d]; W1, W3 [d_ff,d]; W2 [d,d_ff].
    Returns dict(a, u, h [n,d_ff], y [n,d], dx [n,d], dW1, dW3 [d_ff,d], dW2 [d,d_ff]), float64."""
    x, W1, W3, W2, dy = map(_f64, (x, W1, W3, W2, dy))
    n, d = x.shape
    dff = W1.shape[0]
    if W1.shape != (dff, d) or W3.shape != (dff, d) or W2.shape != (d, dff) or dy.shape != (n, d):
        raise ValueError("expected x, dy [n,d], W1, W3 [d_ff,d], W2 [d,d_ff]")
    a = x @ W1.T
    u = x @ W3.T
    sg = _sigmoid(a)
    h = a * sg * u
    y = h @ W2.T
    dh = dy @ W2
    dW2 = dy.T @ h
    da = dh * u * sg * (1.0 + a * (1.0 - sg))
    du = dh * a * sg
    dW1 = da.T @ x
    dW3 = du.T @ x
    dx = da @ W1 + du @ W3
    return dict(a=a, u=u, h=h, y=y, dx=dx, dW1=dW1, dW3=dW3, dW2=dW2)


def gated_mlp_bwd_from_saved(x, a, u, W1, W3, W2, dy):
    """The same backward from given pre-activations a, u (what a forward kept in storage precision):
    returns dict(da, du [n,d_ff], dx, dW1, dW3, dW2).  h is recomputed from the given a, u."""
    x, a, u, W1, W3, W2, dy = map(_f64, (x, a, u, W1, W3, W2, dy))
    sg = _sigmoid(a)
    h = a * sg * u
    dh = dy @ W2
    da = dh * u * sg * (1.0 + a * (1.0 - sg))
    du = dh * a * sg
    return dict(da=da, du=du, h=h, dx=da @ W1 + du @ W3, dW1=da.T @ x, dW3=du.T @ x, dW2=dy.T @ h)


def gemm(A, B, R=None, a_layout: int = 0, b_layout: int = 0):
    """C[M,N] = A B^T (+ R) with A given as [M,K] (a_layout 0) or [K,M] (1) and B as [N,K] (0) or [K,N] (1)."""
    A, B = _f64(A), _f64(B)
    A2 = A.T if a_layout else A
    B2 = B.T if b_layout else B
    C = A2 @ B2.T
    return C if R is None else C + _f64(R)


def transformer_block_fwd_bwd(x, w, dy, B: int, n: int, H: int, causal: bool, eps: float):
    """One pre-norm transformer block over T = B*n tokens of width dm = H*d, forward and backward:

        h1 = RMSNorm(x; g1)        q, k, v = h1 Wq^T, h1 Wk^T, h1 Wv^T      (heads: columns h*d .. (h+1)*d)
        o  = softmax(q k^T / sqrt(d)) v per (sequence, head)                 x2 = x + o Wo^T
        h2 = RMSNorm(x2; g2)       y = x2 + gated_mlp(h2; W1, W3, W2)

    (the pieces the paper's block section lists: two norms, the QKV projection, attention, the FFN).
    x, dy: [T,dm]; w: dict with g1, g2 [dm], Wq, Wk, Wv, Wo [dm,dm], W1, W3 [d_ff,dm], W2 [dm,d_ff].
    Returns y and the gradients dx and d<name> for every entry of w, float64.  Composed from this
    package's own pieces (rmsnorm_fwd_bwd, gated_mlp_fwd_bwd, the attention oracle); the composition is
    pinned against the library's autograd in the tests."""
    from .attention import attn_fwd_bwd
    x, dy = _f64(x), _f64(dy)
    w = {k: _f64(v) for k, v in w.items()}
    T, dm = x.shape
    d = dm // H
    if T != B * n or dm != H * d:
        raise ValueError("expected x [B*n, H*d]")

    def heads(t):      # [T,dm] -> [B,H,n,d]
        return np.ascontiguousarray(t.reshape(B, n, H, d).transpose(0, 2, 1, 3))

    def tokens(t):     # [B,H,n,d] -> [T,dm]
        return np.ascontiguousarray(t.transpose(0, 2, 1, 3).reshape(T, dm))

    zeros = np.zeros_like(x)
    n1 = rmsnorm_fwd_bwd(x, w["g1"], zeros, eps)
    h1 = n1["y"]
    q, k, v = h1 @ w["Wq"].T, h1 @ w["Wk"].T, h1 @ w["Wv"].T
    scale = 1.0 / np.sqrt(d)
    # forward values first (the attention oracle wants dO: run it again once dO is known)
    att0 = attn_fwd_bwd(heads(q), heads(k), heads(v), heads(zeros), causal, scale)
    o = tokens(att0["O"])
    x2 = x + o @ w["Wo"].T
    n2 = rmsnorm_fwd_bwd(x2, w["g2"], zeros, eps)
    h2 = n2["y"]
    mlp = gated_mlp_fwd_bwd(h2, w["W1"], w["W3"], w["W2"], dy)
    y = x2 + mlp["y"]
    # backward
    out = dict(y=y, dW1=mlp["dW1"], dW3=mlp["dW3"], dW2=mlp["dW2"])
    b2 = rmsnorm_fwd_bwd(x2, w["g2"], mlp["dx"], eps)
    out["dg2"] = b2["dg"]
    dx2 = dy + b2["dx"]
    out["dWo"] = dx2.T @ o
    do = dx2 @ w["Wo"]
    att = attn_fwd_bwd(heads(q), heads(k), heads(v), heads(do), causal, scale)
    dq, dk, dv = tokens(att["dQ"]), tokens(att["dK"]), tokens(att["dV"])
    out["dWq"], out["dWk"], out["dWv"] = dq.T @ h1, dk.T @ h1, dv.T @ h1
    dh1 = dq @ w["Wq"] + dk @ w["Wk"] + dv @ w["Wv"]
    b1 = rmsnorm_fwd_bwd(x, w["g1"], dh1, eps)
    out["dg1"] = b1["dg"]
    out["dx"] = dx2 + b1["dx"]
    return out
