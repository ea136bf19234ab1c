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
