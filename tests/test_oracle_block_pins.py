"""Pins of the block-piece oracle (RMSNorm, gated MLP; oracle/block.py) against things other than
itself: closed forms worked by hand, the library's own routines differentiated by autograd,
central finite differences, and identities that hold for any input.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import block as ob


def _rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------------------ RMSNorm
def test_rmsnorm_closed_forms():
    g = np.array([1.0, -2.0, 0.5, 3.0])
    # a constant row c*1: mean square c^2, so y = sign(c) g exactly (eps = 0)
    for c in (2.5, -0.75):
        r = ob.rmsnorm_fwd_bwd(np.full((1, 4), c), g, np.ones((1, 4)), 0.0)
        np.testing.assert_allclose(r["y"][0], math.copysign(1.0, c) * g, rtol=0, atol=1e-15)
        np.testing.assert_allclose(r["r"][0], 1.0 / abs(c), rtol=1e-15)
    # a one-hot row a*e_2: mean square a^2/d, y_2 = sign(a) sqrt(d) g_2, the rest 0
    x = np.zeros((1, 4)); x[0, 2] = -3.0
    r = ob.rmsnorm_fwd_bwd(x, g, np.ones((1, 4)), 0.0)
    np.testing.assert_allclose(r["y"][0], [0, 0, -2.0 * 0.5, 0], atol=1e-15)
    # eps only: x = 0 gives y = 0, r = eps^-1/2, dx = r g dy, dg = 0
    dy = np.array([[1.0, 2.0, 3.0, 4.0]])
    r = ob.rmsnorm_fwd_bwd(np.zeros((1, 4)), g, dy, 0.25)
    np.testing.assert_allclose(r["r"], [2.0])
    np.testing.assert_allclose(r["dx"], 2.0 * g * dy)
    np.testing.assert_allclose(r["dg"], 0.0)
    # d = 1, eps = 0: y = sign(x) g is locally constant in x, so dx = 0; dg = dy * sign(x)
    r = ob.rmsnorm_fwd_bwd(np.array([[-4.0]]), np.array([3.0]), np.array([[5.0]]), 0.0)
    np.testing.assert_allclose(r["y"], [[-3.0]])
    np.testing.assert_allclose(r["dx"], [[0.0]], atol=1e-15)
    np.testing.assert_allclose(r["dg"], [-5.0])


@pytest.mark.parametrize("eps", [0.0, 1e-5, 0.3])
def test_rmsnorm_matches_library_autograd(eps):
    rng = _rng(5)
    n, d = 9, 7
    x, g, dy = rng.standard_normal((n, d)), rng.standard_normal(d), rng.standard_normal((n, d))
    xt = torch.tensor(x, requires_grad=True)
    gt = torch.tensor(g, requires_grad=True)
    yt = torch.nn.functional.rms_norm(xt, (d,), weight=gt, eps=eps)
    yt.backward(torch.tensor(dy))
    r = ob.rmsnorm_fwd_bwd(x, g, dy, eps)
    np.testing.assert_allclose(r["y"], yt.detach().numpy(), rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(r["dx"], xt.grad.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["dg"], gt.grad.numpy(), rtol=1e-12, atol=1e-13)


def test_rmsnorm_finite_differences():
    rng = _rng(6)
    n, d, eps, hstep = 3, 5, 0.01, 1e-6
    x, g, dy = rng.standard_normal((n, d)), rng.standard_normal(d), rng.standard_normal((n, d))
    r = ob.rmsnorm_fwd_bwd(x, g, dy, eps)

    def loss(xx, gg):
        return float((ob.rmsnorm_fwd_bwd(xx, gg, dy, eps)["y"] * dy).sum())

    for i in range(n):
        for k in range(d):
            e = np.zeros_like(x); e[i, k] = hstep
            assert abs((loss(x + e, g) - loss(x - e, g)) / (2 * hstep) - r["dx"][i, k]) < 1e-7
    for k in range(d):
        e = np.zeros_like(g); e[k] = hstep
        assert abs((loss(x, g + e) - loss(x, g - e)) / (2 * hstep) - r["dg"][k]) < 1e-7


def test_rmsnorm_invariants():
    rng = _rng(7)
    n, d = 6, 16
    x, g, dy = rng.standard_normal((n, d)), rng.standard_normal(d), rng.standard_normal((n, d))
    r0 = ob.rmsnorm_fwd_bwd(x, g, dy, 0.0)
    # eps = 0: y does not change when a row is scaled by a positive number, dx scales by 1/alpha,
    # and every dx row is orthogonal to its x row
    r1 = ob.rmsnorm_fwd_bwd(3.0 * x, g, dy, 0.0)
    np.testing.assert_allclose(r1["y"], r0["y"], rtol=1e-13)
    np.testing.assert_allclose(r1["dx"], r0["dx"] / 3.0, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose((r0["dx"] * x).sum(1), 0.0, atol=1e-13)
    # g = 1, eps = 0: every output row has mean square 1
    y1 = ob.rmsnorm_fwd_bwd(x, np.ones(d), dy, 0.0)["y"]
    np.testing.assert_allclose((y1 * y1).mean(1), 1.0, rtol=1e-13)
    # eps > 0: sum_k dx_ik x_ik = eps r_i^2 sum_k dy_ik y_ik (y is homogeneous of degree 0 only for eps = 0)
    eps = 0.2
    r2 = ob.rmsnorm_fwd_bwd(x, g, dy, eps)
    np.testing.assert_allclose((r2["dx"] * x).sum(1), eps * r2["r"] ** 2 * (dy * r2["y"]).sum(1), rtol=1e-12)
    # rows are independent; dg adds over rows
    ra = ob.rmsnorm_fwd_bwd(x[:2], g, dy[:2], eps)
    rb = ob.rmsnorm_fwd_bwd(x[2:], g, dy[2:], eps)
    np.testing.assert_allclose(np.concatenate([ra["dx"], rb["dx"]]), r2["dx"], rtol=1e-14)
    np.testing.assert_allclose(ra["dg"] + rb["dg"], r2["dg"], rtol=1e-13)


# ---------------------------------------------------------------------------- gated MLP
def test_gated_mlp_scalar_closed_forms():
    one = lambda v: np.array([[float(v)]])
    # a = 0: silu(0) = 0 and silu'(0) = 1/2
    r = ob.gated_mlp_fwd_bwd(one(1), one(0), one(2), one(3), one(1))
    assert r["h"][0, 0] == 0.0 and r["y"][0, 0] == 0.0
    np.testing.assert_allclose(r["dW1"], [[3.0]])       # da = dh u / 2 = 3 * 2 / 2, times x = 1
    np.testing.assert_allclose(r["dW3"], [[0.0]])
    np.testing.assert_allclose(r["dW2"], [[0.0]])
    np.testing.assert_allclose(r["dx"], [[0.0]])        # da W1 + du W3 = 3*0 + 0*2
    # a = ln 3: sigmoid = 3/4, silu = (3/4) ln 3, silu' = (3/4)(1 + ln3/4)
    l3 = math.log(3.0)
    r = ob.gated_mlp_fwd_bwd(one(1), one(l3), one(1), one(1), one(1))
    np.testing.assert_allclose(r["y"], [[0.75 * l3]], rtol=1e-15)
    da, du = 0.75 * (1 + l3 / 4), 0.75 * l3
    np.testing.assert_allclose(r["dW1"], [[da]], rtol=1e-15)
    np.testing.assert_allclose(r["dW3"], [[du]], rtol=1e-15)
    np.testing.assert_allclose(r["dW2"], [[0.75 * l3]], rtol=1e-15)
    np.testing.assert_allclose(r["dx"], [[da * l3 + du]], rtol=1e-15)
    # far tails: silu(a) -> a for large a, -> 0 for very negative a, without overflow
    r = ob.gated_mlp_fwd_bwd(one(1), one(800.0), one(1), one(1), one(1))
    np.testing.assert_allclose(r["y"], [[800.0]])
    r = ob.gated_mlp_fwd_bwd(one(1), one(-800.0), one(1), one(1), one(1))
    np.testing.assert_allclose(r["y"], [[0.0]], atol=1e-300)
    assert np.all(np.isfinite(r["dx"]))


def test_gated_mlp_matches_library_autograd():
    rng = _rng(11)
    n, d, dff = 7, 5, 9
    x, dy = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    W1, W3, W2 = rng.standard_normal((dff, d)), rng.standard_normal((dff, d)), rng.standard_normal((d, dff))
    t = {k: torch.tensor(v, requires_grad=True) for k, v in dict(x=x, W1=W1, W3=W3, W2=W2).items()}
    F = torch.nn.functional
    y = F.linear(F.silu(F.linear(t["x"], t["W1"])) * F.linear(t["x"], t["W3"]), t["W2"])
    y.backward(torch.tensor(dy))
    r = ob.gated_mlp_fwd_bwd(x, W1, W3, W2, dy)
    np.testing.assert_allclose(r["y"], y.detach().numpy(), rtol=1e-12, atol=1e-13)
    for k, gk in (("dx", "x"), ("dW1", "W1"), ("dW3", "W3"), ("dW2", "W2")):
        np.testing.assert_allclose(r[k], t[gk].grad.numpy(), rtol=1e-11, atol=1e-12, err_msg=k)


def test_gated_mlp_finite_differences():
    rng = _rng(12)
    n, d, dff, hstep = 3, 2, 4, 1e-6
    x, dy = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    W = dict(W1=rng.standard_normal((dff, d)), W3=rng.standard_normal((dff, d)), W2=rng.standard_normal((d, dff)))
    r = ob.gated_mlp_fwd_bwd(x, W["W1"], W["W3"], W["W2"], dy)

    def loss(xx, ww):
        return float((ob.gated_mlp_fwd_bwd(xx, ww["W1"], ww["W3"], ww["W2"], dy)["y"] * dy).sum())

    for idx in np.ndindex(*x.shape):
        e = np.zeros_like(x); e[idx] = hstep
        assert abs((loss(x + e, W) - loss(x - e, W)) / (2 * hstep) - r["dx"][idx]) < 2e-7
    for name in ("W1", "W3", "W2"):
        for idx in np.ndindex(*W[name].shape):
            e = np.zeros_like(W[name]); e[idx] = hstep
            up, dn = dict(W), dict(W)
            up[name] = W[name] + e; dn[name] = W[name] - e
            assert abs((loss(x, up) - loss(x, dn)) / (2 * hstep) - r["d" + name][idx]) < 2e-7, name


def test_gated_mlp_invariants():
    rng = _rng(13)
    n, d, dff = 6, 4, 8
    x, dy = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    W1, W3, W2 = rng.standard_normal((dff, d)), rng.standard_normal((dff, d)), rng.standard_normal((d, dff))
    r = ob.gated_mlp_fwd_bwd(x, W1, W3, W2, dy)
    # the value branch is linear: (W3, W2) -> (c W3, W2 / c) leaves y, dx, dW1 unchanged and moves the
    # factor between dW3 and dW2
    c = 2.5
    s = ob.gated_mlp_fwd_bwd(x, W1, c * W3, W2 / c, dy)
    for k in ("y", "dx", "dW1"):
        np.testing.assert_allclose(s[k], r[k], rtol=1e-12, atol=1e-13, err_msg=k)
    np.testing.assert_allclose(s["dW3"], r["dW3"] / c, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s["dW2"], r["dW2"] * c, rtol=1e-12, atol=1e-13)
    # permuting the hidden units permutes rows of W1, W3, dW1, dW3 and columns of W2, dW2; y, dx unchanged
    perm = rng.permutation(dff)
    s = ob.gated_mlp_fwd_bwd(x, W1[perm], W3[perm], W2[:, perm], dy)
    np.testing.assert_allclose(s["y"], r["y"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s["dx"], r["dx"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s["dW1"], r["dW1"][perm], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s["dW2"], r["dW2"][:, perm], rtol=1e-12, atol=1e-13)
    # tokens are independent: weight gradients add over token blocks
    ra = ob.gated_mlp_fwd_bwd(x[:2], W1, W3, W2, dy[:2])
    rb = ob.gated_mlp_fwd_bwd(x[2:], W1, W3, W2, dy[2:])
    np.testing.assert_allclose(np.concatenate([ra["y"], rb["y"]]), r["y"], rtol=1e-13)
    for k in ("dW1", "dW3", "dW2"):
        np.testing.assert_allclose(ra[k] + rb[k], r[k], rtol=1e-12, atol=1e-13, err_msg=k)
    # sum_i y_i . dy_i = <dW2, W2> (y is linear in W2)
    np.testing.assert_allclose((r["y"] * dy).sum(), (r["dW2"] * W2).sum(), rtol=1e-12)
    # the backward from stored pre-activations agrees with the one-piece definition
    b = ob.gated_mlp_bwd_from_saved(x, r["a"], r["u"], W1, W3, W2, dy)
    for k in ("dx", "dW1", "dW3", "dW2", "h"):
        np.testing.assert_allclose(b[k], r[k], rtol=1e-13, atol=1e-14, err_msg=k)


# ------------------------------------------------------------- GEMM layouts, the whole block
def test_gemm_layouts_by_hand():
    A = np.array([[1.0, 2.0, 3.0], [4.0, 5.0, 6.0]])            # [M=2, K=3]
    Bm = np.array([[1.0, 0.0, -1.0], [2.0, 1.0, 0.0]])           # [N=2, K=3]
    want = np.array([[-2.0, 4.0], [-2.0, 13.0]])                 # rows of A dotted with rows of B
    np.testing.assert_array_equal(ob.gemm(A, Bm), want)
    np.testing.assert_array_equal(ob.gemm(A.T.copy(), Bm, a_layout=1), want)
    np.testing.assert_array_equal(ob.gemm(A, Bm.T.copy(), b_layout=1), want)
    np.testing.assert_array_equal(ob.gemm(A.T.copy(), Bm.T.copy(), a_layout=1, b_layout=1), want)
    np.testing.assert_array_equal(ob.gemm(A, Bm, R=np.ones((2, 2))), want + 1.0)


@pytest.mark.parametrize("causal", [False, True])
def test_transformer_block_matches_library_autograd(causal):
    """The composed block against the library's own routines under autograd (fp64): rms_norm, linear,
    scaled_dot_product_attention, silu."""
    rng = _rng(21)
    B, n, H, d, dff, eps = 2, 5, 3, 4, 7, 1e-3
    T, dm = B * n, H * d
    x, dy = rng.standard_normal((T, dm)), rng.standard_normal((T, dm))
    w = dict(g1=1 + 0.3 * rng.standard_normal(dm), g2=1 + 0.3 * rng.standard_normal(dm),
             Wq=rng.standard_normal((dm, dm)) / 3, Wk=rng.standard_normal((dm, dm)) / 3, Wv=rng.standard_normal((dm, dm)) / 3,
             Wo=rng.standard_normal((dm, dm)) / 3, W1=rng.standard_normal((dff, dm)) / 3, W3=rng.standard_normal((dff, dm)) / 3,
             W2=rng.standard_normal((dm, dff)) / 3)
    ref = ob.transformer_block_fwd_bwd(x, w, dy, B, n, H, causal, eps)
    F = torch.nn.functional
    tx = torch.tensor(x, requires_grad=True)
    tw = {k: torch.tensor(v, requires_grad=True) for k, v in w.items()}

    def heads(t):
        return t.reshape(B, n, H, d).permute(0, 2, 1, 3)

    h1 = F.rms_norm(tx, (dm,), weight=tw["g1"], eps=eps)
    q, k, v = (heads(F.linear(h1, tw[m])) for m in ("Wq", "Wk", "Wv"))
    o = F.scaled_dot_product_attention(q, k, v, is_causal=causal).permute(0, 2, 1, 3).reshape(T, dm)
    x2 = tx + F.linear(o, tw["Wo"])
    h2 = F.rms_norm(x2, (dm,), weight=tw["g2"], eps=eps)
    y = x2 + F.linear(F.silu(F.linear(h2, tw["W1"])) * F.linear(h2, tw["W3"]), tw["W2"])
    y.backward(torch.tensor(dy))
    np.testing.assert_allclose(ref["y"], y.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(ref["dx"], tx.grad.numpy(), rtol=1e-10, atol=1e-11)
    for name in w:
        np.testing.assert_allclose(ref["d" + name], tw[name].grad.numpy(), rtol=1e-10, atol=1e-11, err_msg=name)
