"""Block pieces (RMSNorm, gated MLP; include/moa_block.h) against the fp64 oracle, through the C ABI.
Bar: max|err|/max|ref| <= 1e-2 per output (bf16 storage, fp32 arithmetic)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2609_33916_b200 import inputs as mi

TOL = 1e-2


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


def _dev(torch, bits):
    return torch.from_numpy(np.ascontiguousarray(bits)).view(torch.bfloat16).cuda()


def _host(t):
    return t.float().cpu().numpy().astype(np.float64)


def _nan_like(torch, shape, dtype=None):
    return torch.full(shape, float("nan"), dtype=dtype or torch.bfloat16, device="cuda")


# ------------------------------------------------------------------------------ RMSNorm
def _run_rmsnorm(rt, inp, eps, give_r=True):
    torch, mb = rt
    n, d = inp["x"].shape
    x, g, dy = (_dev(torch, inp[k]) for k in ("x", "g", "dy"))
    desc = mb.make_rmsnorm_desc(n, d, eps)
    y, dx = _nan_like(torch, (n, d)), _nan_like(torch, (n, d))
    dg = _nan_like(torch, (d,))
    r = _nan_like(torch, (n,), torch.float32)
    ws = torch.full((max(mb.moa_rmsnorm_workspace_bytes(desc), 16),), 0xFF, dtype=torch.uint8, device="cuda")
    mb.moa_rmsnorm_fwd(desc, x, g, y, r)
    mb.moa_rmsnorm_bwd(desc, x, g, r if give_r else None, dy, dx, dg, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    return dict(y=_host(y), r=_host(r), dx=_host(dx), dg=_host(dg))


@pytest.mark.parametrize("n,d", [(1, 8), (5, 64), (33, 128), (257, 768), (100, 1024), (64, 2048), (70, 2056),
                                 (19, 4096), (9, 5120), (7, 8192), (3000, 512), (4099, 2048), (2500, 4096), (1031, 3000), (600, 2560)])
@pytest.mark.parametrize("eps", [1e-5, 0.5])
def test_rmsnorm_matches_oracle(rt, n, d, eps):
    inp = mi.make_norm_inputs(n, d, seed=1000 + n + d)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.rmsnorm_fwd_bwd(f["x"], f["g"], f["dy"], eps)
    for give_r in (True, False):
        got = _run_rmsnorm(rt, inp, eps, give_r)
        for k in ("y", "dx", "dg"):
            assert np.all(np.isfinite(got[k])), k
            assert mi.rel_err(got[k], ref[k]) <= TOL, (k, n, d, mi.rel_err(got[k], ref[k]))
        assert mi.rel_err(got["r"], ref["r"]) <= 1e-5


def test_rmsnorm_is_bitwise_reproducible(rt):
    inp = mi.make_norm_inputs(5000, 1024, seed=3)
    a = _run_rmsnorm(rt, inp, 1e-6)
    b = _run_rmsnorm(rt, inp, 1e-6)
    for k in ("y", "dx", "dg", "r"):
        np.testing.assert_array_equal(a[k], b[k], err_msg=k)


def test_rmsnorm_rows_far_from_unit_scale(rt):
    """Rows scaled by 2^-20 .. 2^20: the normalised output does not change (eps = 0) and nothing overflows."""
    inp = mi.make_norm_inputs(64, 512, seed=4)
    x = mi.bf16_bits_to_f32(inp["x"])
    scales = np.float32(2.0) ** np.arange(-20, 44)[:64].clip(-20, 20).astype(np.float32)
    inp2 = dict(inp, x=mi.f32_to_bf16_bits(x * scales[:, None]))     # powers of two: exact in bf16
    a = _run_rmsnorm(rt, inp, 0.0)
    b = _run_rmsnorm(rt, inp2, 0.0)
    np.testing.assert_allclose(b["y"], a["y"], rtol=1e-2, atol=1e-2)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp2.items()}
    ref = oracle.rmsnorm_fwd_bwd(f["x"], f["g"], f["dy"], 0.0)
    assert mi.rel_err(b["dg"], ref["dg"]) <= TOL
    # dx rows scale like 1/row scale: compare row by row
    for i in range(64):
        assert mi.rel_err(b["dx"][i], ref["dx"][i]) <= TOL, i


# ---------------------------------------------------------------------------- gated MLP
def _run_mlp(rt, inp):
    torch, mb = rt
    n, d = inp["x"].shape
    dff = inp["W1"].shape[0]
    x, W1, W3, W2, dy = (_dev(torch, inp[k]) for k in ("x", "W1", "W3", "W2", "dy"))
    desc = mb.make_mlp_desc(n, d, dff)
    a, u, h = (_nan_like(torch, (n, dff)) for _ in range(3))
    y, dx = _nan_like(torch, (n, d)), _nan_like(torch, (n, d))
    dW1, dW3, dW2 = _nan_like(torch, (dff, d)), _nan_like(torch, (dff, d)), _nan_like(torch, (d, dff))
    ws = torch.full((max(mb.moa_gated_mlp_workspace_bytes(desc), 16),), 0xFF, dtype=torch.uint8, device="cuda")
    mb.moa_gated_mlp_fwd(desc, x, W1, W3, W2, a, u, h, y)
    mb.moa_gated_mlp_bwd(desc, x, W1, W3, W2, a, u, h, dy, dx, dW1, dW3, dW2, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    return {k: _host(v) for k, v in dict(a=a, u=u, h=h, y=y, dx=dx, dW1=dW1, dW3=dW3, dW2=dW2).items()}


MLP_CASES = [
    (128, 64, 256),          # one tile everywhere; the sizes of the paper's own traffic check (n = 512 there)
    (512, 64, 256),
    (1, 8, 8),               # smallest
    (130, 72, 264),          # ragged in every dimension
    (300, 512, 1024),
    (1000, 256, 2048),       # several tiles, K of the weight-gradient GEMMs not a multiple of 64
    (2048, 1024, 4096),
]


@pytest.mark.parametrize("n,d,dff", MLP_CASES)
def test_gated_mlp_matches_oracle(rt, n, d, dff):
    inp = mi.make_mlp_inputs(n, d, dff, seed=2000 + n + d)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.gated_mlp_fwd_bwd(f["x"], f["W1"], f["W3"], f["W2"], f["dy"])
    got = _run_mlp(rt, inp)
    for k in ("a", "u", "h", "y", "dx", "dW1", "dW3", "dW2"):
        assert np.all(np.isfinite(got[k])), k
        e = mi.rel_err(got[k], ref[k])
        assert e <= TOL, (k, n, d, dff, e)


def test_gated_mlp_backward_from_its_stored_activations(rt):
    """The backward reads the bf16 a, u, h its forward stored: against the oracle's backward evaluated on
    exactly those stored values, the gradients agree more closely than against the one-piece definition."""
    n, d, dff = 384, 256, 768
    inp = mi.make_mlp_inputs(n, d, dff, seed=77)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    got = _run_mlp(rt, inp)
    ref = oracle.gated_mlp_bwd_from_saved(f["x"], got["a"], got["u"], f["W1"], f["W3"], f["W2"], f["dy"])
    for k in ("dx", "dW1", "dW3"):
        assert mi.rel_err(got[k], ref[k]) <= 6e-3, (k, mi.rel_err(got[k], ref[k]))
    # dW2 = dy^T h with the stored h
    assert mi.rel_err(got["dW2"], f["dy"].T @ got["h"]) <= 6e-3


def test_gated_mlp_large_preactivations(rt):
    """Weights scaled so that |a| reaches the hundreds: the sigmoid saturates without NaN or inf."""
    n, d, dff = 256, 128, 512
    inp = mi.make_mlp_inputs(n, d, dff, seed=88)
    w1 = mi.bf16_bits_to_f32(inp["W1"]) * np.float32(64.0)
    inp = dict(inp, W1=mi.f32_to_bf16_bits(w1))
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.gated_mlp_fwd_bwd(f["x"], f["W1"], f["W3"], f["W2"], f["dy"])
    got = _run_mlp(rt, inp)
    for k in ("h", "y", "dx", "dW1", "dW3", "dW2"):
        assert np.all(np.isfinite(got[k])), k
        assert mi.rel_err(got[k], ref[k]) <= TOL, (k, mi.rel_err(got[k], ref[k]))


# ------------------------------------------------------------------- random shapes
def _random_block_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(count):
        n = int(rng.choice([1, 7, 64, 127, 128, 129, 255, 257, 500, 1000, 1111]))
        d = 8 * int(rng.integers(1, 80))                 # 8 .. 632
        dff = 8 * int(rng.integers(1, 160))              # 8 .. 1272
        out.append((i, n, d, dff))
    return out


@pytest.mark.parametrize("case", _random_block_cases(24, 20261127), ids=lambda c: f"{c[0]}-n{c[1]}-d{c[2]}-ff{c[3]}")
def test_random_block_shapes(rt, case):
    """Random token counts and widths (multiples of 8, tails in every tile dimension): both pieces against the oracle."""
    i, n, d, dff = case
    inp = mi.make_mlp_inputs(n, d, dff, seed=5000 + i)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.gated_mlp_fwd_bwd(f["x"], f["W1"], f["W3"], f["W2"], f["dy"])
    got = _run_mlp(rt, inp)
    for k in ("a", "u", "h", "y", "dx", "dW1", "dW3", "dW2"):
        assert np.all(np.isfinite(got[k])), k
        e = mi.rel_err(got[k], ref[k])
        assert e <= TOL, (k, case, e)
    ninp = mi.make_norm_inputs(n, d, seed=6000 + i)
    f = {k: mi.to_f64(v, "bf16") for k, v in ninp.items()}
    eps = float(np.random.default_rng(i).choice([0.0, 1e-6, 1e-2]))
    nref = oracle.rmsnorm_fwd_bwd(f["x"], f["g"], f["dy"], eps)
    ngot = _run_rmsnorm(rt, ninp, eps, give_r=bool(i % 2))
    for k in ("y", "dx", "dg"):
        assert np.all(np.isfinite(ngot[k])), k
        assert mi.rel_err(ngot[k], nref[k]) <= TOL, (k, case, mi.rel_err(ngot[k], nref[k]))


def test_gated_mlp_is_bitwise_reproducible(rt):
    inp = mi.make_mlp_inputs(700, 264, 520, seed=99)
    a = _run_mlp(rt, inp)
    b = _run_mlp(rt, inp)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k], err_msg=k)


def test_rmsnorm_long_run_through_the_ring(rt):
    """n = 32768 rows of 2048 (many trips round the shared-memory ring in every CTA): all of y, dx, dg against
    the oracle, and 200 repeated forward+backward launches give identical bits (no stage taken for another)."""
    torch, mb = rt
    n, d, eps = 32768, 2048, 1e-5
    inp = mi.make_norm_inputs(n, d, seed=31)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.rmsnorm_fwd_bwd(f["x"], f["g"], f["dy"], eps)
    first = _run_rmsnorm(rt, inp, eps)
    for k in ("y", "dx", "dg"):
        assert mi.rel_err(first[k], ref[k]) <= TOL, (k, mi.rel_err(first[k], ref[k]))
    x, g, dy = (_dev(torch, inp[k]) for k in ("x", "g", "dy"))
    desc = mb.make_rmsnorm_desc(n, d, eps)
    y, dx, dg = torch.empty_like(x), torch.empty_like(x), torch.empty_like(g)
    r = torch.empty((n,), dtype=torch.float32, device="cuda")
    ws = torch.empty(mb.moa_rmsnorm_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    y0 = dx0 = dg0 = None
    for it in range(200):
        mb.moa_rmsnorm_fwd(desc, x, g, y, r)
        mb.moa_rmsnorm_bwd(desc, x, g, r, dy, dx, dg, ws)
        if it % 50 == 0:
            if y0 is None:
                y0, dx0, dg0 = y.clone(), dx.clone(), dg.clone()
            else:
                assert torch.equal(y, y0) and torch.equal(dx, dx0) and torch.equal(dg, dg0), it
    assert mb.moa_last_device_status() == mb.MOA_OK
    assert torch.equal(y, y0) and torch.equal(dx, dx0) and torch.equal(dg, dg0)


# ------------------------------------------------------------------------------- GEMM
def _bits(rng, shape, scale=1.0):
    return mi.f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


@pytest.mark.parametrize("a_layout,b_layout", [(0, 0), (0, 1), (1, 1), (1, 0)])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (8, 8, 8), (130, 264, 72), (1000, 512, 2048), (384, 1032, 520)])
@pytest.mark.parametrize("with_r", [False, True])
def test_gemm_layouts_match_oracle(rt, a_layout, b_layout, M, N, K, with_r):
    torch, mb = rt
    if a_layout and M % 8:
        pytest.skip("rows of A = [K,M] must be 16-byte multiples")
    rng = np.random.default_rng(M + N + K + 7 * a_layout + 3 * b_layout)
    A = _bits(rng, (K, M) if a_layout else (M, K))
    Bm = _bits(rng, (K, N) if b_layout else (N, K), 1.0 / np.sqrt(K))
    R = _bits(rng, (M, N)) if with_r else None
    ref = oracle.gemm(mi.to_f64(A, "bf16"), mi.to_f64(Bm, "bf16"), None if R is None else mi.to_f64(R, "bf16"), a_layout, b_layout)
    C = _nan_like(torch, (M, N))
    mb.moa_gemm(mb.make_gemm_desc(M, N, K, a_layout, b_layout), _dev(torch, A), _dev(torch, Bm), C,
                R=None if R is None else _dev(torch, R))
    assert mb.moa_last_device_status() == mb.MOA_OK
    got = _host(C)
    assert np.all(np.isfinite(got))
    assert mi.rel_err(got, ref) <= TOL, mi.rel_err(got, ref)


def test_residual_arguments(rt):
    """dx_add of the RMSNorm backward and res of the gated-MLP forward: the same as adding afterwards (in fp64)."""
    torch, mb = rt
    n, d, dff = 300, 512, 1024
    rng = np.random.default_rng(5)
    ninp = mi.make_norm_inputs(n, d, seed=8)
    add = _bits(rng, (n, d))
    f = {k: mi.to_f64(v, "bf16") for k, v in ninp.items()}
    ref = oracle.rmsnorm_fwd_bwd(f["x"], f["g"], f["dy"], 1e-5)
    x, g, dy = (_dev(torch, ninp[k]) for k in ("x", "g", "dy"))
    desc = mb.make_rmsnorm_desc(n, d, 1e-5)
    dx, dg = _nan_like(torch, (n, d)), _nan_like(torch, (d,))
    ws = torch.empty(mb.moa_rmsnorm_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    mb.moa_rmsnorm_bwd(desc, x, g, None, dy, dx, dg, ws, dx_add=_dev(torch, add))
    assert mi.rel_err(_host(dx), ref["dx"] + mi.to_f64(add, "bf16")) <= TOL
    assert mi.rel_err(_host(dg), ref["dg"]) <= TOL
    minp = mi.make_mlp_inputs(n, d, dff, seed=9)
    f = {k: mi.to_f64(v, "bf16") for k, v in minp.items()}
    mref = oracle.gated_mlp_fwd_bwd(f["x"], f["W1"], f["W3"], f["W2"], f["dy"])
    x, W1, W3, W2 = (_dev(torch, minp[k]) for k in ("x", "W1", "W3", "W2"))
    a, u, h = (_nan_like(torch, (n, dff)) for _ in range(3))
    y = _nan_like(torch, (n, d))
    mb.moa_gated_mlp_fwd(mb.make_mlp_desc(n, d, dff), x, W1, W3, W2, a, u, h, y, res=_dev(torch, add))
    assert mb.moa_last_device_status() == mb.MOA_OK
    assert mi.rel_err(_host(y), mref["y"] + mi.to_f64(add, "bf16")) <= TOL


# ------------------------------------------------------- the block, composed from the pieces
def run_block(torch, mb, inp, B, n, H, causal, eps):
    """One pre-norm transformer block forward+backward as a sequence of library calls (every step a kernel of the
    library; this function only passes pointers): RMSNorm, three projections, attention on token-major tensors,
    output projection + residual, RMSNorm, gated MLP + residual; then the backward of each, in reverse."""
    bf = torch.bfloat16
    dev = {k: _dev(torch, v) for k, v in inp.items()}
    T, dm = inp["x"].shape
    d, dff = dm // H, inp["W1"].shape[0]
    E = lambda *s: torch.full(s, float("nan"), dtype=bf, device="cuda")
    nd = mb.make_rmsnorm_desc(T, dm, eps)
    nws = torch.empty(mb.moa_rmsnorm_workspace_bytes(nd), dtype=torch.uint8, device="cuda")
    ad = mb.make_desc(B, H, n, d, causal, 1.0 / np.sqrt(d), layout=mb.MOA_LAYOUT_BNHD)
    aws = torch.empty(max(16, mb.moa_attn_workspace_bytes(ad, mb.MOA_OP_BWD)), dtype=torch.uint8, device="cuda")
    md = mb.make_mlp_desc(T, dm, dff)
    mws = torch.empty(mb.moa_gated_mlp_workspace_bytes(md), dtype=torch.uint8, device="cuda")
    proj = mb.make_gemm_desc(T, dm, dm)                  # y = x W^T
    back = mb.make_gemm_desc(T, dm, dm, 0, 1)            # dx = dy W
    wgrad = mb.make_gemm_desc(dm, dm, T, 1, 1)           # dW = dy^T x
    # ---- forward
    h1, r1 = E(T, dm), torch.empty((T,), dtype=torch.float32, device="cuda")
    mb.moa_rmsnorm_fwd(nd, dev["x"], dev["g1"], h1, r1)
    q, k, v = E(T, dm), E(T, dm), E(T, dm)
    for W, out in (("Wq", q), ("Wk", k), ("Wv", v)):
        mb.moa_gemm(proj, h1, dev[W], out)
    o, L = E(T, dm), torch.empty((B, H, n), dtype=torch.float32, device="cuda")
    mb.moa_attn_fwd(ad, q, k, v, o, L, aws)
    x2 = E(T, dm)
    mb.moa_gemm(proj, o, dev["Wo"], x2, R=dev["x"])
    h2, r2 = E(T, dm), torch.empty((T,), dtype=torch.float32, device="cuda")
    mb.moa_rmsnorm_fwd(nd, x2, dev["g2"], h2, r2)
    a, u, h, y = E(T, dff), E(T, dff), E(T, dff), E(T, dm)
    mb.moa_gated_mlp_fwd(md, h2, dev["W1"], dev["W3"], dev["W2"], a, u, h, y, res=x2)
    # ---- backward
    g = {}
    dh2 = E(T, dm)
    g["dW1"], g["dW3"], g["dW2"] = E(dff, dm), E(dff, dm), E(dm, dff)
    mb.moa_gated_mlp_bwd(md, h2, dev["W1"], dev["W3"], dev["W2"], a, u, h, dev["dy"], dh2, g["dW1"], g["dW3"], g["dW2"], mws)
    dx2, g["dg2"] = E(T, dm), E(dm)
    mb.moa_rmsnorm_bwd(nd, x2, dev["g2"], r2, dh2, dx2, g["dg2"], nws, dx_add=dev["dy"])
    g["dWo"], do = E(dm, dm), E(T, dm)
    mb.moa_gemm(wgrad, dx2, o, g["dWo"])
    mb.moa_gemm(back, dx2, dev["Wo"], do)
    dq, dk, dv = E(T, dm), E(T, dm), E(T, dm)
    mb.moa_attn_bwd(ad, q, k, v, o, L, do, dq, dk, dv, aws)
    dh1 = E(T, dm)
    mb.moa_gemm(back, dq, dev["Wq"], dh1)
    mb.moa_gemm(back, dk, dev["Wk"], dh1, R=dh1)
    mb.moa_gemm(back, dv, dev["Wv"], dh1, R=dh1)
    for W, dt in (("dWq", dq), ("dWk", dk), ("dWv", dv)):
        g[W] = E(dm, dm)
        mb.moa_gemm(wgrad, dt, h1, g[W])
    g["dx"], g["dg1"] = E(T, dm), E(dm)
    mb.moa_rmsnorm_bwd(nd, dev["x"], dev["g1"], r1, dh1, g["dx"], g["dg1"], nws, dx_add=dx2)
    assert mb.moa_last_device_status() == mb.MOA_OK
    g["y"] = y
    return {k_: _host(v_) for k_, v_ in g.items()}


def make_block_inputs(B, n, H, d, dff, seed):
    rng = np.random.default_rng(seed)
    T, dm = B * n, H * d
    f = lambda shape, s=1.0: mi.f32_to_bf16_bits((s * rng.standard_normal(shape)).astype(np.float32))
    return dict(x=f((T, dm)), dy=f((T, dm)), g1=mi.f32_to_bf16_bits((1 + 0.25 * rng.standard_normal(dm)).astype(np.float32)),
                g2=mi.f32_to_bf16_bits((1 + 0.25 * rng.standard_normal(dm)).astype(np.float32)),
                Wq=f((dm, dm), dm ** -0.5), Wk=f((dm, dm), dm ** -0.5), Wv=f((dm, dm), dm ** -0.5), Wo=f((dm, dm), dm ** -0.5),
                W1=f((dff, dm), dm ** -0.5), W3=f((dff, dm), dm ** -0.5), W2=f((dm, dff), dff ** -0.5))


@pytest.mark.parametrize("B,n,H,d,dff,causal", [(1, 128, 2, 64, 256, False), (2, 256, 4, 64, 512, True), (1, 300, 2, 128, 520, True),
                                                (2, 512, 8, 128, 2048, False)])
def test_transformer_block_composed_from_the_pieces(rt, B, n, H, d, dff, causal):
    """The complete block (two norms, QKV projection, attention, output projection, gated MLP, two residual
    connections) forward+backward as 20 library calls against the fp64 block oracle.  Errors of the bf16 stages
    compound along the block, so the bar here is 2e-2 of each tensor's max (each piece alone is held to 1e-2)."""
    torch, mb = rt
    inp = make_block_inputs(B, n, H, d, dff, seed=70 + n)
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    w = {k: f[k] for k in ("g1", "g2", "Wq", "Wk", "Wv", "Wo", "W1", "W3", "W2")}
    ref = oracle.transformer_block_fwd_bwd(f["x"], w, f["dy"], B, n, H, causal, 1e-5)
    got = run_block(torch, mb, inp, B, n, H, causal, 1e-5)
    for k in ref:
        assert np.all(np.isfinite(got[k])), k
        e = mi.rel_err(got[k], ref[k])
        assert e <= 2e-2, (k, e)


def test_gated_mlp_full_bench_size_sampled(rt):
    """The benchmark's size (n 16384, d 2048, d_ff 8192), in the launch configuration the benchmark times: sampled
    token rows (a, u, h, y, dx are row-local) and sampled hidden units (columns of a, u, h, da, du give dW2[:,k],
    dW1[k,:], dW3[k,:]) against fp64 evaluations of the definition."""
    torch, mb = rt
    n, d, dff = 16384, 2048, 8192
    gen = torch.Generator(device="cuda").manual_seed(23)
    bf = torch.bfloat16
    rnd = lambda *shape, s=1.0: (torch.randn(shape, generator=gen, device="cuda") * s).to(bf)
    x, dy = rnd(n, d), rnd(n, d)
    W1, W3, W2 = rnd(dff, d, s=d ** -0.5), rnd(dff, d, s=d ** -0.5), rnd(d, dff, s=dff ** -0.5)
    a, u, h = (_nan_like(torch, (n, dff)) for _ in range(3))
    y, dx = _nan_like(torch, (n, d)), _nan_like(torch, (n, d))
    dW1, dW3, dW2 = _nan_like(torch, (dff, d)), _nan_like(torch, (dff, d)), _nan_like(torch, (d, dff))
    desc = mb.make_mlp_desc(n, d, dff)
    ws = torch.empty(mb.moa_gated_mlp_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    mb.moa_gated_mlp_fwd(desc, x, W1, W3, W2, a, u, h, y)
    mb.moa_gated_mlp_bwd(desc, x, W1, W3, W2, a, u, h, dy, dx, dW1, dW3, dW2, ws)
    assert mb.moa_last_device_status() == mb.MOA_OK
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    xf, dyf, w1, w3, w2 = f64(x), f64(dy), f64(W1), f64(W3), f64(W2)
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([[0, 127, 128, n - 1], rng.integers(0, n, 28)]))
    ref = oracle.gated_mlp_fwd_bwd(xf[rows], w1, w3, w2, dyf[rows])          # row-local outputs of the sampled rows
    for k, t in (("a", a), ("u", u), ("h", h), ("y", y), ("dx", dx)):
        e = mi.rel_err(f64(t[torch.from_numpy(rows).cuda()]), ref[k])
        assert e <= TOL, (k, e)
    units = np.unique(np.concatenate([[0, 127, 128, dff - 1], rng.integers(0, dff, 12)]))
    sig = lambda v: 1.0 / (1.0 + np.exp(-v))
    ak, uk = xf @ w1[units].T, xf @ w3[units].T                                # [n, units]
    hk = ak * sig(ak) * uk
    dhk = dyf @ w2[:, units]
    dak = dhk * uk * sig(ak) * (1.0 + ak * (1.0 - sig(ak)))
    duk = dhk * ak * sig(ak)
    ut = torch.from_numpy(units).cuda()
    assert mi.rel_err(f64(dW2[:, ut]), dyf.T @ hk) <= TOL
    assert mi.rel_err(f64(dW1[ut]), dak.T @ xf) <= TOL
    assert mi.rel_err(f64(dW3[ut]), duk.T @ xf) <= TOL
    for t in (y, dx, dW1, dW3, dW2, a, u, h):
        assert bool(torch.isfinite(t.float()).all())


@pytest.mark.parametrize("B,n,H,d,dff,causal", [(2, 256, 4, 64, 512, True), (1, 333, 2, 128, 384, False), (2, 200, 3, 96, 320, True)])
def test_block_class_packed_projection_matches_oracle_and_the_three_gemm_form(rt, B, n, H, d, dff, causal):
    """block.TransformerBlock with one projection GEMM for Q, K and V (a packed [B,n,3,H,d] array read and written by
    the attention through explicit strides) against the fp64 block oracle, and against the same class with three
    projection GEMMs: the forward agrees bit for bit (same products, same attention), gradients to rounding."""
    torch, mb = rt
    from paper_2609_33916_b200.block import TransformerBlock
    inp = make_block_inputs(B, n, H, d, dff, seed=170 + n)
    dev = {k: _dev(torch, v) for k, v in inp.items()}
    w = {k: dev[k] for k in ("g1", "g2", "Wq", "Wk", "Wv", "Wo", "W1", "W3", "W2")}
    out = {}
    for packed in (True, False):
        blk = TransformerBlock(torch, B, n, H, d, dff, causal, packed_qkv=packed)
        wp = blk.prepare_weights(w)
        assert ("Wqkv" in wp) == packed
        blk.forward(dev["x"], wp)
        blk.backward(dev["x"], wp, dev["dy"])
        torch.cuda.synchronize()
        assert mb.moa_last_device_status() == mb.MOA_OK
        got = {"y": _host(blk.y), "dx": _host(blk.dx)}
        for k_, v_ in blk.grads.items():
            got["d" + k_] = _host(v_)
        out[packed] = got
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    wf = {k: f[k] for k in ("g1", "g2", "Wq", "Wk", "Wv", "Wo", "W1", "W3", "W2")}
    ref = oracle.transformer_block_fwd_bwd(f["x"], wf, f["dy"], B, n, H, causal, 1e-5)
    np.testing.assert_array_equal(out[True]["y"], out[False]["y"])
    for k_ in out[True]:
        assert mi.rel_err(out[True][k_], ref[k_]) <= 2e-2, (k_, mi.rel_err(out[True][k_], ref[k_]))
        assert mi.rel_err(out[True][k_], out[False][k_]) <= 8e-3, k_


def test_block_can_be_captured_in_a_cuda_graph_and_replayed(rt):
    """The calls of a block step allocate nothing and synchronise nothing: recorded once in a CUDA graph, a replay
    gives the bits of a direct run for everything the forward writes, and gradients within rounding of it (the
    attention backward's dQ accumulation order is not fixed in its default mode)."""
    torch, mb = rt
    from paper_2609_33916_b200.block import TransformerBlock
    B, n, H, d, dff = 2, 256, 4, 64, 512
    inp = make_block_inputs(B, n, H, d, dff, seed=5)
    dev = {k: _dev(torch, v) for k, v in inp.items()}
    blk = TransformerBlock(torch, B, n, H, d, dff, True)
    w = blk.prepare_weights({k: dev[k] for k in ("g1", "g2", "Wq", "Wk", "Wv", "Wo", "W1", "W3", "W2")})
    blk.forward(dev["x"], w)
    blk.backward(dev["x"], w, dev["dy"])
    torch.cuda.synchronize()
    y0, dx0 = blk.y.clone(), blk.dx.clone()
    g0 = {k: v.clone() for k, v in blk.grads.items()}
    graph, cap = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=cap):
        s = torch.cuda.current_stream()
        blk.forward(dev["x"], w, s)
        blk.backward(dev["x"], w, dev["dy"], s)
    blk.y.zero_(); blk.dx.zero_()
    for v in blk.grads.values():
        v.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert mb.moa_last_device_status() == mb.MOA_OK
    assert torch.equal(blk.y, y0)
    assert mi.rel_err(_host(blk.dx), _host(dx0)) <= 8e-3
    for k, v in blk.grads.items():
        assert mi.rel_err(_host(v), _host(g0[k])) <= 8e-3, k
