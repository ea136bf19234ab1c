"""The C-ABI library loads and exports every symbol the header declares; host-side
argument checks return the documented codes.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_2609_33916_b200 import binding as mb
from paper_2609_33916_b200 import build as mbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    mbuild.build()
    return mb.lib()


def test_header_symbols_are_exported(lib):
    hdr = "".join(open(os.path.join(ROOT, "include", h)).read() for h in ("moa_attn.h", "moa_block.h"))
    declared = set(re.findall(r"\b(moa_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(mb.EXPORTS), declared ^ set(mb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_strings(lib):
    assert mb.moa_version() >= 100
    assert mb.status_string(mb.MOA_OK) == "ok"
    for s in range(1, 7):
        assert mb.status_string(s) not in ("ok", "unknown status")
    assert mb.status_string(99) == "unknown status"


def test_desc_struct_layout_matches_header():
    assert ctypes.sizeof(mb.moa_attn_desc) == 128        # the same figures are static_asserts in the library
    assert mb.moa_attn_desc.scale.offset == 20
    assert mb.moa_attn_desc.layout.offset == 44
    assert mb.moa_attn_desc.q_stride.offset == 56 and mb.moa_attn_desc.o_stride.offset == 104


def test_workspace_is_linear_in_n(lib):
    def ws(n, mode=mb.MOA_DQ_RED, dtype=mb.MOA_BF16):
        return mb.moa_attn_workspace_bytes(mb.make_desc(1, 32, n, 128, True, 0.1, dtype, mode), mb.MOA_OP_FUSED)
    assert ws(512, mb.MOA_DQ_RED) == 2 * 32 * 512 * 4 + 32 * 512 * 128 * 4
    assert ws(32768) == 64 * ws(512)                      # O(n d): no n^2 term
    assert ws(512, mb.MOA_DQ_SEPARATE_PASS) == 2 * 32 * 512 * 4
    assert ws(512, mb.MOA_DQ_RED, mb.MOA_F32) == 32 * 512 * 4
    assert mb.moa_attn_workspace_bytes(mb.make_desc(1, 32, 512, 128, True, 0.1), mb.MOA_OP_FWD) == 0


def test_materializing_workspace_is_quadratic_and_capped(lib):
    def ws(n, heads=4):
        return mb.moa_attn_workspace_bytes(mb.make_desc(1, heads, n, 128, True, 0.1, materialize=1), mb.MOA_OP_FUSED)
    assert ws(1024) >= 2 * 4 * 1024 * 1024 * 2
    assert ws(2048) > 3.9 * ws(1024)                      # ~n^2
    # heads are processed in groups under a 16 GiB cap for the two arrays
    assert ws(32768, heads=32) <= (16 << 30) + (64 << 20)
    d = mb.make_desc(1, 4, 1024, 128, True, 0.1, materialize=1)
    a = 4096
    assert mb.moa_attn_bwd(d, a, a, a, a, a, a, a, a, a, a, ws_bytes=1 << 40, check=False) == mb.MOA_ERR_UNSUPPORTED
    assert mb.moa_attn_fused_fwd_bwd(d, a, a, a, a, a, a, a, a, a, a, ws_bytes=16, check=False) == mb.MOA_ERR_WORKSPACE
    d32 = mb.make_desc(1, 4, 1024, 128, True, 0.1, mb.MOA_F32, materialize=1)
    assert mb.moa_attn_fwd(d32, a, a, a, a, a, a, ws_bytes=1 << 40, check=False) == mb.MOA_ERR_UNSUPPORTED


def test_argument_errors_need_no_device(lib):
    good = mb.make_desc(1, 1, 128, 64, False, 0.125, mb.MOA_F32)
    a = 4096  # fake, aligned, never dereferenced: checks fail first
    assert mb.moa_attn_fwd(good, 0, a, a, a, a, check=False) == mb.MOA_ERR_INVALID_ARG
    assert mb.moa_attn_fwd(good, a + 2, a, a, a, a, check=False) == mb.MOA_ERR_INVALID_ARG
    for field, val, want in (("n", 0, mb.MOA_ERR_INVALID_ARG), ("d", 96, mb.MOA_ERR_UNSUPPORTED),
                             ("causal", 2, mb.MOA_ERR_INVALID_ARG), ("dtype", 7, mb.MOA_ERR_INVALID_ARG),
                             ("dq_mode", 9, mb.MOA_ERR_INVALID_ARG), ("scale", float("nan"), mb.MOA_ERR_INVALID_ARG)):
        d = mb.make_desc(1, 1, 128, 64, False, 0.125, mb.MOA_F32)
        setattr(d, field, val)
        assert mb.moa_attn_fwd(d, a, a, a, a, a, check=False) == want, field
        assert mb.moa_attn_workspace_bytes(d, mb.MOA_OP_FUSED) == 0
    # backward without / with a short workspace
    d = mb.make_desc(1, 1, 128, 64, False, 0.125, mb.MOA_BF16)
    need = mb.moa_attn_workspace_bytes(d, mb.MOA_OP_BWD)
    assert need > 0
    assert mb.moa_attn_bwd(d, a, a, a, a, a, a, a, a, a, None, check=False) == mb.MOA_ERR_WORKSPACE
    assert mb.moa_attn_bwd(d, a, a, a, a, a, a, a, a, a, a, ws_bytes=need - 1, check=False) == mb.MOA_ERR_WORKSPACE
    assert mb.moa_attn_fused_fwd_bwd(d, a, a, a, a, a, a, a, a, a, a, ws_bytes=need - 1, check=False) == mb.MOA_ERR_WORKSPACE
    with pytest.raises(mb.MoaError):
        mb.moa_attn_fwd(good, 0, a, a, a, a)


def test_other_head_dimensions_argument_checks(lib):
    """Multiples of 8 up to 256 run on the bf16 tensor-core kernels only; above 128 with the plain-red dQ strategy."""
    a = 4096

    def fwd(d, **kw):
        return mb.moa_attn_fwd(mb.make_desc(1, 2, 256, d, True, 0.1, **kw), a, a, a, a, a, check=False)

    def ws(d, **kw):
        return mb.moa_attn_workspace_bytes(mb.make_desc(1, 2, 256, d, True, 0.1, **kw), mb.MOA_OP_FUSED)

    for d in (100, 4, 12, 260, 264, 512):
        assert fwd(d) == mb.MOA_ERR_UNSUPPORTED, d
        assert ws(d) == 0
    for d in (136, 192, 256):
        assert fwd(d, dtype=mb.MOA_F32) == mb.MOA_ERR_UNSUPPORTED
        assert fwd(d, dq_mode=mb.MOA_DQ_BULK_REDUCE) == mb.MOA_ERR_UNSUPPORTED
        assert fwd(d, dq_mode=mb.MOA_DQ_SEPARATE_PASS) == mb.MOA_ERR_UNSUPPORTED
        assert fwd(d, materialize=1) == mb.MOA_ERR_UNSUPPORTED
        # accumulator rows of 256 floats
        assert ws(d) == 2 * (2 * 256 * 4) + 2 * 256 * 256 * 4
    assert fwd(96, dtype=mb.MOA_F32) == mb.MOA_ERR_UNSUPPORTED
    assert fwd(96, path=mb.MOA_PATH_SIMT) == mb.MOA_ERR_UNSUPPORTED
    assert fwd(96, materialize=1) == mb.MOA_ERR_UNSUPPORTED
    assert fwd(32, dq_mode=mb.MOA_DQ_BULK_REDUCE) != mb.MOA_ERR_UNSUPPORTED      # the 64-column kernel has the bulk reduce too
    assert fwd(32, dq_mode=mb.MOA_DQ_BULK_REDUCE, path=mb.MOA_PATH_SIMT) == mb.MOA_ERR_UNSUPPORTED
    # the accumulator rows are as wide as the kernel's head dimension
    assert ws(96) == ws(128) and ws(40) == ws(64) and ws(72) == ws(128)
    assert ws(96, dq_mode=mb.MOA_DQ_SEPARATE_PASS) == ws(128, dq_mode=mb.MOA_DQ_SEPARATE_PASS) < ws(96)
    d96 = mb.make_desc(1, 2, 256, 96, True, 0.1)
    assert mb.moa_attn_fused_rowparallel(d96, a, a, a, a, a, a, a, a, a, 1, a, ws_bytes=1 << 40,
                                         check=False) == mb.MOA_ERR_UNSUPPORTED


def test_shared_kv_heads_argument_checks(lib):
    a = 4096  # fake, aligned, never dereferenced: checks fail first
    def fwd(**kw):
        d = mb.make_desc(1, 8, 256, 128, True, 0.1, **kw)
        return mb.moa_attn_fwd(d, a, a, a, a, a, a, ws_bytes=1 << 40, check=False)
    assert fwd(H_kv=3) == mb.MOA_ERR_INVALID_ARG           # must divide H
    assert fwd(H_kv=16) == mb.MOA_ERR_INVALID_ARG
    assert fwd(H_kv=-1) == mb.MOA_ERR_INVALID_ARG
    assert fwd(H_kv=2, dtype=mb.MOA_F32) == mb.MOA_ERR_UNSUPPORTED      # tensor-core bf16 path only
    assert fwd(H_kv=2, path=mb.MOA_PATH_SIMT) == mb.MOA_ERR_UNSUPPORTED
    assert fwd(H_kv=2, materialize=1) == mb.MOA_ERR_UNSUPPORTED
    assert fwd(layout=2) == mb.MOA_ERR_INVALID_ARG
    assert fwd(layout=1, dtype=mb.MOA_F32) == mb.MOA_ERR_UNSUPPORTED    # token-major: tensor-core bf16 path only
    assert fwd(layout=1, path=mb.MOA_PATH_SIMT) == mb.MOA_ERR_UNSUPPORTED
    assert fwd(layout=1, materialize=1) == mb.MOA_ERR_UNSUPPORTED
    # the workspace does not depend on the number of K/V heads: D, L' and the dQ accumulator are per query head
    w = lambda hkv: mb.moa_attn_workspace_bytes(mb.make_desc(1, 8, 256, 128, True, 0.1, H_kv=hkv), mb.MOA_OP_FUSED)
    assert w(0) == w(8) == w(2) == w(1) > 0


def test_rowparallel_variant_argument_checks(lib):
    a = 4096
    d = mb.make_desc(1, 4, 256, 64, True, 0.1)
    call = lambda desc, sites, wsb=1 << 40: mb.moa_attn_fused_rowparallel(desc, a, a, a, a, a, a, a, a, a, sites, a,
                                                                          ws_bytes=wsb, check=False)
    assert call(d, 0) == mb.MOA_ERR_INVALID_ARG and call(d, 3) == mb.MOA_ERR_INVALID_ARG
    assert call(mb.make_desc(1, 4, 256, 64, True, 0.1, H_kv=2), 2) == mb.MOA_ERR_UNSUPPORTED
    assert call(d, 2, wsb=16) == mb.MOA_ERR_WORKSPACE
    need = mb.moa_attn_workspace_bytes(d, mb.MOA_OP_ROWPARALLEL)
    assert need == 4 * 256 * 4 + 2 * 4 * 256 * 64 * 4          # D + two fp32 accumulators (bf16 tensors)
    d32 = mb.make_desc(1, 4, 256, 64, True, 0.1, mb.MOA_F32)
    assert mb.moa_attn_workspace_bytes(d32, mb.MOA_OP_ROWPARALLEL) == 4 * 256 * 4


def test_decode_argument_checks(lib):
    a = 4096
    call = lambda d, wsb=1 << 40: mb.moa_decode_attn(d, a, a, a, a, a, a, ws_bytes=wsb, check=False)
    assert ctypes.sizeof(mb.moa_decode_desc) == 28
    assert call(mb.make_decode_desc(1, 8, 1024, 128, 0.1, H_kv=3)) == mb.MOA_ERR_INVALID_ARG
    assert call(mb.make_decode_desc(1, 8, 0, 128, 0.1)) == mb.MOA_ERR_INVALID_ARG
    assert call(mb.make_decode_desc(1, 8, 1024, 96, 0.1)) == mb.MOA_ERR_UNSUPPORTED
    d = mb.make_decode_desc(2, 8, 100000, 128, 0.1, H_kv=2)
    need = mb.moa_decode_workspace_bytes(d)
    assert 0 < need <= 1024 * 2 * 8 * 130 * 4                 # segments x heads x (d + 2) floats: independent of n beyond the cap
    assert call(d, wsb=need - 1) == mb.MOA_ERR_WORKSPACE


def test_block_piece_argument_checks(lib):
    a = 4096
    assert ctypes.sizeof(mb.moa_rmsnorm_desc) == 16 and ctypes.sizeof(mb.moa_mlp_desc) == 16
    good = mb.make_rmsnorm_desc(100, 512, 1e-5)
    assert mb.moa_rmsnorm_workspace_bytes(good) > 0
    assert mb.moa_rmsnorm_fwd(good, 0, a, a, None, check=False) == mb.MOA_ERR_INVALID_ARG
    assert mb.moa_rmsnorm_fwd(good, a + 4, a, a, None, check=False) == mb.MOA_ERR_INVALID_ARG
    assert mb.moa_rmsnorm_bwd(good, a, a, None, a, a, a, None, check=False) == mb.MOA_ERR_WORKSPACE
    assert mb.moa_rmsnorm_bwd(good, a, a, None, a, a, a, a, ws_bytes=8, check=False) == mb.MOA_ERR_WORKSPACE
    for n, d, eps, dt, want in ((0, 512, 1e-5, mb.MOA_BF16, mb.MOA_ERR_INVALID_ARG),
                                (10, 100, 1e-5, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED),
                                (10, 16384, 1e-5, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED),
                                (10, 512, -1.0, mb.MOA_BF16, mb.MOA_ERR_INVALID_ARG),
                                (10, 512, float("nan"), mb.MOA_BF16, mb.MOA_ERR_INVALID_ARG),
                                (10, 512, 1e-5, mb.MOA_F32, mb.MOA_ERR_UNSUPPORTED)):
        d_ = mb.make_rmsnorm_desc(n, d, eps, dt)
        assert mb.moa_rmsnorm_fwd(d_, a, a, a, None, check=False) == want, (n, d, eps, dt)
        assert mb.moa_rmsnorm_workspace_bytes(d_) == 0
    m = mb.make_mlp_desc(256, 512, 2048)
    assert mb.moa_gated_mlp_workspace_bytes(m) == 2 * 256 * 2048 * 2
    assert mb.moa_gated_mlp_fwd(m, a, a, a, a, a, a, a, 0, check=False) == mb.MOA_ERR_INVALID_ARG
    assert mb.moa_gated_mlp_fwd(m, a, a, a, a, a, a, a, a, res=a + 8, check=False) == mb.MOA_ERR_INVALID_ARG
    assert ctypes.sizeof(mb.moa_gemm_desc) == 24
    gd = mb.make_gemm_desc(256, 512, 1024)
    assert mb.moa_gemm(gd, a, a, 0, check=False) == mb.MOA_ERR_INVALID_ARG
    assert mb.moa_gemm(gd, a, a, a, R=a + 2, check=False) == mb.MOA_ERR_INVALID_ARG
    for M, N, K, al, bl, dt, want in ((0, 8, 8, 0, 0, mb.MOA_BF16, mb.MOA_ERR_INVALID_ARG), (8, 8, 8, 2, 0, mb.MOA_BF16, mb.MOA_ERR_INVALID_ARG),
                                      (8, 8, 12, 0, 0, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED), (8, 12, 8, 0, 0, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED),
                                      (12, 8, 8, 1, 1, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED), (8, 8, 8, 0, 0, mb.MOA_F32, mb.MOA_ERR_UNSUPPORTED)):
        assert mb.moa_gemm(mb.make_gemm_desc(M, N, K, al, bl, dt), a, a, a, check=False) == want, (M, N, K, al, bl, dt)
    assert mb.moa_gated_mlp_bwd(m, *([a] * 12), None, check=False) == mb.MOA_ERR_WORKSPACE
    for n, d, dff, dt, want in ((0, 512, 2048, mb.MOA_BF16, mb.MOA_ERR_INVALID_ARG),
                                (16, 100, 2048, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED),
                                (16, 512, 2044, mb.MOA_BF16, mb.MOA_ERR_UNSUPPORTED),
                                (16, 512, 2048, mb.MOA_F32, mb.MOA_ERR_UNSUPPORTED)):
        m_ = mb.make_mlp_desc(n, d, dff, dt)
        assert mb.moa_gated_mlp_fwd(m_, *([a] * 8), check=False) == want, (n, d, dff, dt)
        assert mb.moa_gated_mlp_workspace_bytes(m_) == 0


def test_strided_layout_descriptor_checks(lib):
    """MOA_LAYOUT_STRIDED: strides are checked before anything touches a device."""
    good = ((384, 128, 384 * 300), (256, 128, 256 * 300), (384, 128, 384 * 300))
    d = mb.make_desc(1, 3, 300, 128, True, 0.1, layout=mb.MOA_LAYOUT_STRIDED, strides=good)
    assert mb.moa_attn_workspace_bytes(d, mb.MOA_OP_FUSED) > 0
    a = 4096
    for bad in (((100, 128, 115200),) * 3,            # row stride shorter than a row
                ((132, 128, 115200),) * 3,            # not a multiple of 8 elements (16 bytes)
                ((384, 0, 115200),) * 3):             # zero head stride
        d = mb.make_desc(1, 3, 300, 128, True, 0.1, layout=mb.MOA_LAYOUT_STRIDED, strides=bad)
        assert mb.moa_attn_workspace_bytes(d, mb.MOA_OP_FUSED) == 0
        assert mb.moa_attn_fwd(d, a, a, a, a, a, check=False) == mb.MOA_ERR_INVALID_ARG
    # the CUDA-core path has no strided form
    d = mb.make_desc(1, 3, 300, 128, True, 0.1, mb.MOA_F32, layout=mb.MOA_LAYOUT_STRIDED, strides=good)
    assert mb.moa_attn_fwd(d, a, a, a, a, a, check=False) == mb.MOA_ERR_UNSUPPORTED
