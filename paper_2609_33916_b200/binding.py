"""ctypes binding of libmoa_attn.so: the same entry points as include/moa_attn.h.

Argument marshalling only -- every step of the attention path runs in the
library's CUDA kernels.  Tensor arguments may be torch CUDA tensors (their
data_ptr() is passed) or plain integer device addresses.  There is no CPU or
PyTorch fallback: if the library cannot be loaded, `lib()` raises.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libmoa_attn.so")

MOA_OK, MOA_ERR_INVALID_ARG, MOA_ERR_UNSUPPORTED, MOA_ERR_WORKSPACE, MOA_ERR_ARCH, MOA_ERR_CUDA, MOA_ERR_TIMEOUT = range(7)
MOA_ERR_SCRATCH_LIMIT = 7
MOA_STATIC_SCRATCH_BYTES = 16 << 20
MOA_BF16, MOA_F32 = 0, 1
MOA_DQ_AUTO, MOA_DQ_RED, MOA_DQ_BULK_REDUCE, MOA_DQ_SEPARATE_PASS = 0, 1, 2, 3
MOA_PATH_AUTO, MOA_PATH_SIMT, MOA_PATH_TC = 0, 1, 2
MOA_LAYOUT_BHND, MOA_LAYOUT_BNHD, MOA_LAYOUT_STRIDED = 0, 1, 2
MOA_OP_FWD, MOA_OP_BWD, MOA_OP_FUSED, MOA_OP_ROWPARALLEL = 0, 1, 2, 3

#: every symbol include/moa_attn.h declares
EXPORTS = (
    "moa_attn_workspace_bytes", "moa_attn_fwd", "moa_attn_bwd", "moa_attn_fused_fwd_bwd",
    "moa_last_device_status", "moa_launch_count", "moa_status_string", "moa_version",
    "moa_profile_enable", "moa_profile_read", "moa_attn_bwd_static_scratch", "moa_attn_fused_rowparallel",
    "moa_decode_workspace_bytes", "moa_decode_attn",
    "moa_rmsnorm_workspace_bytes", "moa_rmsnorm_fwd", "moa_rmsnorm_bwd",
    "moa_gated_mlp_fwd", "moa_gated_mlp_workspace_bytes", "moa_gated_mlp_bwd", "moa_gemm",
    "moa_selftest_expired_wait", "moa_bwd_pair_mode",
)


class moa_attn_desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("n", ctypes.c_int32), ("d", ctypes.c_int32),
                ("causal", ctypes.c_int32), ("scale", ctypes.c_float), ("dtype", ctypes.c_int32),
                ("dq_mode", ctypes.c_int32), ("materialize", ctypes.c_int32), ("path", ctypes.c_int32),
                ("H_kv", ctypes.c_int32), ("layout", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("q_stride", ctypes.c_int64 * 3), ("kv_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3)]


class moa_decode_desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("H_kv", ctypes.c_int32), ("n", ctypes.c_int32),
                ("d", ctypes.c_int32), ("scale", ctypes.c_float), ("dtype", ctypes.c_int32)]


class moa_rmsnorm_desc(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("d", ctypes.c_int32), ("eps", ctypes.c_float), ("dtype", ctypes.c_int32)]


class moa_gemm_desc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int32), ("N", ctypes.c_int32), ("K", ctypes.c_int32), ("a_layout", ctypes.c_int32),
                ("b_layout", ctypes.c_int32), ("dtype", ctypes.c_int32)]


class moa_mlp_desc(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("d", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("dtype", ctypes.c_int32)]


MOA_KERNEL_KINDS = 6
KERNEL_KIND_NAMES = ("fwd", "preprocess", "bwd_kv", "bwd_dq", "convert", "other")


class moa_profile(ctypes.Structure):
    _fields_ = [("ms", ctypes.c_float * MOA_KERNEL_KINDS), ("launches", ctypes.c_uint32 * MOA_KERNEL_KINDS)]


class MoaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (moa_status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libmoa_attn.so (built in-tree by paper_2609_33916_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_33916_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, dp = ctypes.c_void_p, ctypes.c_size_t, ctypes.POINTER(moa_attn_desc)
        L.moa_attn_workspace_bytes.restype = sz
        L.moa_attn_workspace_bytes.argtypes = [dp, ctypes.c_int]
        L.moa_attn_fwd.restype = ctypes.c_int
        L.moa_attn_fwd.argtypes = [dp] + [vp] * 5 + [vp, sz, vp]
        L.moa_attn_bwd.restype = ctypes.c_int
        L.moa_attn_bwd.argtypes = [dp] + [vp] * 9 + [vp, sz, vp]
        L.moa_attn_bwd_static_scratch.restype = ctypes.c_int
        L.moa_attn_bwd_static_scratch.argtypes = [dp] + [vp] * 9 + [vp]
        L.moa_attn_fused_fwd_bwd.restype = ctypes.c_int
        L.moa_attn_fused_fwd_bwd.argtypes = [dp] + [vp] * 9 + [vp, sz, vp]
        L.moa_attn_fused_rowparallel.restype = ctypes.c_int
        L.moa_attn_fused_rowparallel.argtypes = [dp] + [vp] * 9 + [ctypes.c_int, vp, sz, vp]
        L.moa_decode_workspace_bytes.restype = sz
        L.moa_decode_workspace_bytes.argtypes = [ctypes.POINTER(moa_decode_desc)]
        L.moa_decode_attn.restype = ctypes.c_int
        L.moa_decode_attn.argtypes = [ctypes.POINTER(moa_decode_desc)] + [vp] * 5 + [vp, sz, vp]
        rp = ctypes.POINTER(moa_rmsnorm_desc)
        L.moa_rmsnorm_workspace_bytes.restype = sz
        L.moa_rmsnorm_workspace_bytes.argtypes = [rp]
        L.moa_rmsnorm_fwd.restype = ctypes.c_int
        L.moa_rmsnorm_fwd.argtypes = [rp] + [vp] * 4 + [vp]
        L.moa_rmsnorm_bwd.restype = ctypes.c_int
        L.moa_rmsnorm_bwd.argtypes = [rp] + [vp] * 7 + [vp, sz, vp]
        mp = ctypes.POINTER(moa_mlp_desc)
        L.moa_gated_mlp_workspace_bytes.restype = sz
        L.moa_gated_mlp_workspace_bytes.argtypes = [mp]
        L.moa_gated_mlp_fwd.restype = ctypes.c_int
        L.moa_gated_mlp_fwd.argtypes = [mp] + [vp] * 9 + [vp]
        L.moa_gemm.restype = ctypes.c_int
        L.moa_gemm.argtypes = [ctypes.POINTER(moa_gemm_desc)] + [vp] * 4 + [vp]
        L.moa_gated_mlp_bwd.restype = ctypes.c_int
        L.moa_gated_mlp_bwd.argtypes = [mp] + [vp] * 12 + [vp, sz, vp]
        L.moa_last_device_status.restype = ctypes.c_int
        L.moa_last_device_status.argtypes = [vp]
        L.moa_selftest_expired_wait.restype = ctypes.c_int
        L.moa_selftest_expired_wait.argtypes = [ctypes.c_longlong, vp]
        L.moa_bwd_pair_mode.restype = ctypes.c_int
        L.moa_bwd_pair_mode.argtypes = [ctypes.c_int]
        L.moa_launch_count.restype = ctypes.c_uint64
        L.moa_status_string.restype = ctypes.c_char_p
        L.moa_status_string.argtypes = [ctypes.c_int]
        L.moa_version.restype = ctypes.c_int
        L.moa_profile_enable.restype = ctypes.c_int
        L.moa_profile_enable.argtypes = [ctypes.c_int]
        L.moa_profile_read.restype = ctypes.c_int
        L.moa_profile_read.argtypes = [ctypes.POINTER(moa_profile)]
        _lib = L
    return _lib


def make_desc(B, H, n, d, causal, scale, dtype=MOA_BF16, dq_mode=MOA_DQ_AUTO, materialize=0,
              path=MOA_PATH_AUTO, H_kv=0, layout=0, strides=None) -> moa_attn_desc:
    """H_kv: key/value heads (0 or H: one per query head; a divisor of H: grouped-query attention).
    layout: MOA_LAYOUT_BHND (0), MOA_LAYOUT_BNHD (1: tensors are [B,n,H,d] in memory) or MOA_LAYOUT_STRIDED (2) with
    strides = (q, kv, o), each a (row, head, batch) triple in elements."""
    desc = moa_attn_desc(int(B), int(H), int(n), int(d), int(bool(causal)), float(scale), int(dtype),
                         int(dq_mode), int(materialize), int(path), int(H_kv), int(layout), 0)
    if strides is not None:
        for name, tri in zip(("q_stride", "kv_stride", "o_stride"), strides):
            setattr(desc, name, (ctypes.c_int64 * 3)(*[int(x) for x in tri]))
    return desc


def strides_of(t):
    """(row, head, batch) element strides of a torch tensor viewed as [B, H, n, d] (any permutation or slice of a
    larger buffer whose last dimension is contiguous)."""
    assert t.dim() == 4 and t.stride(3) == 1
    return (t.stride(2), t.stride(1), t.stride(0))


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return ctypes.c_void_p(x)
    return ctypes.c_void_p(x.data_ptr())   # torch tensor


def _nbytes(ws) -> int:
    if ws is None:
        return 0
    return ws.numel() * ws.element_size()


def _stream(stream):
    if stream is None:
        import torch
        if not torch.cuda.is_available():
            return ctypes.c_void_p(0)   # host-side checks only; any launch will report MOA_ERR_CUDA
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def status_string(status: int) -> str:
    return lib().moa_status_string(int(status)).decode()


def moa_version() -> int:
    return int(lib().moa_version())


def moa_launch_count() -> int:
    return int(lib().moa_launch_count())


def moa_attn_workspace_bytes(desc: moa_attn_desc, op: int) -> int:
    return int(lib().moa_attn_workspace_bytes(ctypes.byref(desc), int(op)))


def moa_attn_fwd(desc, Q, K, V, O, L, ws=None, stream=None, ws_bytes=None, check=True) -> int:
    s = lib().moa_attn_fwd(ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(L), _ptr(ws),
                           _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_attn_fwd")
    return s


def moa_attn_bwd(desc, Q, K, V, O, L, dO, dQ, dK, dV, ws=None, stream=None, ws_bytes=None, check=True) -> int:
    s = lib().moa_attn_bwd(ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(L), _ptr(dO),
                           _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws),
                           _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_attn_bwd")
    return s


def moa_attn_bwd_static_scratch(desc, Q, K, V, O, L, dO, dQ, dK, dV, stream=None, check=True) -> int:
    """moa_attn_bwd for callers that cannot allocate: no workspace argument, the library's
    built-in scratch array (MOA_STATIC_SCRATCH_BYTES) is used.  Calls sharing a device must
    not overlap on the GPU; make the first call on a device outside any stream capture."""
    s = lib().moa_attn_bwd_static_scratch(ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(L),
                                          _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV), _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_attn_bwd_static_scratch")
    return s


def moa_attn_fused_fwd_bwd(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws=None, stream=None, ws_bytes=None,
                           check=True) -> int:
    s = lib().moa_attn_fused_fwd_bwd(ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(O),
                                     _ptr(L), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws),
                                     _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_attn_fused_fwd_bwd")
    return s


def moa_attn_fused_rowparallel(desc, Q, K, V, dO, O, L, dQ, dK, dV, atomic_sites, ws=None, stream=None,
                               ws_bytes=None, check=True) -> int:
    s = lib().moa_attn_fused_rowparallel(ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(O),
                                         _ptr(L), _ptr(dQ), _ptr(dK), _ptr(dV), int(atomic_sites), _ptr(ws),
                                         _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_attn_fused_rowparallel")
    return s


def make_rmsnorm_desc(n, d, eps, dtype=MOA_BF16) -> moa_rmsnorm_desc:
    return moa_rmsnorm_desc(int(n), int(d), float(eps), int(dtype))


def moa_rmsnorm_workspace_bytes(desc) -> int:
    return int(lib().moa_rmsnorm_workspace_bytes(ctypes.byref(desc)))


def moa_rmsnorm_fwd(desc, x, g, y, r=None, stream=None, check=True) -> int:
    s = lib().moa_rmsnorm_fwd(ctypes.byref(desc), _ptr(x), _ptr(g), _ptr(y), _ptr(r), _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_rmsnorm_fwd")
    return s


def moa_rmsnorm_bwd(desc, x, g, r, dy, dx, dg, ws=None, stream=None, ws_bytes=None, check=True, dx_add=None) -> int:
    """dx_add (optional, [n,d]): added to dx (the gradient arriving along a residual connection)."""
    s = lib().moa_rmsnorm_bwd(ctypes.byref(desc), _ptr(x), _ptr(g), _ptr(r), _ptr(dy), _ptr(dx_add), _ptr(dx), _ptr(dg), _ptr(ws),
                              _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_rmsnorm_bwd")
    return s


def moa_bwd_pair_mode(mode: int = -1) -> int:
    """Sets (mode 0 or 1) or queries (mode < 0) whether the tensor-core backward runs on CTA pairs; returns the
    mode in force before the call."""
    return int(lib().moa_bwd_pair_mode(int(mode)))


def moa_selftest_expired_wait(limit_cycles=1000000, stream=None) -> int:
    """Enqueues one warp whose bounded wait expires after `limit_cycles`; moa_last_device_status then reports
    MOA_ERR_TIMEOUT once."""
    return int(lib().moa_selftest_expired_wait(int(limit_cycles), _stream(stream)))


def make_gemm_desc(M, N, K, a_layout=0, b_layout=0, dtype=MOA_BF16) -> moa_gemm_desc:
    """C[M,N] = A B^T (+ R); a_layout 0: A is [M,K], 1: A is [K,M]; b_layout 0: B is [N,K], 1: B is [K,N]."""
    return moa_gemm_desc(int(M), int(N), int(K), int(a_layout), int(b_layout), int(dtype))


def moa_gemm(desc, A, B, C, R=None, stream=None, check=True) -> int:
    s = lib().moa_gemm(ctypes.byref(desc), _ptr(A), _ptr(B), _ptr(R), _ptr(C), _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_gemm")
    return s


def make_mlp_desc(n, d, d_ff, dtype=MOA_BF16) -> moa_mlp_desc:
    return moa_mlp_desc(int(n), int(d), int(d_ff), int(dtype))


def moa_gated_mlp_workspace_bytes(desc) -> int:
    return int(lib().moa_gated_mlp_workspace_bytes(ctypes.byref(desc)))


def moa_gated_mlp_fwd(desc, x, W1, W3, W2, a, u, h, y, stream=None, check=True, res=None) -> int:
    """res (optional, [n,d]): added to y (the block's residual connection)."""
    s = lib().moa_gated_mlp_fwd(ctypes.byref(desc), _ptr(x), _ptr(W1), _ptr(W3), _ptr(W2), _ptr(res), _ptr(a), _ptr(u), _ptr(h),
                                _ptr(y), _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_gated_mlp_fwd")
    return s


def moa_gated_mlp_bwd(desc, x, W1, W3, W2, a, u, h, dy, dx, dW1, dW3, dW2, ws=None, stream=None, ws_bytes=None,
                      check=True) -> int:
    s = lib().moa_gated_mlp_bwd(ctypes.byref(desc), _ptr(x), _ptr(W1), _ptr(W3), _ptr(W2), _ptr(a), _ptr(u), _ptr(h),
                                _ptr(dy), _ptr(dx), _ptr(dW1), _ptr(dW3), _ptr(dW2), _ptr(ws),
                                _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_gated_mlp_bwd")
    return s


def make_decode_desc(B, H, n, d, scale, dtype=MOA_BF16, H_kv=0) -> moa_decode_desc:
    return moa_decode_desc(int(B), int(H), int(H_kv), int(n), int(d), float(scale), int(dtype))


def moa_decode_workspace_bytes(desc: moa_decode_desc) -> int:
    return int(lib().moa_decode_workspace_bytes(ctypes.byref(desc)))


def moa_decode_attn(desc, q, K, V, out, lse=None, ws=None, stream=None, ws_bytes=None, check=True) -> int:
    s = lib().moa_decode_attn(ctypes.byref(desc), _ptr(q), _ptr(K), _ptr(V), _ptr(out), _ptr(lse), _ptr(ws),
                              _nbytes(ws) if ws_bytes is None else ws_bytes, _stream(stream))
    if check and s != MOA_OK:
        raise MoaError(s, "moa_decode_attn")
    return s


def moa_last_device_status(stream=None) -> int:
    return int(lib().moa_last_device_status(_stream(stream)))


def moa_profile_enable(on: bool) -> int:
    return int(lib().moa_profile_enable(int(bool(on))))


def moa_profile_read() -> dict:
    """{kind name: (total ms, launches)} since the last read."""
    p = moa_profile()
    s = lib().moa_profile_read(ctypes.byref(p))
    if s != MOA_OK:
        raise MoaError(s, "moa_profile_read")
    return {KERNEL_KIND_NAMES[k]: (float(p.ms[k]), int(p.launches[k])) for k in range(MOA_KERNEL_KINDS)}
