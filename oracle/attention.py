"""ctypes binding of the plain-C fp64 oracle (attn_oracle.c).

TEST INFRASTRUCTURE ONLY (see the package docstring).  Everything here is
argument marshalling: the arithmetic lives in attn_oracle.c, which states the
definition it follows (softmax attention with explicit n x n arrays S/P and dS,
the arrays the paper calls A and GS, and the analytic softmax backward).

Inputs are numpy float64 arrays shaped [B, H, n, d] (or [n, d] for the one-head
calls).  bf16 / fp32 test inputs are widened to float64 exactly before they get
here, so input quantisation is never counted as error.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_lib = None


def _cpu_tag() -> str:
    """Short tag of this host's CPU feature flags: the library is compiled with
    -march=native, so a copy built on another machine must not be reused."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as f:
        src = f.read()
    return hashlib.sha1(flags.encode() + src).hexdigest()[:12]


def _so_path() -> str:
    return os.path.join(_HERE, f"_attn_oracle_{_cpu_tag()}.so")


def build(force: bool = False) -> str:
    """Compile attn_oracle.c with gcc (-O3 -march=native -fopenmp) if needed."""
    so = _so_path()
    if force or not os.path.exists(so):
        tmp = so + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, so)
    return so


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        ci, cd = ctypes.c_int, ctypes.c_double
        lib.moa_oracle_num_threads.restype = ci
        lib.moa_oracle_attn.restype = ci
        lib.moa_oracle_attn.argtypes = [ci, ci, ci, ci, ci, cd] + [dp] * 9
        lib.moa_oracle_attn_head.restype = None
        lib.moa_oracle_attn_head.argtypes = [ci, ci, ci, cd] + [dp] * 12
        lib.moa_oracle_attn_rows.restype = ci
        lib.moa_oracle_attn_rows.argtypes = [ci, ci, ci, cd] + [dp] * 4 + [ci, ip] + [dp] * 3
        lib.moa_oracle_attn_cols.restype = ci
        lib.moa_oracle_attn_cols.argtypes = [ci, ci, ci, cd] + [dp] * 4 + [ci, ip] + [dp] * 2
        _lib = lib
    return _lib


def num_threads() -> int:
    """OpenMP threads the oracle will use (OMP_NUM_THREADS or the core count)."""
    return int(_load().moa_oracle_num_threads())


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def attn_fwd_bwd(Q, K, V, dO, causal: bool, scale: float):
    """All heads.  Returns dict with O, L, dQ, dK, dV (float64; L is [B,H,n])."""
    Q, K, V, dO = map(_f64, (Q, K, V, dO))
    if Q.ndim != 4 or not (Q.shape == K.shape == V.shape == dO.shape):
        raise ValueError("expected four [B,H,n,d] arrays of one shape")
    B, H, n, d = Q.shape
    O = np.empty_like(Q); dQ = np.empty_like(Q); dK = np.empty_like(Q); dV = np.empty_like(Q)
    L = np.empty((B, H, n), dtype=np.float64)
    if B * H * n * d == 0:
        return dict(O=O, L=L, dQ=dQ, dK=dK, dV=dV)
    rc = _load().moa_oracle_attn(B, H, n, d, int(bool(causal)), float(scale),
                                 _p(Q), _p(K), _p(V), _p(dO),
                                 _p(O), _p(L), _p(dQ), _p(dK), _p(dV))
    if rc != 0:
        raise MemoryError("oracle could not allocate its n x n arrays")
    return dict(O=O, L=L, dQ=dQ, dK=dK, dV=dV)


def attn_fwd_bwd_gqa(Q, K, V, dO, causal: bool, scale: float):
    """Grouped-query attention written out from its definition: Q, dO are [B,H,n,d] and K, V are
    [B,H_kv,n,d] with H_kv dividing H; query head h attends to K/V head h // (H/H_kv).  Every query
    head is an ordinary attention head over a copy of its K/V head, and a shared K/V head's gradient
    is the sum of the gradients of its copies (the head sharing the paper's decode section treats).
    Returns O, L, dQ as [B,H,...] and dK, dV as [B,H_kv,n,d]."""
    Q, K, V, dO = map(_f64, (Q, K, V, dO))
    B, H, n, d = Q.shape
    Hkv = K.shape[1]
    if K.shape != (B, Hkv, n, d) or V.shape != K.shape or dO.shape != Q.shape or Hkv < 1 or H % Hkv:
        raise ValueError("expected Q, dO [B,H,n,d] and K, V [B,H_kv,n,d] with H_kv dividing H")
    G = H // Hkv
    r = attn_fwd_bwd(Q, np.repeat(K, G, axis=1), np.repeat(V, G, axis=1), dO, causal, scale)
    r["dK"] = r["dK"].reshape(B, Hkv, G, n, d).sum(axis=2)
    r["dV"] = r["dV"].reshape(B, Hkv, G, n, d).sum(axis=2)
    return r


def attn_head_full(Q, K, V, dO, causal: bool, scale: float):
    """One head ([n,d] inputs); additionally returns the n x n arrays P and dS
    and the row vector D, for the invariants the tests check."""
    Q, K, V, dO = map(_f64, (Q, K, V, dO))
    n, d = Q.shape
    O = np.empty_like(Q); dQ = np.empty_like(Q); dK = np.empty_like(Q); dV = np.empty_like(Q)
    L = np.empty(n); D = np.empty(n)
    P = np.empty((n, n)); dS = np.empty((n, n))
    _load().moa_oracle_attn_head(n, d, int(bool(causal)), float(scale),
                                 _p(Q), _p(K), _p(V), _p(dO),
                                 _p(O), _p(L), _p(dQ), _p(dK), _p(dV), _p(P), _p(dS), _p(D))
    return dict(O=O, L=L, dQ=dQ, dK=dK, dV=dV, P=P, dS=dS, D=D)


def attn_rows(Q, K, V, dO, causal: bool, scale: float, rows):
    """Sampled query rows of one head: O[rows], L[rows], dQ[rows]."""
    Q, K, V, dO = map(_f64, (Q, K, V, dO))
    n, d = Q.shape
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    if rows.size and (rows.min() < 0 or rows.max() >= n):
        raise IndexError("row out of range")
    O = np.empty((rows.size, d)); dQ = np.empty((rows.size, d)); L = np.empty(rows.size)
    rc = _load().moa_oracle_attn_rows(n, d, int(bool(causal)), float(scale),
                                      _p(Q), _p(K), _p(V), _p(dO), rows.size,
                                      rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                      _p(O), _p(L), _p(dQ))
    if rc != 0:
        raise MemoryError("oracle row scratch")
    return dict(O=O, L=L, dQ=dQ)


def attn_cols(Q, K, V, dO, causal: bool, scale: float, cols):
    """Sampled key columns of one head: dK[cols], dV[cols]."""
    Q, K, V, dO = map(_f64, (Q, K, V, dO))
    n, d = Q.shape
    cols = np.ascontiguousarray(cols, dtype=np.int32)
    if cols.size and (cols.min() < 0 or cols.max() >= n):
        raise IndexError("column out of range")
    dK = np.empty((cols.size, d)); dV = np.empty((cols.size, d))
    rc = _load().moa_oracle_attn_cols(n, d, int(bool(causal)), float(scale),
                                      _p(Q), _p(K), _p(V), _p(dO), cols.size,
                                      cols.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                      _p(dK), _p(dV))
    if rc != 0:
        raise MemoryError("oracle column scratch")
    return dict(dK=dK, dV=dV)
