"""fp64 oracle of decode attention: one new query per head over a cache of n keys and values.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Plain numpy, the definition written out:
for every batch element b and query head h, with the K/V head kv = h // (H / H_kv) that head reads,

    s_j = scale * sum_k q[b,h,k] * K[b,kv,j,k]        j = 0 .. n-1   (the whole cache is visible)
    p   = softmax(s)
    o[b,h,:] = sum_j p_j * V[b,kv,j,:]

(the paper's decode section: a single query over the KV cache, O(n) work per token, with the
grouped-query / multi-query head sharing its companion derivation treats).  Also returns the
logsumexp of s, which a caller needs to merge results over cache segments.
"""
from __future__ import annotations

import numpy as np


def decode_attn(q, K, V, scale: float):
    """q [B,H,d]; K, V [B,H_kv,n,d] with H_kv dividing H.  Returns dict(o [B,H,d], lse [B,H]), float64."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    B, H, d = q.shape
    Hkv, n = K.shape[1], K.shape[2]
    if K.shape != (B, Hkv, n, d) or V.shape != K.shape or Hkv < 1 or H % Hkv or n < 1:
        raise ValueError("expected q [B,H,d] and K, V [B,H_kv,n,d] with H_kv dividing H and n >= 1")
    G = H // Hkv
    o = np.empty((B, H, d))
    lse = np.empty((B, H))
    for b in range(B):
        for h in range(H):
            kv = h // G
            s = scale * (K[b, kv] @ q[b, h])          # [n]
            m = s.max()
            e = np.exp(s - m)
            l = e.sum()
            o[b, h] = (e / l) @ V[b, kv]
            lse[b, h] = m + np.log(l)
    return dict(o=o, lse=lse)
