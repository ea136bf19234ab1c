"""Seeded synthetic inputs and dtype conversions shared by the tests, the
benchmark and the smoke check.

This module holds none of the attention arithmetic: it draws numbers, rounds
them to the storage type and widens them again.  Both the CPU oracle and the
CUDA library are fed from the arrays made here, so the two sides see identical
bits.

Recipe (the paper's own workloads are synthetic sweeps over n with fixed B and
D, Sec. 3): Q, K, V, dO are i.i.d. N(0,1), drawn in that order from
numpy.random.default_rng(seed).standard_normal in float32, memory order
[B,H,n,d]; for the bf16 configurations each value is rounded to bfloat16 with
round-to-nearest-even.  scale = 1/sqrt(d), so scores are ~N(0,1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    n: int
    d: int
    causal: bool
    dtype: str  # "bf16" or "f32"
    seed: int

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def model_flops(self) -> float:
        """4 n^2 d forward + 10 n^2 d backward per head, halved when causal."""
        f = 14.0 * self.B * self.H * float(self.n) ** 2 * self.d
        return f * (0.5 if self.causal else 1.0)


#: The five configurations of the benchmark contract.
CONFIGS = {
    "c1_tiny_f32": Workload("c1_tiny_f32", 1, 1, 128, 64, False, "f32", 0),
    "c2_small_bf16": Workload("c2_small_bf16", 4, 8, 1024, 64, False, "bf16", 1),
    "c3_causal_mid": Workload("c3_causal_mid", 2, 16, 4096, 128, True, "bf16", 2),
    "c4_long": Workload("c4_long", 1, 16, 16384, 128, False, "bf16", 3),
}
# a small non-causal case for profiler captures: larger than L2 in total, short kernels
# the shape of the paper's own GPU tables (B = 2, no heads, D = 64), for the atomic-site comparison
CONFIGS["paper_b2_n2048_d64"] = Workload("paper_b2_n2048_d64", 2, 1, 2048, 64, False, "bf16", 6)
CONFIGS["paper_b2_n8192_d64"] = Workload("paper_b2_n8192_d64", 2, 1, 8192, 64, False, "bf16", 7)
CONFIGS["prof_h8_n8192"] = Workload("prof_h8_n8192", 1, 8, 8192, 128, False, "bf16", 5)
CONFIGS["prof_d64_h32_n8192"] = Workload("prof_d64_h32_n8192", 1, 32, 8192, 64, False, "bf16", 11)     # the same at 64 columns
# head dimensions above 128 (the two-pass kernels): the profiler case's shape at d = 256 and 192, and a causal one
CONFIGS["d256_h8_n8192"] = Workload("d256_h8_n8192", 1, 8, 8192, 256, False, "bf16", 8)
CONFIGS["d192_h8_n8192"] = Workload("d192_h8_n8192", 1, 8, 8192, 192, False, "bf16", 9)
CONFIGS["d256_h16_n4096_causal"] = Workload("d256_h16_n4096_causal", 2, 16, 4096, 256, True, "bf16", 10)
C5_SIZES = (512, 1024, 2048, 4096, 8192, 16384, 32768)
for _n in C5_SIZES:
    CONFIGS[f"c5_causal_n{_n}"] = Workload(f"c5_causal_n{_n}", 1, 32, _n, 128, True, "bf16", 4)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even.
    Inputs here are finite, so NaN handling is not needed."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f64(a: np.ndarray, dtype: str) -> np.ndarray:
    """Widen a stored tensor (bf16 bit patterns or float32) to float64, exactly."""
    if dtype == "bf16":
        return bf16_bits_to_f32(a).astype(np.float64)
    return np.asarray(a, dtype=np.float32).astype(np.float64)


def make_inputs(B: int, H: int, n: int, d: int, seed: int, dtype: str = "bf16",
                gain: float = 1.0) -> dict:
    """Q, K, V, dO as stored arrays: uint16 bf16 bit patterns or float32,
    each [B,H,n,d].  `gain` multiplies Q before rounding (used by the
    large-score test that exercises the softmax max-subtraction)."""
    rng = np.random.default_rng(seed)
    out = {}
    for name in ("Q", "K", "V", "dO"):
        x = rng.standard_normal((B, H, n, d), dtype=np.float32)
        if name == "Q" and gain != 1.0:
            x *= np.float32(gain)
        out[name] = f32_to_bf16_bits(x) if dtype == "bf16" else x
    return out


def make_workload_inputs(w: Workload) -> dict:
    return make_inputs(w.B, w.H, w.n, w.d, w.seed, w.dtype)


def make_norm_inputs(n: int, d: int, seed: int) -> dict:
    """RMSNorm inputs as bf16 bit patterns: x, dy [n,d] ~ N(0,1) and a gain g [d] ~ 1 + 0.25 N(0,1)."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, d), dtype=np.float32)
    g = (1.0 + 0.25 * rng.standard_normal(d)).astype(np.float32)
    dy = rng.standard_normal((n, d), dtype=np.float32)
    return {k: f32_to_bf16_bits(v) for k, v in dict(x=x, g=g, dy=dy).items()}


def make_mlp_inputs(n: int, d: int, d_ff: int, seed: int) -> dict:
    """Gated-MLP inputs as bf16 bit patterns: x, dy [n,d] ~ N(0,1); W1, W3 [d_ff,d] ~ N(0,1/d) and
    W2 [d,d_ff] ~ N(0,1/d_ff) (so that the pre-activations and y have unit scale)."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, d), dtype=np.float32)
    W1 = rng.standard_normal((d_ff, d), dtype=np.float32) / np.float32(np.sqrt(d))
    W3 = rng.standard_normal((d_ff, d), dtype=np.float32) / np.float32(np.sqrt(d))
    W2 = rng.standard_normal((d, d_ff), dtype=np.float32) / np.float32(np.sqrt(d_ff))
    dy = rng.standard_normal((n, d), dtype=np.float32)
    return {k: f32_to_bf16_bits(v) for k, v in dict(x=x, W1=W1, W3=W3, W2=W2, dy=dy).items()}


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """The parity metric: max|got - ref| / max|ref| over a whole tensor."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    den = float(np.max(np.abs(ref))) if ref.size else 0.0
    if ref.size == 0:
        return 0.0
    num = float(np.max(np.abs(got - ref)))
    if not np.isfinite(num):
        return float("inf")
    return num / den if den > 0 else num
