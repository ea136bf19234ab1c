"""Seeded random sweep of shapes and options through the C ABI against the fp64 oracle:
sizes around tile boundaries (128, 256), both head dims, causal or not, every dQ strategy,
both contraction paths and the materialising variant."""
import math

import numpy as np
import pytest

import oracle
from paper_2609_33916_b200 import inputs as mi

pytestmark = pytest.mark.gpu


def _cases(count, seed):
    rng = np.random.default_rng(seed)
    edge = [1, 2, 63, 64, 65, 127, 128, 129, 191, 255, 256, 257, 383, 384, 385, 511, 512, 513, 640]
    out = []
    for i in range(count):
        n = int(rng.choice(edge)) if rng.random() < 0.7 else int(rng.integers(1, 700))
        d = int(rng.choice([64, 128]))
        causal = bool(rng.integers(0, 2))
        B, Hh = int(rng.integers(1, 3)), int(rng.integers(1, 4))
        kind = rng.integers(0, 10)
        if kind < 6:        # tensor-core path, one of the dQ strategies
            path, mat = 2, 0
            dq = int(rng.choice([1, 2, 3]))
        elif kind < 8:      # SIMT path
            path, mat, dq = 1, 0, int(rng.choice([1, 3]))
        else:               # materialising variant
            path, mat, dq = 0, 1, 0
        out.append((i, B, Hh, n, d, causal, dq, path, mat))
    return out


@pytest.mark.parametrize("case", _cases(48, 20261125), ids=lambda c: f"{c[0]}-n{c[3]}-d{c[4]}-c{int(c[5])}-dq{c[6]}-p{c[7]}-m{c[8]}")
def test_random_case(case):
    import gpu_harness as H
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    i, B, Hh, n, d, causal, dq, path, mat = case
    scale = float(np.random.default_rng(i).uniform(0.5, 1.5)) / math.sqrt(d)
    inp = mi.make_inputs(B, Hh, n, d, seed=9000 + i, dtype="bf16")
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.attn_fwd_bwd(f["Q"], f["K"], f["V"], f["dO"], causal, scale)
    got = H.run_library(inp, "bf16", causal, scale, dq_mode=dq, path=path, materialize=mat)
    H.assert_close(got, ref, H.TOL_BF16, tag=str(case))
    assert mi.rel_err(got["L"], ref["L"]) <= 1e-3


def _gqa_cases(count, seed):
    """Tensor-core path only: random shared-K/V-head groupings and both memory layouts."""
    rng = np.random.default_rng(seed)
    edge = [1, 64, 127, 128, 129, 255, 256, 257, 384, 385, 513, 640]
    out = []
    for i in range(count):
        n = int(rng.choice(edge)) if rng.random() < 0.7 else int(rng.integers(1, 700))
        d = int(rng.choice([64, 128, 64, 128, 96, 80, 32, 112]))     # the others run with zero-filled columns
        causal = bool(rng.integers(0, 2))
        Hkv = int(rng.integers(1, 4))
        G = int(rng.choice([1, 2, 3, 5]))
        B = int(rng.integers(1, 3))
        dq = int(rng.choice([0, 1, 2, 3]))
        layout = int(rng.integers(0, 2))
        op = "split" if rng.random() < 0.3 else "fused"
        out.append((i, B, Hkv * G, Hkv, n, d, causal, dq, layout, op))
    return out


@pytest.mark.parametrize("case", _gqa_cases(40, 20261126),
                         ids=lambda c: f"{c[0]}-H{c[2]}kv{c[3]}-n{c[4]}-d{c[5]}-c{int(c[6])}-dq{c[7]}-l{c[8]}-{c[9]}")
def test_random_grouped_heads_and_layouts(case):
    import gpu_harness as H
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    i, B, Hq, Hkv, n, d, causal, dq, layout, op = case
    scale = float(np.random.default_rng(100 + i).uniform(0.5, 1.5)) / math.sqrt(d)
    q = mi.make_inputs(B, Hq, n, d, seed=9500 + i, dtype="bf16")
    kv = mi.make_inputs(B, Hkv, n, d, seed=9700 + i, dtype="bf16")
    inp = {"Q": q["Q"], "dO": q["dO"], "K": kv["K"], "V": kv["V"]}
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.attn_fwd_bwd_gqa(f["Q"], f["K"], f["V"], f["dO"], causal, scale)
    got = H.run_library(inp, "bf16", causal, scale, dq_mode=dq, layout=layout, op=op)
    H.assert_close(got, ref, H.TOL_BF16, tag=str(case))
    assert mi.rel_err(got["L"], ref["L"]) <= 1e-3
