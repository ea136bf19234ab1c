"""bench.py's own multi-rank bookkeeping, run as real ranks on CPU (gloo): process group, shard plan, barriers,
max-over-ranks timing, whole-job value and the JSON line.  The library call is replaced at the call site by a sleep
proportional to the rank's model flops (--stub-ms-per-tflop), so no GPU is needed and the arithmetic can be checked."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(world, extra):
    port = _free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(world), "--steps", "3",
                                       "--warmup", "3", "--dist-backend", "gloo", "--stub-ms-per-tflop", "4"] + extra,
                                      cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-800:]
    lines = [l for l in outs[0][0].splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 prints one line
    for o, _ in outs[1:]:
        assert not [l for l in o.splitlines() if l.startswith("{")]      # the others print none
    return json.loads(lines[0])


def test_plan_is_a_partition():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_33916_b200 import inputs as mi
    w = mi.CONFIGS["c4_long"]
    for world in (1, 2, 3, 8, 16):
        plans = [bench.rank_plan(w, world, r, "heads") for r in range(world)]
        assert sum(p["heads"] for p in plans) == w.B * w.H
        assert [p["first_head"] for p in plans] == [sum(q["heads"] for q in plans[:i]) for i in range(world)]
        assert abs(sum(p["flops"] for p in plans) - w.model_flops) <= 1e-6 * w.model_flops
    assert [bench.rank_plan(w, 8, r, "heads")["heads"] for r in range(8)] == [2] * 8        # config 4: 2 heads per GPU on 8
    # shared K/V heads: whole groups stay on one rank
    p = bench.rank_plan(w, 4, 1, "heads", hkv=4)
    assert (p["H"], p["H_kv"], p["first_head"]) == (4, 1, 4)
    # replicas: everybody runs everything
    assert all(bench.rank_plan(w, 4, r, "replicas")["heads"] == 16 for r in range(4))


def test_two_ranks_partition_the_heads():
    j = _launch(2, ["--workload", "c4_long", "--shard", "heads"])
    assert j["n_gpus"] == 2 and j["scaling"] == "strong" and j["stub"] is True
    assert j["shards"]["heads_per_rank"] == [8, 8]
    # 7.697 TFLOP per step in all; each rank sleeps 4 ms per TFLOP of its half: about 15.4 ms per step
    total_tflop = 14 * 16 * 16384.0 ** 2 * 128 / 1e12
    assert 0.5 * total_tflop * 4 <= j["ms_per_step"] <= 0.5 * total_tflop * 4 * 1.5
    assert j["value"] == pytest.approx(total_tflop / (j["ms_per_step"] * 1e-3), rel=1e-9)
    assert "16 heads partitioned over 2 ranks" in j["config"]["parallelism"]


def test_three_ranks_uneven_partition_and_slowest_rank_sets_the_time():
    j = _launch(3, ["--workload", "c4_long", "--shard", "heads"])
    assert j["shards"]["heads_per_rank"] == [6, 5, 5]
    per_head_tflop = 14 * 16384.0 ** 2 * 128 / 1e12
    assert j["ms_per_step"] >= 6 * per_head_tflop * 4           # the rank with six heads
    assert j["value"] == pytest.approx(16 * per_head_tflop / (j["ms_per_step"] * 1e-3), rel=1e-9)


def test_two_ranks_as_replicas_is_weak_scaling():
    j = _launch(2, ["--workload", "c3_causal_mid"])
    assert j["scaling"] == "weak" and j["shards"]["heads_per_rank"] == [32, 32]
    total_tflop = 0.5 * 14 * 32 * 4096.0 ** 2 * 128 / 1e12
    assert j["value"] == pytest.approx(2 * total_tflop / (j["ms_per_step"] * 1e-3), rel=1e-9)
