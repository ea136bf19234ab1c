#!/usr/bin/env python
"""Benchmark of the fused attention forward+backward path.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--dq-mode M]
  python bench.py --impl reference ...      # times the fp64 CPU oracle instead

A step is one moa_attn_fused_fwd_bwd call (forward, preprocess, backward, dQ
conversion) over one batch of synthetic bf16 inputs.  The metric is model
TFLOP/s: 4 n^2 d forward + 10 n^2 d backward per head, halved when causal.
With N > 1 (launched by torch.distributed.run, one rank per GPU) there are two modes, neither with a
collective on the data path, because (batch, head) pairs are independent:
  --shard replicas (default)  every rank runs the whole workload on its own GPU; the value is the sum
                              over ranks divided by the slowest rank's time ("scaling": "weak")
  --shard heads               the workload's B*H heads are partitioned into contiguous blocks, one per
                              rank (config 4: 16 heads -> 2 per GPU on 8); total work is fixed
                              ("scaling": "strong")

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused attn fwd+bwd TFLOP/s and % of B200 dense BF16 tensor peak"
NOMINAL_BF16_TFLOPS = 2250.0   # datasheet dense bf16, for context
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def load_traffic_record(kernel: str):
    """The committed record of the last ncu DRAM-traffic capture of `kernel` (profiles/traffic.json, written by
    `python -m paper_2609_33916_b200.profile_summary`), or None."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            return json.load(f).get(kernel)
    except Exception:
        return None


# ------------------------------------------------------------------- clock sampling
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs
    (read-only queries)."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._stop.clear()
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
            self._thr = None

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------- CPU oracle legs
def time_oracle_sample(w, budget_s: float):
    """Times the oracle, as it stands, on a bounded sample of workload `w`: whole heads
    (forward + backward, all n^2 work of each) when one head fits the budget, otherwise
    sampled query rows of head (0,0).  Returns (tflops, seconds, cores, description)."""
    import numpy as np
    import oracle
    from paper_2609_33916_b200 import inputs as mi

    cores = oracle.num_threads()
    # calibrate on a small head
    nc = min(w.n, 1024)
    cal = mi.make_inputs(1, 1, nc, w.d, seed=99, dtype=w.dtype)
    f = {k: mi.to_f64(v, w.dtype) for k, v in cal.items()}
    t0 = time.perf_counter()
    oracle.attn_fwd_bwd(f["Q"], f["K"], f["V"], f["dO"], w.causal, w.scale)
    rate = 14.0 * nc * nc * w.d / max(time.perf_counter() - t0, 1e-6)     # flop/s, dense count
    head_flops_dense = 14.0 * float(w.n) ** 2 * w.d
    head_model = head_flops_dense * (0.5 if w.causal else 1.0)
    est_head = head_flops_dense / rate * 1.6          # large n runs slower per flop than the calibration
    mem_ok = 2.0 * w.n * w.n * 8 < 24e9
    inp = mi.make_inputs(1, 1, w.n, w.d, seed=w.seed, dtype=w.dtype)
    f = {k: mi.to_f64(v, w.dtype) for k, v in inp.items()}
    if est_head <= budget_s and mem_ok:
        heads = max(1, min(w.B * w.H, int(budget_s / est_head)))
        t0 = time.perf_counter()
        for _ in range(heads):
            oracle.attn_fwd_bwd(f["Q"], f["K"], f["V"], f["dO"], w.causal, w.scale)
        dt = time.perf_counter() - t0
        return heads * head_model / dt / 1e12, dt, cores, f"{heads} of {w.B * w.H} heads, full fwd+bwd"
    # row sample: S, P, O, dP, dS, dQ of r rows = 8 n d executed flops per row (4 n d
    # forward + 4 n d of the backward); credited as that share of the model count
    per_row = 8.0 * w.n * w.d
    r = int(max(8, min(w.n, budget_s * rate / 1.6 / per_row)))
    rows = np.linspace(0, w.n - 1, r).astype(np.int32)
    t0 = time.perf_counter()
    oracle.attn_rows(f["Q"][0, 0], f["K"][0, 0], f["V"][0, 0], f["dO"][0, 0], w.causal, w.scale, rows)
    dt = time.perf_counter() - t0
    credit = per_row * r * (0.5 if w.causal else 1.0)
    return credit / dt / 1e12, dt, cores, (f"{r} query rows of head (0,0): S,P,O,dP,dS,dQ only, "
                                             f"8nd flop per row credited")


def time_oracle_one_thread(w, budget_s: float):
    """The same sample with OMP_NUM_THREADS=1, in a child process (the thread count is read when the oracle's library
    is loaded).  The paper found that over-threading small n costs its CPU kernels up to 14.5x (Sec. 3, CPU scaling),
    so for the small configurations both counts are timed and the better one is named."""
    import subprocess
    code = ("import json, sys; sys.path.insert(0, %r); import bench; from paper_2609_33916_b200 import inputs as mi; "
            "v, dt, c, d = bench.time_oracle_sample(mi.CONFIGS[%r], %f); print(json.dumps(dict(value=v, seconds=dt, cores=c, sample=d)))"
            % (ROOT, w.name, budget_s))
    r = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, OMP_NUM_THREADS="1"), capture_output=True,
                       text=True, timeout=600)
    if r.returncode != 0:
        return None
    return json.loads(r.stdout.strip().splitlines()[-1])


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    if "LOCAL_RANK" in os.environ and os.environ.get("OMP_NUM_THREADS") == "1":
        # torch.distributed.run pins OMP_NUM_THREADS=1 for its workers; the oracle is meant to use
        # the host's cores as it does when run directly
        os.environ["OMP_NUM_THREADS"] = str(len(os.sched_getaffinity(0)))
    total_budget = 150.0
    per_step = total_budget / max(1, args.steps + args.warmup)
    vals, secs, cores, desc = [], [], 0, ""
    for i in range(args.warmup + args.steps):
        v, dt, cores, desc = time_oracle_sample(w, per_step)
        if i >= args.warmup:
            vals.append(v)
            secs.append(dt)
    value = sum(vals) / len(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def workload_config(w, args):
    return {"workload": w.name, "B": w.B, "H": w.H, "n": w.n, "d": w.d, "causal": w.causal,
            "scale": "1/sqrt(d)", "dq_mode": args.dq_mode, "path": args.path, "materialize": getattr(args, "materialize", 0),
            "l2": "inputs+outputs per step exceed the 126 MB L2; no explicit flush",
            "parallelism": (f"{w.B * w.H} heads partitioned over {args.gpus} ranks" if getattr(args, "shard", "replicas") == "heads" and args.gpus > 1
                            else f"independent replicas x{args.gpus}")}


def rank_plan(w, world: int, rank: int, shard: str, hkv: int = 0) -> dict:
    """What one rank computes.  replicas: the whole workload.  heads: a contiguous block of the flattened (batch, head)
    pairs -- heads are independent, so the block is handed to the library as B = 1, H = count (with shared K/V heads
    the unit is a K/V head with its group of query heads)."""
    from paper_2609_33916_b200 import sharding
    per_head = w.model_flops / (w.B * w.H)
    if shard == "replicas" or world == 1:
        return {"B": w.B, "H": w.H, "H_kv": hkv, "first_head": 0, "heads": w.B * w.H, "flops": w.model_flops}
    if shard != "heads":
        raise ValueError(f"unknown shard mode {shard}")
    group = (w.H // hkv) if hkv else 1
    units = w.B * w.H // group                   # K/V heads (or plain heads) to hand out
    first, count = sharding.head_shard(units, world, rank)
    return {"B": 1, "H": count * group, "H_kv": count if hkv else 0, "first_head": first * group, "heads": count * group,
            "flops": per_head * count * group}


def job_value(flops_per_rank: list, ms_slowest: float) -> float:
    """Whole-job TFLOP/s: the flops all ranks processed per step over the slowest rank's time per step."""
    from paper_2609_33916_b200 import sharding
    return sharding.aggregate_rate(flops_per_rank, [ms_slowest * 1e-3] * len(flops_per_rank)) / 1e12


def run_stub(args, w):
    """Testing aid (--stub-ms-per-tflop): the rank and shard bookkeeping of a multi-rank run -- process group, shard
    plan, barriers, max-over-ranks timing, whole-job value, the JSON line -- with the library call replaced by a
    sleep proportional to the rank's flops.  Needs no GPU; run with --dist-backend gloo."""
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch
        import torch.distributed as dist
        dist.init_process_group(args.dist_backend)
    plan = rank_plan(w, world, rank, args.shard, args.hkv)

    def barrier():
        if dist is not None:
            dist.barrier()

    def gather(x: float) -> list:
        if dist is None:
            return [x]
        import torch
        t = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(t, torch.tensor([x], dtype=torch.float64))
        return [float(v.item()) for v in t]

    def step():
        time.sleep(plan["flops"] / 1e12 * args.stub_ms_per_tflop * 1e-3)

    for _ in range(args.warmup):
        step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    ms_mine = (time.perf_counter() - t0) * 1e3 / args.steps
    barrier()
    ms_all, flops_all = gather(ms_mine), gather(plan["flops"])
    line = {"metric": METRIC, "value": job_value(flops_all, max(ms_all)), "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": max(ms_all), "higher_is_better": True,
            "scaling": "strong" if (args.shard == "heads" and world > 1) else "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": workload_config(w, args), "stub": True,
            "shards": {"heads_per_rank": [int(round(f / (w.model_flops / (w.B * w.H)))) for f in flops_all],
                       "first_head_rank": plan["first_head"]}}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


# ---------------------------------------------------------------------------- decode
DECODE_WORKLOADS = {
    # name: (B, H, H_kv, n, d, dtype)
    "decode_gqa_n32768": (8, 32, 8, 32768, 128, "bf16"),       # 1.07 GB of cache, groups of 4 query heads
    "decode_mha_n8192": (16, 32, 32, 8192, 128, "bf16"),       # 2.15 GB, one K/V head per query head
    "decode_paper_n1m": (1, 1, 1, 1048576, 64, "f32"),         # the paper's largest cache, its fp32, one head: 0.54 GB
}


def run_decode(args):
    """Decode attention (one query per head over a resident K/V cache): a second bench line, not the
    contract's default.  The path is HBM-bound, so the roofline entry is achieved GB/s of the
    algorithmic bytes (the cache, read once, plus q and out) against the measured copy bandwidth."""
    import numpy as np
    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    import oracle

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    B, H, Hkv, n, d, dtype = DECODE_WORKLOADS[args.decode]
    mbuild.build()
    mb.lib()
    peaks, peaks_kind = load_peaks()
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    gen = torch.Generator(device="cuda").manual_seed(11)
    q = torch.randn((B, H, d), generator=gen, device="cuda").to(tdt)
    K = torch.randn((B, Hkv, n, d), generator=gen, device="cuda").to(tdt)
    V = torch.randn((B, Hkv, n, d), generator=gen, device="cuda").to(tdt)
    out = torch.empty((B, H, d), dtype=tdt, device="cuda")
    lse = torch.empty((B, H), dtype=torch.float32, device="cuda")
    scale = 1.0 / math.sqrt(d)
    desc = mb.make_decode_desc(B, H, n, d, scale, mb.MOA_BF16 if dtype == "bf16" else mb.MOA_F32, H_kv=Hkv)
    ws = torch.empty(max(mb.moa_decode_workspace_bytes(desc), 16), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    esz = 2 if dtype == "bf16" else 4
    alg_bytes = 2.0 * B * Hkv * n * d * esz + 2.0 * B * H * d * esz + 4.0 * B * H

    def step():
        mb.moa_decode_attn(desc, q, K, V, out, lse, ws, stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    l0 = mb.moa_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    sampler.stop()
    launches = mb.moa_launch_count() - l0
    ms = e0.elapsed_time(e1) / args.steps
    gbs = alg_bytes / (ms * 1e-3) / 1e9
    # end to end: the cache stays on the device (it is the state of a running decode); the new
    # query comes from pinned host memory and the result goes back, every step
    hq = q.cpu().pin_memory()
    hout = torch.empty((B, H, d), dtype=tdt).pin_memory()
    t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0e.record(stream)
    for _ in range(args.steps):
        q.copy_(hq, non_blocking=True)
        step()
        hout.copy_(out, non_blocking=True)
    t1e.record(stream)
    torch.cuda.synchronize()
    e2e_ms = t0e.elapsed_time(t1e) / args.steps
    st = mb.moa_last_device_status(stream)
    if st != mb.MOA_OK:
        raise SystemExit(f"device status: {mb.status_string(st)}")
    line = {
        "metric": "decode attention: GB/s of K/V cache read (one query per head)", "value": gbs, "unit": "GB/s",
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
        "config": {"workload": args.decode, "B": B, "H": H, "H_kv": Hkv, "n": n, "d": d, "scale": "1/sqrt(d)",
                   "l2": "the cache of one step exceeds the 126 MB L2; no explicit flush"},
        "tokens_per_s": B / (ms * 1e-3),
        "clocks": sampler.summary(),
        "e2e": {"value": alg_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": B * H * d * esz,
                "d2h_bytes_per_step": B * H * d * esz, "ms_per_step": e2e_ms,
                "how": "cache resident on the device; the step's query comes from pinned host memory and its output goes back"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode_split_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                     "peak_source": f"{peaks_kind} hbm_gbs (copy bandwidth)",
                     "algorithmic_bytes_per_step": alg_bytes},
    }
    if not args.no_cpu_baseline:
        heads = min(B * H, 4)
        hb = min(B, max(1, heads // H)) if H <= heads else 1
        qs = q[:hb, :heads].float().cpu().numpy().astype(np.float64)
        ks = K[:hb, :max(1, heads * Hkv // H)].float().cpu().numpy().astype(np.float64)
        vs = V[:hb, :max(1, heads * Hkv // H)].float().cpu().numpy().astype(np.float64)
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 5.0:
            oracle.decode_attn(qs, ks, vs, scale)
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        sample_bytes = 2.0 * ks.shape[0] * ks.shape[1] * n * d * esz
        line["cpu_baseline"] = {"value": sample_bytes / dt / 1e9, "unit": "GB/s", "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"{qs.shape[0]}x{qs.shape[1]} query heads over {ks.shape[1]} K/V head(s), numpy fp64",
                                "seconds": dt * reps}
    print(json.dumps(line))
    return 0


BLOCK_WORKLOADS = {
    # name: (piece, n tokens, d, d_ff)
    "rmsnorm_n65536_d2048": ("rmsnorm", 65536, 2048, 0),           # the paper's longest RMSNorm sweep point, a model-sized row
    "rmsnorm_n65536_d4096": ("rmsnorm", 65536, 4096, 0),
    "mlp_n16384_d2048_ff8192": ("mlp", 16384, 2048, 8192),          # config 4's tokens, 16 heads x 128, d_ff = 4 d
    "mlp_n8192_d4096_ff16384": ("mlp", 8192, 4096, 16384),
    "mlp_n4096_d1024_ff4096": ("mlp", 4096, 1024, 4096),              # small case for profiler captures (0.4 GB moved per step)
    "mlp_paper_n512_d64_ff256": ("mlp", 512, 64, 256),              # the paper's own traffic-check size (B=2, N=256, D=64, DFF=256)
    # one product C[M,N] = A[M,K] B[N,K]^T through moa_gemm: (piece, M, K, N)
    "gemm_m8192_n8192_k8192": ("gemm", 8192, 8192, 8192),
    "gemm_m16384_n2048_k2048": ("gemm", 16384, 2048, 2048),            # one projection of the block at config 4's tokens
    "gemm_m8192_n2048_k2048": ("gemm", 8192, 2048, 2048),              # small case for profiler captures
    # the whole pre-norm block (two norms, QKV projection, attention, output projection, gated MLP, residuals),
    # composed from library calls: (piece, B, n, H, d, d_ff, causal)
    "block_c4_b1_n16384_h16_d128_ff8192": ("block", 1, 16384, 16, 128, 8192, False),   # config 4's attention inside a block
    "block_c3_b2_n4096_h16_d128_ff8192": ("block", 2, 4096, 16, 128, 8192, True),      # config 3's
    "block_small_b2_n1024_h8_d128_ff4096": ("block", 2, 1024, 8, 128, 4096, True),     # small case for profiler captures
    "block_paper_b2_n256_h1_d64_ff256": ("block", 2, 256, 1, 64, 256, False),          # the paper's traffic-check size
}


def run_block(args):
    """Block pieces (RMSNorm, gated MLP): one step = forward + backward of the piece.  Further bench
    lines, not the contract's default.  RMSNorm is HBM-bound (roofline: algorithmic bytes against
    the measured copy bandwidth), the gated MLP is a dense contraction (model FLOPs against the
    measured dense bf16 peak)."""
    import numpy as np
    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    import oracle

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    if BLOCK_WORKLOADS[args.block][0] == "block":
        return run_whole_block(args)
    piece, n, d, dff = BLOCK_WORKLOADS[args.block]
    mbuild.build()
    mb.lib()
    peaks, peaks_kind = load_peaks()
    bf = torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(17)
    stream = torch.cuda.current_stream()
    rnd = lambda *shape, s=1.0: (torch.randn(shape, generator=gen, device="cuda") * s).to(bf)
    x, dy = rnd(n, d), rnd(n, d)
    dx = torch.empty_like(x)
    uploads, result = [x, dy], dx          # what the end-to-end step moves
    if piece == "gemm":
        Wb = rnd(dff, d, s=1.0 / math.sqrt(d))
        C = torch.empty((n, dff), dtype=bf, device="cuda")
        desc = mb.make_gemm_desc(n, dff, d, 0, 0)
        uploads, result = [x], C

        def step():
            mb.moa_gemm(desc, x, Wb, C, None, stream)

        alg = 2.0 * n * d * dff
        unit, kernel = "TFLOP/s", "tc_gemm_kernel"
        metric = "bf16 GEMM C = A B^T: TFLOP/s"
    elif piece == "rmsnorm":
        eps = 1e-5
        g = (1.0 + 0.25 * torch.randn((d,), generator=gen, device="cuda")).to(bf)
        y, dg = torch.empty_like(x), torch.empty_like(g)
        r = torch.empty((n,), dtype=torch.float32, device="cuda")
        desc = mb.make_rmsnorm_desc(n, d, eps)
        ws = torch.empty(max(mb.moa_rmsnorm_workspace_bytes(desc), 16), dtype=torch.uint8, device="cuda")

        def step():
            mb.moa_rmsnorm_fwd(desc, x, g, y, r, stream)
            mb.moa_rmsnorm_bwd(desc, x, g, r, dy, dx, dg, ws, stream)

        # forward: read x, write y, r; backward: read x, dy, r, write dx (+ g, dg and the dg partials: O(d))
        alg = 5.0 * n * d * 2 + 8.0 * n
        unit, kernel = "GB/s", "rmsnorm_bwd_kernel"
        metric = "RMSNorm forward+backward: GB/s of algorithmic bytes"
    else:
        W1, W3 = rnd(dff, d, s=1.0 / math.sqrt(d)), rnd(dff, d, s=1.0 / math.sqrt(d))
        W2 = rnd(d, dff, s=1.0 / math.sqrt(dff))
        a, u, h = (torch.empty((n, dff), dtype=bf, device="cuda") for _ in range(3))
        y = torch.empty_like(x)
        dW1, dW3, dW2 = torch.empty_like(W1), torch.empty_like(W3), torch.empty_like(W2)
        desc = mb.make_mlp_desc(n, d, dff)
        ws = torch.empty(max(mb.moa_gated_mlp_workspace_bytes(desc), 16), dtype=torch.uint8, device="cuda")

        def step():
            mb.moa_gated_mlp_fwd(desc, x, W1, W3, W2, a, u, h, y, stream)
            mb.moa_gated_mlp_bwd(desc, x, W1, W3, W2, a, u, h, dy, dx, dW1, dW3, dW2, ws, stream)

        alg = 18.0 * n * d * dff           # 3 GEMMs forward, 6 backward, 2 n d d_ff each
        unit, kernel = "TFLOP/s", "tc_gemm_kernel"
        metric = "gated MLP forward+backward: model TFLOP/s (18 n d d_ff per step)"

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    l0 = mb.moa_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    sampler.stop()
    launches = mb.moa_launch_count() - l0
    ms = e0.elapsed_time(e1) / args.steps
    value = alg / (ms * 1e-3) / (1e9 if piece == "rmsnorm" else 1e12)
    # end to end: the step's activations (x, dy) come from pinned host memory, dx goes back; weights stay resident
    hup = [t.cpu().pin_memory() for t in uploads]
    hres = torch.empty(tuple(result.shape), dtype=bf).pin_memory()
    t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    esteps = max(4, min(args.steps, 10))
    t0e.record(stream)
    for _ in range(esteps):
        for t, ht in zip(uploads, hup):
            t.copy_(ht, non_blocking=True)
        step()
        hres.copy_(result, non_blocking=True)
    t1e.record(stream)
    torch.cuda.synchronize()
    e2e_ms = t0e.elapsed_time(t1e) / esteps
    st = mb.moa_last_device_status(stream)
    if st != mb.MOA_OK:
        raise SystemExit(f"device status: {mb.status_string(st)}")
    if piece == "rmsnorm":
        roof = {"bound": "hbm", "kernel": kernel, "achieved": value, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": value / peaks["hbm_gbs"], "traffic": None, "peak_source": f"{peaks_kind} hbm_gbs (copy bandwidth)",
                "algorithmic_bytes_per_step": alg,
                "note": "whole step (forward, backward, dg reduction) against the copy bandwidth"}
    else:
        roof = {"bound": "tensor", "kernel": kernel, "achieved": value, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": value / peaks["bf16_tflops"], "traffic": None,
                "peak_source": f"{peaks_kind} bf16_tflops (cuBLAS burst)",
                "frac_of_sustained": value / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                "model_flops_per_step": alg,
                "note": ("one product against the dense bf16 peak" if piece == "gemm" else
                         "whole step (the nine GEMMs of forward and backward) against the dense bf16 peak")}
    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.block, **({"M": n, "K": d, "N": dff} if piece == "gemm" else {"n": n, "d": d, "d_ff": dff}),
                   "l2": "the arrays of one step exceed the 126 MB L2; no explicit flush" if n * d * 10 > 126e6 or n * dff * 2 > 126e6
                   else "small case: resident in L2 between steps (not a bandwidth figure)"},
        "tokens_per_s": n / (ms * 1e-3),
        "clocks": sampler.summary(),
        "e2e": {"value": alg / (e2e_ms * 1e-3) / (1e9 if piece == "rmsnorm" else 1e12), "unit": unit,
                "h2d_bytes_per_step": sum(t.numel() for t in uploads) * 2, "d2h_bytes_per_step": result.numel() * 2,
                "ms_per_step": e2e_ms,
                "how": ("A from pinned host memory and C back every step; B resident" if piece == "gemm" else
                        "x and dy from pinned host memory and dx back every step; gain / weights resident")},
        "gpu_launches": int(launches),
        "roofline": roof,
    }
    if not args.no_cpu_baseline:
        rows = 4096 if piece == "rmsnorm" else (256 if piece == "gemm" else (64 if d * dff > 1 << 20 else n))
        f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
        t0 = time.perf_counter()
        reps = 0
        if piece == "gemm":
            xs, wb = f64(x[:rows]), f64(Wb)
            t0 = time.perf_counter()
            while time.perf_counter() - t0 < 5.0:
                oracle.gemm(xs, wb)
                reps += 1
        elif piece == "rmsnorm":
            xs, gs, ds = f64(x[:rows]), f64(g), f64(dy[:rows])
            while time.perf_counter() - t0 < 5.0:
                oracle.rmsnorm_fwd_bwd(xs, gs, ds, eps)
                reps += 1
        else:
            xs, ds, w1, w3, w2 = f64(x[:rows]), f64(dy[:rows]), f64(W1), f64(W3), f64(W2)
            t0 = time.perf_counter()
            while time.perf_counter() - t0 < 10.0:
                oracle.gated_mlp_fwd_bwd(xs, w1, w3, w2, ds)
                reps += 1
        dt = (time.perf_counter() - t0) / reps
        sample = alg * rows / n
        line["cpu_baseline"] = {"value": sample / dt / (1e9 if piece == "rmsnorm" else 1e12), "unit": unit,
                                "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"{rows} of {n} tokens (all columns / full weights), numpy fp64", "seconds": dt * reps}
    print(json.dumps(line))
    return 0


def run_whole_block(args):
    """The complete pre-norm transformer block, forward+backward, as the fixed sequence of library calls of
    paper_2609_33916_b200/block.py (14 calls with the packed Q/K/V projection).  Metric: model TFLOP/s of the block."""
    import numpy as np
    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    from paper_2609_33916_b200.block import TransformerBlock, WEIGHTS
    import oracle

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    _, B, n, H, d, dff, causal = BLOCK_WORKLOADS[args.block]
    mbuild.build()
    mb.lib()
    peaks, peaks_kind = load_peaks()
    T, dm = B * n, H * d
    bf = torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(19)
    rnd = lambda *shape, s=1.0: (torch.randn(shape, generator=gen, device="cuda") * s).to(bf)
    x, dy = rnd(T, dm), rnd(T, dm)
    w = dict(g1=(1.0 + 0.25 * torch.randn((dm,), generator=gen, device="cuda")).to(bf),
             g2=(1.0 + 0.25 * torch.randn((dm,), generator=gen, device="cuda")).to(bf),
             Wq=rnd(dm, dm, s=dm ** -0.5), Wk=rnd(dm, dm, s=dm ** -0.5), Wv=rnd(dm, dm, s=dm ** -0.5), Wo=rnd(dm, dm, s=dm ** -0.5),
             W1=rnd(dff, dm, s=dm ** -0.5), W3=rnd(dff, dm, s=dm ** -0.5), W2=rnd(dm, dff, s=dff ** -0.5))
    blk = TransformerBlock(torch, B, n, H, d, dff, causal)
    w = blk.prepare_weights(w)          # the stacked projection weight [Wq; Wk; Wv], built once outside the step
    stream = torch.cuda.current_stream()
    flops = blk.model_flops()

    def direct_step():
        blk.forward(x, w, stream)
        blk.backward(x, w, dy, stream)

    step = direct_step
    launches_per_replay = None
    if args.graph:
        # the calls allocate nothing and synchronise nothing: after a warm-up call the launches of a step are
        # recorded once and the timed region replays them (what a launch-bound size such as the paper's gains)
        direct_step()
        torch.cuda.synchronize()
        cap, graph, user_stream = torch.cuda.Stream(), torch.cuda.CUDAGraph(), stream
        lc0 = mb.moa_launch_count()
        with torch.cuda.graph(graph, stream=cap):
            stream = torch.cuda.current_stream()
            direct_step()
        launches_per_replay = mb.moa_launch_count() - lc0
        stream = user_stream

        def step():
            graph.replay()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    l0 = mb.moa_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    sampler.stop()
    launches = mb.moa_launch_count() - l0 if launches_per_replay is None else launches_per_replay * args.steps
    ms = e0.elapsed_time(e1) / args.steps
    value = flops / (ms * 1e-3) / 1e12
    # per-kind kernel time of one more step (outside the timed region)
    mb.moa_profile_read()
    mb.moa_profile_enable(True)
    direct_step()
    torch.cuda.synchronize()
    mb.moa_profile_enable(False)
    prof = {k: [round(v[0], 4), v[1]] for k, v in mb.moa_profile_read().items() if v[1]}
    # end to end: x and dy from pinned host memory, dx back, every step; weights resident
    hx, hdy = x.cpu().pin_memory(), dy.cpu().pin_memory()
    hdx = torch.empty((T, dm), dtype=bf).pin_memory()
    esteps = max(4, min(args.steps, 10))
    t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0e.record(stream)
    for _ in range(esteps):
        x.copy_(hx, non_blocking=True)
        dy.copy_(hdy, non_blocking=True)
        step()
        hdx.copy_(blk.dx, non_blocking=True)
    t1e.record(stream)
    torch.cuda.synchronize()
    e2e_ms = t0e.elapsed_time(t1e) / esteps
    st = mb.moa_last_device_status(stream)
    if st != mb.MOA_OK:
        raise SystemExit(f"device status: {mb.status_string(st)}")
    att = 14.0 * B * H * float(n) ** 2 * d * (0.5 if causal else 1.0)
    line = {
        "metric": "transformer block forward+backward: model TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.block, "B": B, "n": n, "H": H, "d": d, "d_model": dm, "d_ff": dff, "causal": causal,
                   "cuda_graph": bool(args.graph),
                   "l2": "the activations of one step exceed the 126 MB L2; no explicit flush" if T * dff * 2 > 126e6
                   else "small case: mostly resident in L2 between steps"},
        "model_flops": {"total": flops, "attention": att, "projections": 24.0 * T * dm * dm, "gated_mlp": 18.0 * T * dm * dff},
        "tokens_per_s": T / (ms * 1e-3),
        "clocks": sampler.summary(),
        "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": 2 * T * dm * 2,
                "d2h_bytes_per_step": T * dm * 2, "ms_per_step": e2e_ms,
                "how": "x and dy from pinned host memory and dx back every step; weights resident"},
        "gpu_launches": int(launches),
        "per_kind_ms": prof,
        "roofline": {"bound": "tensor", "kernel": "whole step (attention, GEMMs)", "achieved": value, "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": value / peaks["bf16_tflops"], "traffic": None,
                     "peak_source": f"{peaks_kind} bf16_tflops (cuBLAS burst)",
                     "frac_of_sustained": value / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])},
    }
    if not args.no_cpu_baseline:
        # the oracle block on a shorter sequence of the same widths (attention is O(n^2): the rate differs by piece)
        ns = min(n, 256)
        f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
        ws = {k: f64(v) for k, v in w.items()}
        xs, ds = f64(x[:ns]), f64(dy[:ns])
        t0 = time.perf_counter()
        oracle.transformer_block_fwd_bwd(xs, ws, ds, 1, ns, H, causal, 1e-5)
        dt = time.perf_counter() - t0
        sf = 24.0 * ns * dm * dm + 14.0 * H * float(ns) ** 2 * d * (0.5 if causal else 1.0) + 18.0 * ns * dm * dff
        line["cpu_baseline"] = {"value": sf / dt / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"one sequence of {ns} tokens, same widths and weights, numpy fp64 + the C attention oracle",
                                "seconds": dt}
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- sweep
def run_sweep(args):
    """Config-5 style sweep: for each n and each strategy (the three dQ modes of the fused path
    and the n x n-materialising variant) one JSON line with time, TFLOP/s, per-kernel times and
    peak device bytes; then the local scaling exponents log2(t(2n)/t(n)) per strategy.  Not the
    contract line: a study table."""
    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    from paper_2609_33916_b200 import inputs as mi
    mbuild.build()
    torch.cuda.set_device(0)
    peaks, peaks_kind = load_peaks()
    strategies = [("fused_red", 1, 0), ("fused_bulk_reduce", 2, 0), ("fused_separate_pass", 3, 0), ("materialize", 0, 1)]
    sizes = [int(x) for x in args.sweep_sizes.split(",")] if args.sweep_sizes else list(mi.C5_SIZES)
    times = {}
    for n in sizes:
        w = mi.CONFIGS[f"c5_causal_n{n}"] if f"c5_causal_n{n}" in mi.CONFIGS else mi.Workload(f"sweep_n{n}", 1, 32, n, 128, True, "bf16", 4)
        shape = (w.B, w.H, w.n, w.d)
        gen = torch.Generator(device="cuda").manual_seed(w.seed)
        Q, K, V, dO = (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(4))
        O, dQ, dK, dV = (torch.empty(shape, dtype=torch.bfloat16, device="cuda") for _ in range(4))
        L = torch.empty((w.B, w.H, w.n), dtype=torch.float32, device="cuda")
        io_bytes = sum(t.numel() * t.element_size() for t in (Q, K, V, dO, O, dQ, dK, dV, L))
        for name, dq_mode, mat in strategies:
            desc = mb.make_desc(w.B, w.H, w.n, w.d, w.causal, w.scale, mb.MOA_BF16, dq_mode, mat, 0)
            ws_bytes = mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_FUSED)
            free, _ = torch.cuda.mem_get_info()
            line = {"sweep": "c5", "n": n, "strategy": name, "workspace_bytes": ws_bytes, "io_bytes": io_bytes,
                    "peak_device_bytes": io_bytes + ws_bytes}
            if ws_bytes + (1 << 30) > free:
                line["skipped"] = f"needs {ws_bytes / 2**30:.1f} GiB of workspace"
                print(json.dumps(line), flush=True)
                continue
            ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
            stream = torch.cuda.current_stream()
            steps = 3 if n >= 16384 else (5 if n >= 4096 else 20)
            for _ in range(3):
                mb.moa_attn_fused_fwd_bwd(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws, stream)
            torch.cuda.synchronize()
            mb.moa_profile_read(); mb.moa_profile_enable(True)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                mb.moa_attn_fused_fwd_bwd(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            mb.moa_profile_enable(False)
            prof = mb.moa_profile_read()
            st = mb.moa_last_device_status(stream)
            ms = e0.elapsed_time(e1) / steps
            tf = w.model_flops / (ms * 1e-3) / 1e12
            times[(name, n)] = ms
            line.update({"ms": ms, "tflops": tf, "pct_of_measured_burst_peak": 100 * tf / peaks["bf16_tflops"],
                         "status": mb.status_string(st),
                         "per_kernel_ms": {k: v[0] / max(1, v[1]) * (v[1] / steps) for k, v in prof.items() if v[1]}})
            if mat:   # HBM-bound variant: n^2 traffic per head = P^T and dS^T written once and read once
                npad = (n + 127) // 128 * 128
                tri = 0.5 if w.causal else 1.0
                line["nxn_bytes_moved_model"] = 8.0 * w.B * w.H * npad * npad * tri
                line["nxn_gbs"] = line["nxn_bytes_moved_model"] / (ms * 1e-3) / 1e9
            print(json.dumps(line), flush=True)
            del ws
            torch.cuda.empty_cache()
        del Q, K, V, dO, O, dQ, dK, dV, L
        torch.cuda.empty_cache()
    for name, _, _ in strategies:
        exps = {}
        for a, b in zip(sizes[:-1], sizes[1:]):
            if (name, a) in times and (name, b) in times and b == 2 * a:
                exps[f"{a}->{b}"] = math.log2(times[(name, b)] / times[(name, a)])
        print(json.dumps({"sweep": "c5", "strategy": name, "local_time_exponent": exps}), flush=True)
    return 0


# ------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="moa", choices=["moa", "reference"])
    ap.add_argument("--workload", default="c4_long")
    ap.add_argument("--dq-mode", type=int, default=0)
    ap.add_argument("--path", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--materialize", type=int, default=0)
    ap.add_argument("--graph", action="store_true",
                    help="record the step into a CUDA graph once and time replays (launch-bound small sizes)")
    ap.add_argument("--decode", default="", choices=[""] + sorted(DECODE_WORKLOADS),
                    help="time decode attention on that workload instead of the fused forward+backward")
    ap.add_argument("--block", default="", choices=[""] + sorted(BLOCK_WORKLOADS),
                    help="time a block piece (RMSNorm or gated MLP, forward+backward) instead of the attention step")
    ap.add_argument("--rowparallel", type=int, default=0,
                    help="1 or 2: time the row-parallel single-kernel comparison variant with that many atomic sites")
    ap.add_argument("--layout", type=int, default=0, help="0: tensors [B,H,n,d] (every named config); 1: [B,n,H,d]")
    ap.add_argument("--hkv", type=int, default=0,
                    help="key/value heads (grouped-query attention); 0: one per query head, as in every named config")
    ap.add_argument("--sweep", action="store_true", help="config-5 strategy sweep (study table, not the contract line)")
    ap.add_argument("--sweep-sizes", default="")
    ap.add_argument("--dist-backend", default="nccl", help="control-plane backend for N > 1 (nccl; gloo for tests)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: every rank runs the whole workload (weak), or the heads are partitioned over the ranks (strong)")
    ap.add_argument("--stub-ms-per-tflop", type=float, default=0.0,
                    help="testing aid: replace the library call by a sleep of this many ms per TFLOP (no GPU needed)")
    ap.add_argument("--all-ranks-on-device0", action="store_true",
                    help="testing aid: every rank uses cuda:0 (ranks never wait on one another's kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "moa" else args.warmup

    if args.decode or args.block:
        # single-GPU legs: under a multi-rank launch rank 0 alone runs them
        if int(os.environ.get("RANK", "0")) != 0:
            return 0
        return run_decode(args) if args.decode else run_block(args)
    from paper_2609_33916_b200 import inputs as mi
    w = mi.CONFIGS[args.workload]
    if args.impl == "reference":
        return run_reference(args, w)
    if args.sweep:
        return run_sweep(args)
    if args.stub_ms_per_tflop > 0:
        return run_stub(args, w)

    import torch
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    if args.all_ranks_on_device0:
        local_rank = 0
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        if args.dist_backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(args.dist_backend)
    if rank == 0:
        mbuild.build()
    if dist is not None:
        dist.barrier()
    mb.lib()
    peaks, peaks_kind = load_peaks()

    plan = rank_plan(w, world, rank, args.shard, args.hkv)      # this rank's share: everything, or a block of heads
    if plan["heads"] == 0:
        raise SystemExit(f"rank {rank}: more ranks than heads to hand out ({w.B * w.H} heads, {world} ranks)")
    B, H, n, d = plan["B"], plan["H"], w.n, w.d
    hkv = plan["H_kv"]
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16      # config 1 is the fp32 path
    desc = mb.make_desc(B, H, n, d, w.causal, w.scale, mb.MOA_F32 if w.dtype == "f32" else mb.MOA_BF16, args.dq_mode, args.materialize, args.path,
                        H_kv=hkv, layout=args.layout)
    shape = (B, n, H, d) if args.layout else (B, H, n, d)
    kv_shape = (B, n, hkv or H, d) if args.layout else (B, hkv or H, n, d)       # K, V, dK, dV
    shapes_in = (shape, kv_shape, kv_shape, shape)            # Q, K, V, dO
    shapes_out = (shape, shape, kv_shape, kv_shape)           # O, dQ, dK, dV
    base_mem = torch.cuda.memory_allocated()
    gen = torch.Generator(device="cuda").manual_seed(w.seed + 1000 * rank)
    Q, K, V, dO = (torch.randn(sh, generator=gen, device="cuda", dtype=torch.float32).to(tdt)
                   for sh in shapes_in)
    O, dQ, dK, dV = (torch.empty(sh, dtype=tdt, device="cuda") for sh in shapes_out)
    L = torch.empty((B, H, n), dtype=torch.float32, device="cuda")
    ws_bytes = mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_FUSED)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    resident_bytes = torch.cuda.memory_allocated() - base_mem
    stream = torch.cuda.current_stream()

    if args.rowparallel:
        ws_bytes = mb.moa_attn_workspace_bytes(desc, mb.MOA_OP_ROWPARALLEL)
        ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")

    def step():
        if args.rowparallel:
            mb.moa_attn_fused_rowparallel(desc, Q, K, V, dO, O, L, dQ, dK, dV, args.rowparallel, ws, stream)
        else:
            mb.moa_attn_fused_fwd_bwd(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws, stream)

    direct_step = step
    if args.graph:
        # the library allocates nothing and synchronises nothing: after one warm-up call (which resolves
        # the per-device symbols) the step is recorded once and the timed region replays it
        direct_step()
        torch.cuda.synchronize()
        cap = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        user_stream = stream
        lc0 = mb.moa_launch_count()
        with torch.cuda.graph(graph, stream=cap):
            stream = torch.cuda.current_stream()
            direct_step()
        launches_per_replay = mb.moa_launch_count() - lc0     # kernels recorded in the graph
        stream = user_stream

        def step():
            graph.replay()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda" if args.dist_backend == "nccl" else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(x: float) -> float:
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda" if args.dist_backend == "nccl" else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    for _ in range(args.warmup):
        step()
    st = mb.moa_last_device_status(stream)
    if st != mb.MOA_OK:
        raise SystemExit(f"device status after warm-up: {mb.status_string(st)}")

    # ---- timed region: K steps, device-resident inputs ----
    sampler = ClockSampler(physical_gpu_index(local_rank))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    launches0 = mb.moa_launch_count()
    step_ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    wall0 = time.perf_counter()
    e0.record(stream)
    step_ev[0].record(stream)
    for i in range(args.steps):
        step()
        step_ev[i + 1].record(stream)
    e1.record(stream)
    barrier()
    wall_ms = (time.perf_counter() - wall0) * 1e3 / args.steps
    launches = mb.moa_launch_count() - launches0
    if args.graph:
        launches = launches_per_replay * args.steps        # replays launch the recorded kernels without host calls
    sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    # per-kernel durations: a separate pass after the timed region, so that the event pairs the
    # library records around every launch do not sit inside the timed steps
    mb.moa_profile_read()
    mb.moa_profile_enable(True)
    for _ in range(max(3, min(args.steps, 10))):
        direct_step()
    torch.cuda.synchronize()
    mb.moa_profile_enable(False)
    prof = mb.moa_profile_read()
    ms_per_step = ms_total / args.steps
    per_step = sorted(step_ev[i].elapsed_time(step_ev[i + 1]) for i in range(args.steps))
    # device time (CUDA events) and wall clock side by side: the paper found 17 % host overhead
    # hiding in wall-clock timings (Sec. 3), so both are reported
    timing = {"ms_min": per_step[0], "ms_median": statistics.median(per_step), "ms_mean": ms_per_step,
              "wall_ms_per_step_incl_final_sync": wall_ms}
    flops_step = plan["flops"]                       # this rank's model flops per step
    flops_job = sum_over_ranks(flops_step)           # all ranks'
    value = flops_job / (ms_per_step * 1e-3) / 1e12
    peak_bytes = torch.cuda.max_memory_allocated() - base_mem

    # ---- end to end: pinned host inputs -> device, call, results -> pinned host ----
    # Every step copies its own inputs from pinned host memory and reads all its results back.
    # The three legs run on three streams over two buffer sets, so step k+1's upload and step
    # k-1's download overlap step k's kernels (the library call takes the stream it runs on).
    hQ, hK, hV, hdO = (t.cpu().pin_memory() for t in (Q, K, V, dO))
    hO, hdQ, hdK, hdV = (torch.empty(sh, dtype=tdt).pin_memory() for sh in shapes_out)
    hL = torch.empty((B, H, n), dtype=torch.float32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (hQ, hK, hV, hdO))
    d2h = sum(t.numel() * t.element_size() for t in (hO, hdQ, hdK, hdV, hL))
    sets = []
    for _ in range(2):
        ins = [torch.empty(sh, dtype=tdt, device="cuda") for sh in shapes_in]
        outs = [torch.empty(sh, dtype=tdt, device="cuda") for sh in shapes_out]
        sets.append({"in": ins, "out": outs, "L": torch.empty((B, H, n), dtype=torch.float32, device="cuda"),
                     "ws": torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda"),
                     "up": torch.cuda.Event(), "done": torch.cuda.Event(), "down": torch.cuda.Event()})
    s_up, s_run, s_down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_step(k):
        b = sets[k % 2]
        with torch.cuda.stream(s_up):
            s_up.wait_event(b["done"])           # the previous user of this set has finished computing
            for dst, src in zip(b["in"], (hQ, hK, hV, hdO)):
                dst.copy_(src, non_blocking=True)
            b["up"].record(s_up)
        with torch.cuda.stream(s_run):
            s_run.wait_event(b["up"])
            s_run.wait_event(b["down"])          # its previous results have been read back
            if args.rowparallel:
                mb.moa_attn_fused_rowparallel(desc, b["in"][0], b["in"][1], b["in"][2], b["in"][3], b["out"][0], b["L"],
                                              b["out"][1], b["out"][2], b["out"][3], args.rowparallel, b["ws"], s_run)
            else:
                mb.moa_attn_fused_fwd_bwd(desc, b["in"][0], b["in"][1], b["in"][2], b["in"][3], b["out"][0], b["L"],
                                          b["out"][1], b["out"][2], b["out"][3], b["ws"], s_run)
            b["done"].record(s_run)
        with torch.cuda.stream(s_down):
            s_down.wait_event(b["done"])
            for dst, src in zip((hO, hdQ, hdK, hdV), b["out"]):
                dst.copy_(src, non_blocking=True)
            hL.copy_(b["L"], non_blocking=True)
            b["down"].record(s_down)

    for k in range(2):
        e2e_step(k)
    barrier()
    e2e_steps = max(4, args.steps)      # the same K steps as the device-resident leg (pipeline fill and drain included)
    t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0e.record(s_up)
    for k in range(e2e_steps):
        e2e_step(k)
    s_down.wait_stream(s_run)
    t1e.record(s_down)
    barrier()
    e2e_ms = max_over_ranks(t0e.elapsed_time(t1e)) / e2e_steps
    e2e_value = flops_job / (e2e_ms * 1e-3) / 1e12
    st = mb.moa_last_device_status(stream)
    if st != mb.MOA_OK:
        raise SystemExit(f"device status: {mb.status_string(st)}")

    # ---- roofline of the dominant kernel (the key-tile-parallel backward) ----
    heads = B * H
    causal_f = 0.5 if w.causal else 1.0
    alg_flops = {"fwd": 4.0 * heads * n * n * d * causal_f, "bwd_kv": 10.0 * heads * n * n * d * causal_f,
                 "bwd_dq": 0.0}
    if prof["bwd_dq"][1] > 0:   # separate pass: dQ's 2 n^2 d moves to that kernel (its recompute is not credited)
        alg_flops["bwd_kv"] = 8.0 * heads * n * n * d * causal_f
        alg_flops["bwd_dq"] = 2.0 * heads * n * n * d * causal_f
    # algorithmic HBM bytes per launch (bf16 tensors read and written once, fp32 row vectors, the fp32 dQ accumulator
    # added into and read back by the conversion): what the method must move, for comparison with measured traffic
    kvh = (hkv or H) * B
    alg_bytes = {"fwd": 2.0 * n * d * (2 * heads + 2 * kvh) + 4.0 * heads * n,
                 "bwd_kv": 2.0 * n * d * (2 * heads + 4 * kvh) + 8.0 * heads * n + 4.0 * heads * n * d,
                 "bwd_dq": 2.0 * n * d * (3 * heads + 2 * kvh) + 8.0 * heads * n}
    dominant = max(("fwd", "bwd_kv", "bwd_dq"), key=lambda k: prof[k][0])
    dom_ms = prof[dominant][0] / max(1, prof[dominant][1])
    achieved = alg_flops[dominant] / (dom_ms * 1e-3) / 1e12 if dom_ms > 0 else None
    # Denominator: MEASURED_PEAKS holds a burst figure (a kernel timed alone or in a sub-second run, clocks near
    # their maximum) and a sustained one (a seconds-long loop under the power cap).  The one that applies follows
    # from the timed region's own length; both fractions are carried.
    long_run = ms_total >= 1000.0
    peak_name = "bf16_tflops_sustained" if long_run else "bf16_tflops"
    peak = peaks[peak_name]
    # DRAM traffic of the dominant kernel: from the committed record of an ncu capture (profiles/traffic.json), for
    # the kernel family that was captured only, scaled by tokens (traffic is linear in B*H*n); null otherwise
    traffic, traffic_source = None, None
    rec = load_traffic_record(dominant)
    fam = rec and rec.get("family", {})
    if rec and dominant == "bwd_kv" and d == fam.get("d") and bool(w.causal) == bool(fam.get("causal")) and \
            not hkv and not args.layout and not args.materialize and args.path in (0, 2) and \
            (args.dq_mode or 2) == fam.get("dq_mode") and not mb.moa_bwd_pair_mode(-1):
        traffic = rec["dram_bytes_per_launch"] / rec["tokens"] * heads * n
        traffic_source = (f"extrapolated from an ncu capture of {rec['case']} ({rec['dram_bytes_per_launch'] / 1e6:.1f} MB "
                          f"read+written per launch), scaled by tokens")
    roofline = {"bound": "tensor", "kernel": dominant, "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": (achieved / peak) if achieved else None,
                "frac_of_burst": (achieved / peaks["bf16_tflops"]) if achieved else None,
                "frac_of_sustained": (achieved / peaks["bf16_tflops_sustained"]) if achieved else None,
                "traffic": traffic, "traffic_source": traffic_source,
                "algorithmic_hbm_bytes": alg_bytes.get(dominant),
                "peak_source": f"{peaks_kind} {peak_name}: the timed region ran {ms_total / 1e3:.2f} s "
                               f"({'a second or more: sustained' if long_run else 'under a second: burst'})",
                "kernel_ms": dom_ms,
                "per_kernel_ms": {k: (v[0] / max(1, v[1]), v[1]) for k, v in prof.items() if v[1]}}
    # clock-normalised figure: ms x median SM MHz under load (runs at different power-capped clocks compare on it)
    clk = sampler.summary()
    if clk.get("sm_mhz"):
        timing["ms_times_sm_mhz"] = ms_per_step * clk["sm_mhz"]
        timing["value_at_max_clock"] = value * clk["sm_max_mhz"] / clk["sm_mhz"] if clk.get("sm_max_mhz") else None

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if (args.shard == "heads" and world > 1) else "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": workload_config(w, args),
        "pct_of_peak": {"of_measured_burst": 100 * value / world / peaks["bf16_tflops"],
                        "of_measured_sustained": 100 * value / world / peaks["bf16_tflops_sustained"],
                        "of_nominal_2250": 100 * value / world / NOMINAL_BF16_TFLOPS, "peaks": peaks_kind},
        "hbm_bytes": {"resident_inputs_outputs_workspace": resident_bytes, "peak_allocated": peak_bytes,
                      "workspace": ws_bytes, "one_nxn_fp32_array_all_heads_not_allocated": 4 * heads * n * n},
        "clocks": clk,
        "timing": timing,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms, "how": "pinned host buffers; upload, kernels and download on three streams, "
                                              "two device buffer sets; every step moves all its inputs and outputs"},
        "gpu_launches": int(launches),
        "roofline": roofline,
    }
    if args.hkv:
        line["config"]["H_kv"] = args.hkv
    if args.layout:
        line["config"]["layout"] = "[B,n,H,d]"
    if args.graph:
        line["config"]["launch"] = "one CUDA graph replay per step"
    if args.rowparallel:
        line["config"]["variant"] = f"row-parallel single kernel, {args.rowparallel} atomic site(s), fp32 CUDA cores"
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.hkv and not args.layout and not args.rowparallel:
        v, dt, cores, desc_s = time_oracle_sample(w, 20.0)
        line["cpu_baseline"] = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                                "sample": desc_s, "seconds": dt}
        if w.n <= 1024 and cores > 1:       # small n: one thread may beat all cores (the paper's over-threading finding)
            one = time_oracle_one_thread(w, 10.0)
            if one:
                line["cpu_baseline"]["one_thread"] = one
                if one["value"] > v:
                    line["cpu_baseline"].update(value=one["value"], cores=1, sample=one["sample"], seconds=one["seconds"],
                                                all_cores={"value": v, "cores": cores, "seconds": dt})
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
