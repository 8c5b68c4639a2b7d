#!/usr/bin/env python
"""Benchmark of the masked parallel-drafting attention hot path (mask evaluator + tile
classifier + forward + backward + partition driver) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one call of ``peagle_attn_partitioned`` over the whole workload.  The metric is useful
(unmasked) TFLOP/s: 14 * P * head_dim * n_q_heads per step, P = allowed (query, key) pairs.
With N > 1 every rank runs an independent replica of the workload on its own GPU (the path has
no exchange step); the value is the sum over ranks divided by the slowest rank's time.
``--impl reference`` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_01469_b200 import inputs  # noqa: E402

METRIC = "masked-attn fwd+bwd useful TFLOP/s"
UNIT = "TFLOP/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel come from
# profiles/traffic.json, which records next to each figure the SHA-256 of the kernel's source
# files at the time of the ncu capture; a figure whose sources have changed since reads as null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")
CSRC = os.path.join(ROOT, "paper_2602_01469_b200", "csrc")
BWD_KERNEL = {64: "bwd64_kernel", 128: "bwd128_kernel"}
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def grid(w: inputs.Workload, i: int, n: int):
    """Metadata of sequence i of a workload: the full grid, or its COD-subsampled version."""
    return inputs.full_grid(n, w.K) if w.cod_r is None else inputs.cod_grid(n, w.K, w.cod_r, w.seed + i)


def allowed_pairs(w: inputs.Workload) -> int:
    """Allowed (query, key) pairs: a token (anchor a, depth d) sees the a+1 real tokens up to its
    anchor and its d chain tokens (all present: the kept sets are nested along chains)."""
    total = 0
    for i, n in enumerate(w.seq_lens):
        a, d = grid(w, i, n)
        total += int(a.astype(np.int64).sum() + d.astype(np.int64).sum() + a.shape[0])
    return total


def useful_flops(w: inputs.Workload):
    p = allowed_pairs(w)
    fwd = 4 * p * w.head_dim * w.n_q_heads
    bwd = 10 * p * w.head_dim * w.n_q_heads
    return fwd, bwd


def source_hash(files) -> str:
    import hashlib
    h = hashlib.sha256()
    for name in sorted(files):
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of `kernel` on `workload` from the recorded ncu capture, or None when
    there is no record or the kernel's sources are no longer the ones that were profiled."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(workload, {}).get(kernel)
        if rec and source_hash(rec["sources"]) == rec["sources_sha256"]:
            return int(rec["dram_bytes_per_launch"])
    except (OSError, ValueError, KeyError):
        pass
    return None


def config_dict(w: inputs.Workload, T: int, n_parts: int) -> dict:
    """The workload description both arms print."""
    f_fwd, f_bwd = useful_flops(w)
    return {"workload": w.name, "seq_lens": list(w.seq_lens) if len(w.seq_lens) < 4 else
            f"{len(w.seq_lens)} sequences", "K": w.K, "total_tokens": T,
            "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
            "partitions": n_parts, "allowed_pairs": allowed_pairs(w),
            "useful_tflop_per_step": (f_fwd + f_bwd) / 1e12,
            "l2": "inputs (>1 GB) larger than L2, no flush", "parallelism": "replicas"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: one nvidia-smi process
    in loop mode (a sample every 100 ms), read when the region ends."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.samples = []
        self.proc = None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i",
                 str(self.idx), "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.3)          # let the first sample arrive before the region starts
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *a):
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=10)
        except Exception:
            self.proc.kill()
            out = ""
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) >= 6:
                try:
                    self.samples.append((float(f[0]), float(f[1]), f[2:6]))
                except ValueError:
                    pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for s in self.samples for n, v in zip(names, s[2]) if v.lower() == "active"})
        # the first samples predate the timed region: use the busy half (highest power draw is not
        # reported here, so take the samples from the middle on)
        busy = self.samples[len(self.samples) // 3:] or self.samples
        return {"sm_mhz": float(np.median([s[0] for s in busy])),
                "sm_min_mhz": float(min(s[0] for s in busy)),
                "sm_max_mhz": self.samples[0][1], "reasons": reasons, "samples": len(self.samples)}


# ------------------------------------------------------------------ CPU oracle arm
def oracle_sample(w: inputs.Workload, budget_s: float, seed: int = 0):
    """Times the fp64 oracle (forward + backward) on random query rows of the workload's longest
    sequence, all heads, until about ``budget_s`` seconds are spent.  Returns useful TFLOP/s."""
    from oracle import partition as opart
    from oracle import peagle_oracle as orc

    i_long = int(np.argmax(w.seq_lens))
    n = w.seq_lens[i_long]
    anchor, depth = grid(w, i_long, n)
    T = int(anchor.shape[0])
    Q, K, V, dO = inputs.make_tensors(T, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seed)
    Qf, Kf, Vf, dOf = (t.float().numpy() for t in (Q, K, V, dO))
    rng = np.random.default_rng(seed)
    rows_done, pairs_done, t_spent = 0, 0, 0.0
    chunk = max(8, orc.num_threads())
    while t_spent < budget_s:
        rows = np.sort(rng.choice(T, size=chunk, replace=False)).astype(np.int32)
        t0 = time.perf_counter()
        orc.attn_fwd(anchor, depth, Qf, Kf, Vf, w.scale, rows=rows)
        orc.attn_bwd(anchor, depth, Qf, Kf, Vf, dOf, w.scale, rows=rows)
        t_spent += time.perf_counter() - t0
        rows_done += len(rows)
        pairs_done += int(np.sum(anchor[rows] + 1 + depth[rows]))
        if t_spent < budget_s / 8:
            chunk *= 2
    flops = 14 * pairs_done * w.head_dim * w.n_q_heads
    return {"value": flops / t_spent / 1e12, "unit": UNIT, "cores": orc.num_threads(),
            "kind": "oracle",
            "sample": f"{rows_done} random query rows x {w.n_q_heads} heads of {w.name} "
                      f"(n={n}, K={w.K}), fwd+bwd, {t_spent:.1f} s"}, t_spent, flops


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import partition as opart

    def oracle_assign(anchor, depth, K, bounds):       # Algorithm 1 as the oracle side states it
        P = inputs.position_sets(anchor, depth, K)
        A, _, _ = opart.assign_segments(P, len(bounds) - 1, bounds[-1], B=bounds)
        return np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)

    cu, _, _, parts = inputs.build_case(w, oracle_assign)
    per_step = max(2.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(w, per_step / 4)
    tot_t, tot_f, last = 0.0, 0, None
    for i in range(args.steps):
        last, t, f = oracle_sample(w, per_step, seed=i + 1)
        tot_t += t
        tot_f += f
    value = tot_f / tot_t / 1e12
    last["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(w, int(cu[-1]), len(parts)),
        "note": "each step is a bounded sample of query rows; the value is useful FLOPs of the "
                "sample / time",
        "cpu_baseline": last,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------ CUDA arm
def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's figure (all-reduce MAX over the process group); x itself on one rank."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist

    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicas_value(world: int, flops_per_replica: float, ms_step: float) -> float:
    """Whole-job useful TFLOP/s of `world` independent replicas that all finish within ms_step."""
    return world * flops_per_replica / (ms_step * 1e-3) / 1e12


def run_cuda(args, w):
    import torch
    import torch.distributed as dist

    from paper_2602_01469_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    ctx = binding.Context(local_rank)
    cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
    T = int(cu[-1])
    Qc, Kc, Vc, dOc = inputs.make_tensors(T, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seed)
    Q, K, V, dO = (t.to(dev) for t in (Qc, Kc, Vc, dOc))
    d_anchor, d_depth = torch.from_numpy(anchor).to(dev), torch.from_numpy(depth).to(dev)
    O = torch.empty_like(Q)
    dQ = torch.empty_like(Q)
    dK, dV = torch.empty_like(K), torch.empty_like(V)
    LSE = torch.empty(w.n_q_heads, T, dtype=torch.float32, device=dev)
    prob = binding.Problem(cu, d_anchor, d_depth, w.K, w.n_q_heads, w.n_kv_heads, w.head_dim, w.scale)
    bparts = [binding.Partition(p["seq"], p["q"], p["k"]) for p in parts]
    stream = torch.cuda.current_stream()

    sharded = args.parallelism == "partitions"
    if sharded:
        # partition sharding: this rank's share of the query partitions against the full K / V,
        # partial fp32 dK / dV sums completed by one all-reduce (NCCL), then rounded
        from paper_2602_01469_b200 import sharding
        my_parts = [bparts[i] for i in sharding.deal_partitions(parts, world)[rank]]
        dK_acc = torch.zeros(T, w.n_kv_heads, w.head_dim, dtype=torch.float32, device=dev)
        dV_acc = torch.zeros_like(dK_acc)

    def step():
        if not sharded:
            binding.peagle_attn_partitioned(ctx, prob, bparts, Q, K, V, dO, O, LSE, dQ, dK, dV, stream)
            return
        dK_acc.zero_()
        dV_acc.zero_()
        binding.peagle_attn_partitioned_acc(ctx, prob, my_parts, Q, K, V, dO, O, LSE, dQ, dK_acc,
                                            dV_acc, stream)
        sharding.sum_over_ranks([dK_acc, dV_acc], world)
        binding.peagle_cast_grads(ctx, dK_acc, dV_acc, dK, dV, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if binding.peagle_poll_status(ctx) != 0:
        raise RuntimeError("device-side error during warm-up")
    binding.peagle_timing_enable(ctx, True)
    binding.peagle_timing_read(ctx)
    launches0 = binding.peagle_launch_count(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        barrier()
    ms_total = e0.elapsed_time(e1)
    (k_fwd_ms, k_bwd_ms), (n_fwd, n_bwd) = binding.peagle_timing_read(ctx)
    binding.peagle_timing_enable(ctx, False)
    launches = binding.peagle_launch_count(ctx) - launches0
    if binding.peagle_poll_status(ctx) != 0:
        raise RuntimeError("device-side error during the timed region")
    ms_total = max_over_ranks(ms_total, world, dev)
    ms_step = ms_total / args.steps
    f_fwd, f_bwd = useful_flops(w)
    # replicas: every rank does the whole workload; partitions: the ranks share one workload
    value = replicas_value(1 if sharded else world, f_fwd + f_bwd, ms_step)

    # ---- end to end through the host entry point (pinned host buffers, copies timed)
    hQ, hK, hV, hdO = (t.pin_memory() for t in (Qc, Kc, Vc, dOc))
    hO, hdQ = torch.empty_like(hQ).pin_memory(), torch.empty_like(hQ).pin_memory()
    hdK, hdV = torch.empty_like(hK).pin_memory(), torch.empty_like(hV).pin_memory()
    hLSE = torch.empty(w.n_q_heads, T, dtype=torch.float32).pin_memory()
    hprob = binding.Problem(cu, anchor, depth, w.K, w.n_q_heads, w.n_kv_heads, w.head_dim, w.scale)

    def host_step():
        if not sharded:
            binding.peagle_attn_partitioned_host(ctx, hprob, bparts, hQ, hK, hV, hdO, hO, hLSE, hdQ, hdK, hdV)
            return
        # sharded: host -> device copies, this rank's step, device -> host reads of its results
        for d, h in ((Q, hQ), (K, hK), (V, hV), (dO, hdO)):
            d.copy_(h, non_blocking=True)
        step()
        for h, d in ((hO, O), (hLSE, LSE), (hdQ, dQ), (hdK, dK), (hdV, dV)):
            h.copy_(d, non_blocking=True)
        torch.cuda.synchronize()

    host_step()
    barrier()
    e2e_steps = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        host_step()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, world, dev)
    nbytes = lambda *ts: int(sum(t.numel() * t.element_size() for t in ts))  # noqa: E731
    h2d = nbytes(hQ, hK, hV, hdO) + 2 * anchor.nbytes
    d2h = nbytes(hO, hLSE, hdQ, hdK, hdV)

    if rank == 0:
        peaks, peak_kind = load_peaks()
        peak = float(peaks["bf16_tflops"])
        if sharded:   # the timed launches are rank 0's: its partitions' share of the useful work
            share = sum(int((anchor[b:e].astype(np.int64) + 1 + depth[b:e]).sum())
                        for b, e in (parts[i]["q"] for i in sharding.deal_partitions(parts, world)[rank]))
            share /= float(allowed_pairs(w))
            f_fwd, f_bwd = f_fwd * share, f_bwd * share
        bwd_ms_launch = k_bwd_ms / max(n_bwd, 1)
        fwd_ms_launch = k_fwd_ms / max(n_fwd, 1)
        launches_per_step = max(n_bwd // args.steps, 1)
        achieved = (f_bwd / launches_per_step) / (bwd_ms_launch * 1e-3) / 1e12
        roofline = {
            "kernel": BWD_KERNEL[w.head_dim], "bound": "tensor",
            "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
            "traffic": ncu_traffic(w.name, BWD_KERNEL[w.head_dim]),
            "traffic_unit": "bytes per launch (ncu, DRAM)",
            "peak_source": f"{peak_kind} bf16_tflops (burst)",
            "ms_per_launch": bwd_ms_launch, "launches_timed": int(n_bwd),
            "fwd_kernel": {"achieved": (f_fwd / launches_per_step) / (fwd_ms_launch * 1e-3) / 1e12,
                           "ms_per_launch": fwd_ms_launch, "launches_timed": int(n_fwd)},
            "step_frac_of_peak": value / world / peak,
            "step_frac_of_sustained": value / world / float(peaks.get("bf16_tflops_sustained", peak)),
        }
        f_fwd, f_bwd = useful_flops(w)
        cpu, _, _ = oracle_sample(w, args.cpu_seconds) if world == 1 and args.cpu_seconds > 0 else (None, 0, 0)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": dict(config_dict(w, T, len(parts)), parallelism=args.parallelism),
            "clocks": clocks.summary(),
            "e2e": {"value": (1 if sharded else world) * (f_fwd + f_bwd) / e2e_s / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * e2e_s},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_rope(args, w):
    """The rotary prologue and its backward on the workload's token grid: an HBM-bound side line
    (one read and one write of every element per direction), timed with CUDA events."""
    import torch

    from paper_2602_01469_b200 import binding

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    cu, anchor, depth, _ = inputs.build_case(w, binding.peagle_assign_segments)
    T, Hq, Hkv, D = int(cu[-1]), w.n_q_heads, w.n_kv_heads, w.head_dim
    qkv, gQ, gK, gV = (t.to(dev) for t in inputs.make_fused_rows(T, Hq, Hkv, D, w.seed))
    d_anchor, d_depth = torch.from_numpy(anchor).to(dev), torch.from_numpy(depth).to(dev)
    Q, K, V, gx = torch.empty_like(gQ), torch.empty_like(gK), torch.empty_like(gV), torch.empty_like(qkv)
    stream = torch.cuda.current_stream()

    def step():
        binding.peagle_rope_qkv_fwd(ctx, qkv, d_anchor, d_depth, Hq, Hkv, D, 500000.0, Q, K, V, stream)
        binding.peagle_rope_qkv_bwd(ctx, gQ, gK, gV, d_anchor, d_depth, Hq, Hkv, D, 500000.0, gx, stream)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(0) as clocks:
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    # per direction: every element of the fused row read once and written once, 8 bytes of metadata
    bytes_step = 2 * (2 * qkv.numel() * 2 + 8 * T)
    peaks, src = load_peaks()
    peak = float(peaks["hbm_gbs"])
    gbs = bytes_step / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "rotary prologue fwd+bwd GB/s", "value": gbs, "unit": "GB/s", "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "total_tokens": T, "n_q_heads": Hq, "n_kv_heads": Hkv,
                   "head_dim": D, "l2": "tensors (%.2f GB) larger than L2, no flush" % (bytes_step / 2e9)},
        "clocks": clocks.summary(), "gpu_launches": 2 * args.steps,
        "roofline": {"kernel": "rope_kernel", "bound": "hbm", "achieved": gbs, "peak": peak,
                     "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                     "peak_source": "%s hbm_gbs" % src},
    }))


def run_gemm(args, w):
    """The three projection products of the layer slice at the workload's shape (rows = expanded
    tokens, d_model = args.d_model, fused width (Hq + 2 Hkv) D): a tensor-bound side line."""
    import torch

    from paper_2602_01469_b200 import binding

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    T, dm = w.total_tokens, args.d_model
    nqkv = (w.n_q_heads + 2 * w.n_kv_heads) * w.head_dim
    X, W, _ = inputs.make_layer_tensors(T, dm, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seed)
    X, W = X.to(dev), W.to(dev)
    Y = torch.empty(T, nqkv, dtype=torch.bfloat16, device=dev)
    dXa = torch.zeros(T, dm, dtype=torch.float32, device=dev)
    dWa = torch.zeros(nqkv, dm, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        binding.peagle_gemm_bf16(ctx, X, dm, 0, W, dm, 0, Y, nqkv, 0, T, nqkv, dm, stream)      # Y = X W^T
        binding.peagle_gemm_bf16(ctx, Y, nqkv, 0, W, dm, 1, dXa, dm, 1, T, dm, nqkv, stream)    # dX += Y W
        binding.peagle_gemm_bf16(ctx, Y, nqkv, 1, X, dm, 1, dWa, dm, 1, nqkv, dm, T, stream)    # dW += Y^T X

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert binding.peagle_poll_status(ctx) == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(0) as clocks:
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    flops = 3 * 2.0 * T * nqkv * dm
    peaks, src = load_peaks()
    peak = float(peaks["bf16_tflops"])
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "layer projection GEMMs (forward, input grad, weight grad) TFLOP/s", "value": tf,
        "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "rows": T, "d_model": dm, "fused_width": nqkv,
                   "l2": "operands (%.2f GB) larger than L2, no flush" % ((T * (dm + nqkv) * 2) / 1e9)},
        "clocks": clocks.summary(), "gpu_launches": 3 * args.steps,
        "roofline": {"kernel": "gemm_kernel", "bound": "tensor", "achieved": tf, "peak": peak,
                     "unit": UNIT, "frac": tf / peak, "traffic": None, "peak_source": "%s bf16_tflops (burst)" % src},
    }))
    ctx.close()


def run_layer(args, w):
    """The layer slice as Section 3.2 trains it: per segment the fused projection (its own rows and
    the depth-0 rows it sees, projected again), the rotary prologue, masked attention forward and
    backward, and the gradients back through the projection into dX / dW.  A side line: time per
    pass and the useful work of its attention and projection parts."""
    import torch

    from paper_2602_01469_b200 import binding

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
    T, dm = int(cu[-1]), args.d_model
    nqkv = (w.n_q_heads + 2 * w.n_kv_heads) * w.head_dim
    X, W, dO = (t.to(dev) for t in inputs.make_layer_tensors(T, dm, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seed))
    prob = binding.Problem(cu, torch.from_numpy(anchor).to(dev), torch.from_numpy(depth).to(dev), w.K,
                           w.n_q_heads, w.n_kv_heads, w.head_dim, w.scale)
    bparts = [binding.Partition(p["seq"], p["q"], p["k"]) for p in parts]
    O = torch.empty(T, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    LSE = torch.empty(w.n_q_heads, T, dtype=torch.float32, device=dev)
    dX = torch.empty(T, dm, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(nqkv, dm, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        binding.peagle_layer_partitioned(ctx, prob, bparts, X, W, 10000.0, dO, O, LSE, dX, dW, stream)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert binding.peagle_poll_status(ctx) == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(0) as clocks:
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    # rows projected per pass: every segment's own rows with all heads (forward, dX, dW: three
    # products over the fused width) and the earlier depth-0 rows it sees with the K / V heads only
    own = sum(p["q"][1] - p["q"][0] for p in parts)
    seen = sum(sum(e - b for b, e in p["k"]) for p in parts) - own
    kvw = 2 * w.n_kv_heads * w.head_dim
    f_gemm = 3 * 2.0 * dm * (own * nqkv + seen * kvw)
    f_fwd, f_bwd = useful_flops(w)
    peaks, src = load_peaks()
    peak = float(peaks["bf16_tflops"])
    tf = (f_gemm + f_fwd + f_bwd) / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "layer slice (projection, rotary, masked attention; forward+backward per segment) useful TFLOP/s",
        "value": tf, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "rows": T, "segments": len(parts), "d_model": dm, "fused_width": nqkv,
                   "rows_projected_again": int(seen), "attention_tflop": (f_fwd + f_bwd) / 1e12,
                   "projection_tflop": f_gemm / 1e12, "l2": "tensors larger than L2, no flush"},
        "clocks": clocks.summary(),
        "roofline": {"kernel": "whole pass", "bound": "tensor", "achieved": tf, "peak": peak, "unit": UNIT,
                     "frac": tf / peak, "traffic": None, "peak_source": "%s bf16_tflops (burst)" % src},
    }))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=inputs.HEADLINE, choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--op", default="attention", choices=["attention", "rope", "gemm", "layer"],
                    help="attention: the hot path (default); rope: the rotary prologue side line; "
                         "gemm: the layer slice's projection products side line; layer: the whole layer slice, "
                         "segment by segment")
    ap.add_argument("--d-model", type=int, default=2880, help="hidden width for --op gemm / layer")
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "partitions"],
                    help="with --gpus N > 1: N independent replicas of the workload (default), or one "
                         "workload whose query partitions are dealt out over the ranks (dK / dV "
                         "summed by an all-reduce); use a workload with several partitions")
    ap.add_argument("--cpu-seconds", type=float, default=15.0,
                    help="CPU time for the oracle baseline (0 = skip)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    w = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    elif args.op == "rope":
        run_rope(args, w)
    elif args.op == "gemm":
        run_gemm(args, w)
    elif args.op == "layer":
        run_layer(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
