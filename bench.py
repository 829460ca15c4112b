#!/usr/bin/env python
"""Benchmark of the QK4PV8 hot path on B200.

A step is one pass of the whole path over one batch of the Llama-3.1-8B-shaped causal
prefill workload (batch 1, 32 q heads / 8 kv heads, head_dim 128, 16384 tokens): stage 1
(means, scales, NVFP4 quantization of Q and K, Delta_S, FP8 V) followed by the prefill
attention kernel.  `value` is attention TFLOPS (4 N^2 d H_q / 2 per step) over the whole
step with inputs resident in HBM; `e2e` is the same with pinned-host inputs copied in and
the BF16 output copied back inside the timed region.  The paged decode workload is timed
separately in the same run and reported under "decode" in GB/s of KV-cache bytes.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run) every rank runs the same workload on its own
batch element: the path shards by (batch, head) with no data-path collective, so scaling is
weak and `value` is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "QK4PV8 prefill TFLOPS @16K-128K; decode KV GB/s vs HBM peak"
KERNELS_PER_STEP = 5  # column statistics (Q and K in one launch), K quantize + Delta_S, Q quantize, V quantize, prefill
# Nominal dense tensor rates relative to BF16: FP4 4x, FP8 2x.  Per (query, key) pair the path does
# 2d FP4 FLOP and 2d FP8 FLOP, so F attention FLOPs take (F/2)/(4P) + (F/2)/(2P) = 3F/(8P): the
# mixed-precision bound in attention FLOP/s is 8/3 of the BF16 peak P.
MIXED_OVER_BF16 = 8.0 / 3.0
NOMINAL_MIXED_TFLOPS = 6000.0   # the same bound from the nominal dense peaks (9 PF/s FP4, 4.5 PF/s FP8)
NOMINAL_HBM_GBS = 8000.0        # nominal HBM3e bandwidth the decode figure is also stated against
KV_BYTES_PER_TOKEN_HEAD = 64 + 8 + 128 + 2 * 4  # K codes, K scales, V, Delta_S for a 4-head GQA group


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ts, line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            mx = float(parts[2])
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(float(parts[1]))
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if not sm:
            sm = [float(l.split(",")[1]) for _, l in self.lines[-3:] if len(l.split(",")) >= 9]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


_DIST_DEVICE = "cuda"   # where the rank-to-rank reductions live: "cuda" under NCCL, "cpu" under gloo


def dist_setup(n, backend="nccl"):
    """One process per GPU, rendezvous from the torchrun environment.  `backend="gloo"` runs the same
    rank plumbing on CPU (used by the multi-rank tests; the data path itself has no collective)."""
    global _DIST_DEVICE
    if n <= 1:
        return 0, 1, 0
    import torch.distributed as dist
    rank, world, local = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"]), int(os.environ.get("LOCAL_RANK", 0))
    if backend == "nccl":
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        _DIST_DEVICE = "cuda"
    else:
        dist.init_process_group(backend)
        _DIST_DEVICE = "cpu"
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if _DIST_DEVICE == "cuda" and torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x: float, world) -> float:
    if world <= 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=_DIST_DEVICE)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, flops_per_rank: float, ms_per_step: float) -> float:
    """Weak scaling: every rank runs its own batch element; the job's TFLOPS is the work of all ranks over
    the slowest rank's time."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def rank_seed(base_seed: int, rank: int) -> int:
    """Batch element of a rank: rank r takes element r of a global batch (distinct seeds, same shape)."""
    return base_seed + 100 * rank


# ------------------------------------------------------------------------------------------
def cpu_oracle_sample(w, steps: int, rows_per_head: int):
    """The oracle, as it stands, on a bounded sample of the prefill workload: stage 1 on the full tensors, then
    `rows_per_head` evenly spaced query rows of every head against all their keys; the two parts are timed
    separately so that the attention rate does not depend on how many rows share one stage-1 pass.
    Returns (attention FLOPs of the sample, [(stage-1 seconds, attention seconds)] per step, description)."""
    from oracle import mpfa_oracle as orc
    import numpy as np
    q, k, v = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    stride = max(1, w.N_q // rows_per_head)
    idx = np.arange(stride - 1, w.N_q, stride, dtype=np.int32)
    rows = np.stack([np.zeros(len(idx) * w.H_q, np.int32), np.repeat(np.arange(w.H_q, dtype=np.int32), len(idx)),
                     np.tile(idx, w.H_q)], axis=1)
    pairs = float((idx.astype(np.int64) + 1 + (w.N_kv - w.N_q)).clip(0, w.N_kv).sum() * w.H_q)
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        z = orc.stage1(q, k, v)
        t1 = time.perf_counter()
        orc.prefill_rows(z, rows, w.softmax_scale, w.causal)
        times.append((t1 - t0, time.perf_counter() - t1))
    return pairs * 4 * 128, times, f"{len(rows)} (head, query row) pairs (every {stride}th row of each head) against all " \
                                  f"their keys; stage 1 on the full tensors timed separately"


def cpu_baseline_record(flops, times, sample, cores):
    """value = attention FLOPs of the sample / attention seconds (stage 1 excluded, as the kernel figures are)."""
    s1 = sum(t[0] for t in times) / len(times)
    att = sum(t[1] for t in times) / len(times)
    return {"value": flops / att / 1e12, "unit": "TFLOPS", "cores": cores, "kind": "oracle", "sample": sample,
            "attention_seconds": att, "seconds_per_query_key_pair": att / (flops / 512.0), "stage1_seconds_full_tensors": s1}


def cpu_oracle_config1_full():
    """Config 1 (256 tokens, one head, non-causal) through the oracle in full: stage 1 + attention of all rows."""
    from oracle import mpfa_oracle as orc
    from paper_2609_33135_b200 import workloads as wl
    w = wl.config1_tiny()
    q, k, v = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    orc.prefill_rows(orc.stage1(q, k, v), rows, w.softmax_scale, w.causal)   # first call loads the library
    reps = 20
    t0 = time.perf_counter()
    for _ in range(reps):
        z = orc.stage1(q, k, v)
        orc.prefill_rows(z, rows, w.softmax_scale, w.causal)
    sec = (time.perf_counter() - t0) / reps
    return {"workload": w.name, "seconds_stage1_plus_attention": sec, "tflops": w.flops / sec / 1e12,
            "sample": "the whole config: all 256 rows against all 256 keys, stage 1 included"}


def cpu_oracle_decode_sample(n_requests: int = 2):
    """Config 5 through the oracle on a bounded sample: the first `n_requests` requests, all 32 heads each; the cache
    (stage 1 of each request's K/V with frozen statistics) is built outside the timed part, as on the GPU."""
    from oracle import mpfa_oracle as orc
    from paper_2609_33135_b200 import workloads as wl
    import numpy as np
    w = wl.config5_decode()
    tokens, sec = 0, 0.0
    for b in range(n_requests):
        k, v = w.kv_for_request(b, "cpu")
        kb, vb = orc.bf16_bits(k), orc.bf16_bits(v)
        z = orc.stage1(orc.bf16_bits(w.q_sample[b:b + 1].contiguous()), kb, vb)
        zq = orc.stage1(orc.bf16_bits(w.q_new[b:b + 1].contiguous()), kb, vb, frozen=z)
        L = int(w.seq_lens[b])
        t0 = time.perf_counter()
        orc.decode(zq.q_codes[:, :, 0], zq.q_sf[:, :, 0], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0, w.softmax_scale,
                   np.array([L], np.int32))
        sec += time.perf_counter() - t0
        tokens += L
    bytes_ = float(tokens) * w.H_kv * KV_BYTES_PER_TOKEN_HEAD
    return {"workload": w.name, "value": bytes_ / sec / 1e9, "unit": "GB/s", "seconds": sec, "tokens": tokens,
            "sample": f"requests 0..{n_requests - 1} of 32 (all 32 heads each), decode attention only; the cache is built before the timed part"}


def run_reference(args, rank):
    """Reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from paper_2609_33135_b200 import workloads as wl
    w = wl.config2_llama()
    cores = os.cpu_count() or 1
    flops, times, sample = cpu_oracle_sample(w, args.warmup + args.steps, rows_per_head=args.ref_rows_per_head)
    times = times[args.warmup:]
    rec = cpu_baseline_record(flops, times, sample, cores)
    ms = 1e3 * rec["attention_seconds"]
    val = rec["value"]
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "nvfp4/fp8 emulated in f32", "data": "synthetic",
        "config": {"workload": w.name, "B_per_gpu": 1, "H_q": 32, "H_kv": 8, "head_dim": 128, "N": w.N_q, "causal": True},
        "cpu_baseline": rec,
        "e2e": {"value": val, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------
def bench_decode(steps, warmup, peaks, small):
    """Paged decode (config 5): KV GB/s = sum_r L_r * H_kv * 208 B / time."""
    from paper_2609_33135_b200 import decode_cache, workloads as wl
    lo, hi = (2048, 8192) if small else (16384, 131072)
    w = wl.config5_decode(32, lo, hi)
    st = decode_cache.build_cache(w, kv_device="cuda", want_f32=False)
    for _ in range(warmup):
        decode_cache.decode_step(st)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record()
        decode_cache.decode_step(st)
        b.record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    bytes_ = float(w.total_tokens) * w.H_kv * KV_BYTES_PER_TOKEN_HEAD
    mean = sum(ms) / len(ms)
    gbs = bytes_ / (mean * 1e-3) / 1e9
    # the serving step: write one new token per request into the cache (frozen statistics), then decode
    from paper_2609_33135_b200 import binding as B_
    g = torch.Generator(device="cuda").manual_seed(1007)
    k_new = torch.randn(w.B, 1, w.H_kv, 128, generator=g, device="cuda").to(torch.bfloat16)
    v_new = torch.randn(w.B, 1, w.H_kv, 128, generator=g, device="cuda").to(torch.bfloat16)
    pos = (st.seq_lens - 1).to(torch.int32)   # the slot of each request's last token (always has a page)
    evs2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs2:
        a.record()
        B_.mpfa_append_kv_paged(k_new, v_new, w.H_q, B_.MPFA_SMOOTH, st.stats, st.v_scale, st.kv, st.page_table, pos)
        decode_cache.decode_step(st)
        b.record()
    torch.cuda.synchronize()
    ms_append = sum(a.elapsed_time(b) for a, b in evs2) / len(evs2)
    return {"workload": w.name, "value": gbs, "unit": "GB/s", "ms_mean": mean, "ms_min": min(ms),
            "ms_append_plus_decode": ms_append,
            "kv_bytes": bytes_, "tokens": w.total_tokens, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
            "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "gpu_launches_per_step": 2,
            "l2": "3.9 GB of cache per step vs 126 MB L2", "status": int(st.status.item())}


def bench_prefill_paged(w, k, v, s1, out_ref, steps, warmup):
    """The same prefill with K, V, scales and Delta_S read from a paged low-bit cache (64-token pages in a
    shuffled pool) instead of contiguous tensors; the result must equal the contiguous kernel's bit for bit."""
    from paper_2609_33135_b200 import binding as B_
    dev = k.device
    n_pages = (w.N_kv + 63) // 64
    kv = B_.PagedKV.empty(n_pages, w.H_q, w.H_kv, with_delta=True, device=dev)
    g = torch.Generator().manual_seed(1006)
    table = torch.randperm(n_pages, generator=g).to(torch.int32).to(dev).view(1, -1).contiguous()
    B_.mpfa_quantize_kv_paged(k[0], v[0], 0, w.H_q, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, s1.stats.request(0), 1.0, kv,
                              table[0], None)
    seq = torch.tensor([w.N_kv], dtype=torch.int32, device=dev)
    out = torch.empty_like(out_ref)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    run = lambda: B_.mpfa_prefill_paged(s1.q, kv, table, seq, s1.stats, 1.0, w.softmax_scale, out, None, status)
    for _ in range(warmup):
        run()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record()
        run()
        b.record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    mean = sum(ms) / len(ms)
    return {"workload": w.name + "_from_pages", "value": w.flops / (mean * 1e-3) / 1e12, "unit": "TFLOPS", "ms_mean": mean,
            "ms_min": min(ms), "pages": n_pages, "page_order": "shuffled", "gpu_launches_per_step": 1,
            "equals_contiguous_bitwise": bool(torch.equal(out.view(torch.uint16), out_ref.view(torch.uint16))),
            "status": int(status.item())}


def bench_prefill_sustained(binding, s1, w, out, status, local, seconds=2.0):
    """The attention kernel back to back for about two seconds (clocks settle under the power cap)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    binding.prefill(s1, w.causal, w.softmax_scale, out=out, status=status)
    e1.record()
    torch.cuda.synchronize()
    n = max(10, int(seconds * 1e3 / e0.elapsed_time(e1)))
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.2)
    t0 = time.time()
    e0.record()
    for _ in range(n):
        binding.prefill(s1, w.causal, w.softmax_scale, out=out, status=status)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    ms = e0.elapsed_time(e1) / n
    return {"value": w.flops / (ms * 1e-3) / 1e12, "unit": "TFLOPS", "ms": ms, "launches": n,
            "seconds": e0.elapsed_time(e1) * 1e-3, "clocks": clocks, "status": int(status.item())}


def bench_compensation_overhead(binding, s1, w, reps=5):
    """Cost of the compensation term by placement (Sections 5.2 and 7.4): the attention kernel with the rank-one
    seed MMA, without Delta_S, and with Delta_S added element-wise by the softmax threads; same quantized
    inputs, runs interleaved."""
    dev = s1.q.codes.device
    out = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    modes = {"mma": (s1.delta, 0), "none": (None, 0), "elementwise": (s1.delta, binding.MPFA_VARIANT_COMP_ELEMENTWISE)}
    t = {m: [] for m in modes}
    for i in range(reps + 1):
        for m, (delta, variant) in modes.items():
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            binding.mpfa_prefill_variant(s1.q, s1.k, s1.v_fp8, delta, s1.stats, s1.v_scale, w.causal, w.softmax_scale,
                                         variant, out, None, status)
            b.record()
            torch.cuda.synchronize()
            if i >= 1:
                t[m].append(a.elapsed_time(b))
    ms = {m: sum(v) / len(v) for m, v in t.items()}
    return {"ms_with": ms["mma"], "ms_without": ms["none"], "overhead_frac": ms["mma"] / ms["none"] - 1.0,
            "ms_elementwise": ms["elementwise"], "elementwise_overhead_frac": ms["elementwise"] / ms["none"] - 1.0,
            "status": int(status.item())}


def bench_mma_peaks(binding, dev):
    """Tensor-core rates of this GPU for the three MMA kinds of the path (M = 128, N = 128, operands resident in
    shared / tensor memory, one CTA per SM, a few milliseconds each, best of three): the measured counterpart of
    the nominal 4x / 2x ratios.  The mixed bound takes equal FP4 and FP8 FLOPs per (query, key) pair."""
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = {}
    for name, kind, iters in (("bf16_ss", 0, 20000), ("e4m3_ts", 2, 20000), ("nvfp4_ss", 3, 10000)):
        best = 0.0
        for _ in range(3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            flops = binding.mpfa_bench_mma_peak(kind, 128, iters, status)
            b.record()
            torch.cuda.synchronize()
            best = max(best, flops / (a.elapsed_time(b) * 1e-3) / 1e12)
        out[name] = best
    out["mixed_fp4_fp8"] = 1.0 / (0.5 / out["nvfp4_ss"] + 0.5 / out["e4m3_ts"])
    out["unit"] = "TFLOP/s"
    out["status"] = int(status.item())
    out["how"] = "mpfa_bench_mma_peak: back-to-back tcgen05.mma, M=128 N=128, CUDA events, best of 3 bursts"
    return out


def time_calls(fn, steps, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    return sum(ms) / len(ms), min(ms)


def stage1_bytes(w):
    """Algorithmic HBM bytes of stage 1: two passes over Q and K (statistics, quantize; Delta_S comes out of the K
    quantize pass), packed codes + scales written (0.5625 B per element), Delta_S written, V read and written."""
    nq, nk = w.q.numel(), w.k.numel()
    return (2 * 2 + 0.5625) * (nq + nk) + 2.0 * w.B * w.N_kv * w.H_q + 3 * w.v.numel()


def bench_prefill_config(binding, wl, name, seed, N, H_q, peaks, mma, local, with_compensation, with_variants=False):
    """One more prefill length of the metric (configs 3 and 4), inputs drawn on the device: attention kernel alone,
    the whole step with stage 1, stage-1 GB/s, fractions of the bounds, clocks sampled during the timed steps."""
    dev = torch.device("cuda", local)
    w = wl.prefill_workload(name, seed, 1, N, H_q, 8, True, device=str(dev))
    s1 = binding.stage1(w.q, w.k, w.v)
    ws = binding.quantize_workspace(1, H_q, 8, dev)
    out = torch.empty(1, N, H_q, 128, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    steps = 5 if N <= 65536 else 3
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.2)
    t0 = time.time()
    k_ms, k_min = time_calls(lambda: binding.prefill(s1, True, w.softmax_scale, out=out, status=status), steps, 3)
    q_ms, _ = time_calls(lambda: binding.stage1(w.q, w.k, w.v, workspace=ws, out=s1), steps, 2)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    tf = w.flops / (k_ms * 1e-3) / 1e12
    rec = {"workload": w.name, "H_q": H_q, "H_kv": 8, "N": N, "kernel_ms": k_ms, "kernel_ms_min": k_min,
           "prefill_kernel_tflops": tf, "step_tflops": w.flops / ((k_ms + q_ms) * 1e-3) / 1e12,
           "frac_of_mixed_bound_from_bf16_peak": tf / (peaks["bf16"] * MIXED_OVER_BF16),
           "frac_of_mixed_bound_from_measured_mma": tf / mma["mixed_fp4_fp8"] if mma else None,
           "frac_of_nominal_mixed_bound": tf / NOMINAL_MIXED_TFLOPS,
           "stage1_ms": q_ms, "stage1_gbs": stage1_bytes(w) / (q_ms * 1e-3) / 1e9,
           "stage1_frac_of_hbm_peak": stage1_bytes(w) / (q_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
           "clocks": clocks, "data": "synthetic, drawn on the device", "status": int(status.item())}
    if with_compensation:
        rec["compensation_mma"] = bench_compensation_overhead(binding, s1, w, reps=2)
    if with_variants:
        # Section 3.1's precision assignments on the same quantized Q and K: NVFP4 + FP8 (the product path) against
        # NVFP4 + BF16 (P in BF16, V unquantized, second MMA kind::f16), attention kernel alone
        vt = binding.mpfa_pack_v_bf16(w.v)
        run = lambda: binding.mpfa_prefill_variant(s1.q, s1.k, vt, s1.delta, s1.stats, 1.0, True, w.softmax_scale,
                                                   binding.MPFA_VARIANT_PV_BF16, out, None, status)
        b_ms, b_min = time_calls(run, steps, 2)
        del vt
        # NVFP4 + NVFP4: P quantized per row and 16 keys on the softmax path, handed over through shared memory with its
        # block scales, V as the token-axis FP4 operand, second MMA block-scaled FP4
        g = float(w.v.abs().max().float().item()) / (6.0 * 448.0)
        v4 = binding.mpfa_quantize_v_fp4(w.v, g)
        run4 = lambda: binding.mpfa_prefill_variant(s1.q, s1.k, v4, s1.delta, s1.stats, g, True, w.softmax_scale,
                                                    binding.MPFA_VARIANT_PV_FP4, out, None, status)
        f_ms, f_min = time_calls(run4, steps, 2)
        rec["precision_variants"] = {"nvfp4_qk_fp8_pv_ms": k_ms, "nvfp4_qk_bf16_pv_ms": b_ms,
                                     "nvfp4_qk_bf16_pv_tflops": w.flops / (b_ms * 1e-3) / 1e12,
                                     "fp8_pv_speedup_over_bf16_pv": b_ms / k_ms,
                                     "nvfp4_qk_nvfp4_pv_ms": f_ms,
                                     "nvfp4_qk_nvfp4_pv_tflops": w.flops / (f_ms * 1e-3) / 1e12,
                                     "fp8_pv_speedup_over_nvfp4_pv": f_ms / k_ms, "status": int(status.item())}
        del v4
    return rec


def bench_two_tile_arrangement(binding, s1, w, out, status, steps):
    """The same attention launch in the two-query-tile arrangement (Section 5.1's two stages), for the comparison."""
    binding.mpfa_set_prefill_arrangement(1)
    try:
        ms, mn = time_calls(lambda: binding.prefill(s1, w.causal, w.softmax_scale, out=out, status=status), steps, 3)
    finally:
        binding.mpfa_set_prefill_arrangement(0)
    return {"ms": ms, "ms_min": mn, "value": w.flops / (ms * 1e-3) / 1e12, "unit": "TFLOPS", "status": int(status.item())}


def run_ours(args, rank, world, local):
    from paper_2609_33135_b200 import binding, workloads as wl
    binding.lib()  # fail loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the QK4PV8 path has no CPU fallback")
    peaks = load_peaks()
    dev = torch.device("cuda", local)
    N = args.seq_len
    if args.shape == "qwen":   # config 3: 40 q heads / 8 kv heads
        w = wl.prefill_workload(f"cfg3_qwen14b_causal_{N}", rank_seed(1003, rank), 1, N, 40, 8, True)
    else:
        w = wl.config2_llama(N, seed=rank_seed(1002, rank))   # rank r: batch element r
    hq, hk, hv = w.q.pin_memory(), w.k.pin_memory(), w.v.pin_memory()
    q, k, v = hq.to(dev), hk.to(dev), hv.to(dev)
    s1 = binding.stage1(q, k, v)           # allocates outputs once; steps reuse them
    ws = binding.quantize_workspace(w.B, w.H_q, w.H_kv, dev)
    out = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    host_out = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(kernel_events=None):
        binding.stage1(q, k, v, workspace=ws, out=s1)
        if kernel_events is not None:
            kernel_events[0].record()
        binding.prefill(s1, w.causal, w.softmax_scale, out=out, status=status)
        if kernel_events is not None:
            kernel_events[1].record()

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()

    # ---- timed region: K steps, device-timed, barrier + synchronize on both sides
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    kev = [(ev(), ev()) for _ in range(args.steps)]
    barrier(world)
    e0, e1 = ev(), ev()
    t_wall0 = time.time()
    e0.record()
    for i in range(args.steps):
        step(kev[i])
    e1.record()
    barrier(world)
    t_wall1 = time.time()
    total_ms = max_over_ranks(e0.elapsed_time(e1), world)
    clocks = sampler.stop(t_wall0, t_wall1)
    ms_step = total_ms / args.steps
    kernel_ms = sum(a.elapsed_time(b) for a, b in kev) / args.steps
    assert int(status.item()) == 0, f"device status {int(status.item())}"

    # ---- end to end: pinned host inputs in, BF16 output back, every step.  Three streams and two buffer
    # sets, so that the upload of step i+1 and the download of step i-1 run while step i computes (the copy
    # engines work in both directions at once); every step still uploads its own Q, K, V and downloads its
    # own output.
    class Slot:
        pass
    slots = []
    for _ in range(2):
        sl = Slot()
        sl.q, sl.k, sl.v = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        sl.s1 = binding.stage1(q, k, v)
        sl.ws = binding.quantize_workspace(w.B, w.H_q, w.H_kv, dev)
        sl.out = torch.empty_like(out)
        sl.host_out = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
        sl.status = torch.zeros(1, dtype=torch.int32, device=dev)
        sl.in_ready, sl.in_free, sl.done, sl.out_free = ev(), ev(), ev(), ev()
        slots.append(sl)
    torch.cuda.synchronize()
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def run_e2e(n):
        for i in range(n):
            sl = slots[i % 2]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(sl.in_free)      # the kernels of step i-2 have read these inputs
                sl.q.copy_(hq, non_blocking=True)
                sl.k.copy_(hk, non_blocking=True)
                sl.v.copy_(hv, non_blocking=True)
                sl.in_ready.record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(sl.in_ready)
                if i >= 2:
                    s_cmp.wait_event(sl.out_free)    # the download of step i-2 has read this output buffer
                binding.stage1(sl.q, sl.k, sl.v, workspace=sl.ws, out=sl.s1)
                binding.prefill(sl.s1, w.causal, w.softmax_scale, out=sl.out, status=sl.status)
                sl.in_free.record(s_cmp)
                sl.done.record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(sl.done)
                sl.host_out.copy_(sl.out, non_blocking=True)
                sl.out_free.record(s_out)

    run_e2e(2)
    torch.cuda.synchronize()
    barrier(world)
    e0, e1 = ev(), ev()
    e0.record(s_in)
    run_e2e(args.steps)
    e1.record(s_out)
    torch.cuda.synchronize()
    barrier(world)
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world) / args.steps
    _ = float(slots[(args.steps - 1) % 2].host_out[0, 0, 0, 0])  # the host reads the result
    assert all(int(sl.status.item()) == 0 for sl in slots)
    assert torch.equal(slots[0].host_out, out.cpu()), "end-to-end result differs from the device-resident run"

    flops = w.flops
    value = whole_job_value(world, flops, ms_step)
    mma = None
    if rank == 0:
        try:
            mma = bench_mma_peaks(binding, dev)
        except Exception as e:
            mma = None
    long_run = total_ms > 2000.0
    bf16_peak = peaks["bf16_sustained"] if long_run else peaks["bf16"]
    peak = bf16_peak * MIXED_OVER_BF16
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    result = {
        "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "nvfp4 (QK^T) + fp8 e4m3 (PV), f32 accumulate", "data": "synthetic",
        "config": {"workload": w.name, "B_per_gpu": 1, "H_q": w.H_q, "H_kv": w.H_kv, "head_dim": 128, "N": N,
                   "causal": True, "parallelism": f"dp{world} (independent batch elements, no collective)",
                   "l2": f"inputs_exceed_l2 (Q+K+V {(q.numel() + k.numel() + v.numel()) * 2 / 1e6:.0f} MB, "
                         f"output {out.numel() * 2 / 1e6:.0f} MB per step vs 126 MB L2)",
                   "step": "quantize_qk + quantize_v + prefill"},
        "clocks": clocks,
        "e2e": {"value": whole_job_value(world, flops, e2e_ms), "unit": "TFLOPS", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": (q.numel() + k.numel() + v.numel()) * 2, "d2h_bytes_per_step": out.numel() * 2},
        "gpu_launches": KERNELS_PER_STEP * args.steps,
        "roofline": {"kernel": "prefill_kernel", "bound": "tensor", "achieved": achieved, "peak": peak,
                     "unit": "TFLOP/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC_BYTES.get((w.H_q, N), {}).get("bytes"),
                     "traffic_source": NCU_TRAFFIC_BYTES.get((w.H_q, N), {}).get("source"),
                     "peak_measured": mma["mixed_fp4_fp8"] if mma else None,
                     "frac_of_peak_measured": achieved / mma["mixed_fp4_fp8"] if mma else None,
                     "peak_nominal": NOMINAL_MIXED_TFLOPS, "frac_of_peak_nominal": achieved / NOMINAL_MIXED_TFLOPS,
                     "mma_rates_measured": mma,
                     "kernel_ms": kernel_ms,
                     "peak_note": f"{peaks['source']} bf16 {'sustained' if long_run else 'burst'} {bf16_peak} TF/s x 8/3 "
                                  "(nominal fp4 4x / fp8 2x of bf16; equal FP4 and FP8 FLOPs per pair)",
                     "exp_ceiling_tflops_at_sampled_clock":
                         (148 * 16 * clocks["sm_mhz"] * 1e6 * 512 / 1e12) if clocks.get("sm_mhz") else None},
        "prefill_kernel_only": {"value": achieved, "unit": "TFLOPS", "ms": kernel_ms,
                                "note": "attention kernel alone, quantization excluded (as the paper times it)"},
        "quantize_ms": ms_step - kernel_ms,
    }
    # stage 1 against HBM (algorithmic bytes: see stage1_bytes)
    q_bytes = stage1_bytes(w)
    result["quantize"] = {"ms": ms_step - kernel_ms, "algorithmic_bytes": q_bytes,
                          "value": q_bytes / ((ms_step - kernel_ms) * 1e-3) / 1e9, "unit": "GB/s",
                          "frac_of_hbm_peak": q_bytes / ((ms_step - kernel_ms) * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    if rank == 0:
        if args.compensation or not args.no_decode:
            try:
                result["compensation_mma"] = bench_compensation_overhead(binding, s1, w)
            except Exception as e:
                result["compensation_mma"] = {"error": repr(e)}
        if not args.no_decode:
            try:
                result["prefill_sustained"] = bench_prefill_sustained(binding, s1, w, out, status, local)
            except Exception as e:
                result["prefill_sustained"] = {"error": repr(e)}
            try:
                result["decode"] = bench_decode(max(3, args.steps // 2), 3, peaks, args.small_decode)
            except Exception as e:  # decode is a secondary line; never lose the main one
                result["decode"] = {"error": repr(e)}
            try:
                result["prefill_paged"] = bench_prefill_paged(w, k, v, s1, out, max(3, args.steps // 2), 3)
            except Exception as e:
                result["prefill_paged"] = {"error": repr(e)}
        try:
            result["prefill_two_tile_arrangement"] = bench_two_tile_arrangement(binding, s1, w, out, status, max(3, args.steps // 2))
        except Exception as e:
            result["prefill_two_tile_arrangement"] = {"error": repr(e)}
        if world == 1 and not args.no_configs:
            # the other lengths of the metric (configs 3 and 4), after the main buffers are released
            del slots
            torch.cuda.empty_cache()
            by_cfg = {}
            for key, name, seed, N2, hq2, comp in (("cfg3_32k", "cfg3_qwen14b_causal_32768", 1003, 32768, 40, False),
                                                   ("cfg3_64k", "cfg3_qwen14b_causal_65536", 1003, 65536, 40, False),
                                                   ("cfg4_128k", "cfg4_long_causal_131072", 1004, 131072, 32, True)):
                try:
                    by_cfg[key] = bench_prefill_config(binding, wl, name, seed, N2, hq2, peaks, mma, local, comp, with_variants=(N2 == 65536))
                except Exception as e:
                    by_cfg[key] = {"error": repr(e)}
                torch.cuda.empty_cache()
            result["prefill_by_config"] = by_cfg
        if "decode" in result and "value" in result["decode"]:
            result["decode"]["frac_of_nominal_hbm"] = result["decode"]["value"] / NOMINAL_HBM_GBS
            result["decode"]["nominal_hbm_gbs"] = NOMINAL_HBM_GBS
        if world == 1 and not args.no_cpu:
            cores = os.cpu_count() or 1
            fl, times, sample = cpu_oracle_sample(w, 1, rows_per_head=args.cpu_rows_per_head)
            result["cpu_baseline"] = cpu_baseline_record(fl, times, sample, cores)
            if not args.no_configs:
                try:
                    result["cpu_baseline"]["config1_full"] = cpu_oracle_config1_full()
                    result["cpu_baseline"]["config5_decode"] = cpu_oracle_decode_sample()
                except Exception as e:
                    result["cpu_baseline"]["other_configs_error"] = repr(e)
        print(json.dumps(result))


# DRAM bytes per prefill launch from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum), keyed by
# (q heads, sequence length); lengths without a capture report no traffic figure.
NCU_TRAFFIC_BYTES = {
    (32, 16384): {"bytes": 143500000, "source": "profiles/prefill_kernel_llama_shape.md section 1 (65.4 MB read + 78.1 MB written per launch)"},
    (32, 131072): {"bytes": 44430000000, "source": "profiles/prefill_kernel_128k_and_paged_source.md section 1 (43.4 GB read + 1.03 GB written)"},
}


def _spawned_rank(rank, n, port, argv):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.argv = argv
    main()


def spawn_ranks(n, fn=_spawned_rank):
    """`python bench.py --gpus N` without a launcher: start the N ranks here (one process per GPU, rendezvous on
    127.0.0.1), the same as `python -m torch.distributed.run --nproc-per-node N bench.py --gpus N ...`."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    mp.spawn(fn, args=(n, port, list(sys.argv)), nprocs=n, join=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seq-len", type=int, default=16384)
    ap.add_argument("--shape", default="llama", choices=["llama", "qwen"], help="32:8 (configs 2, 4) or 40:8 heads (config 3)")
    ap.add_argument("--no-decode", action="store_true",
                    help="main line only: skip decode, prefill from pages and the compensation-placement timing")
    ap.add_argument("--compensation", action="store_true", help="time the compensation placements even with --no-decode")
    ap.add_argument("--small-decode", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the 32K / 64K / 128K lines (prefill_by_config)")
    ap.add_argument("--cpu-rows-per-head", type=int, default=8192)
    ap.add_argument("--ref-rows-per-head", type=int, default=512,
                    help="reference arm: query rows per head in each step's sample")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args, int(os.environ.get("RANK", 0)))
        return
    if args.gpus > 1 and "RANK" not in os.environ:
        spawn_ranks(args.gpus)
        return
    rank, world, local = dist_setup(args.gpus)
    try:
        run_ours(args, rank, world, local)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
