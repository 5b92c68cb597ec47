#!/usr/bin/env python
"""Benchmark of the eOptShrinkQ hot path on B200.

One step = one pass of the whole hot path over the Llama-3.1-8B-shaped 32k-token cache
(32 layers x 8 KV heads x {K,V}, T = 32768, n = 1024, d = 128, fp16; 16384 blocks, 4 GiB):
``eosq_encode`` at b = 2 of every block, then ``eosq_scores`` of 32 query heads (G = 4 per KV
head) against the compressed keys.  The headline value is encode throughput in GB/s of fp16 KV
read; the score pass is reported beside it.  Inputs are seeded synthetic spiked blocks
(paper_2605_02905_b200/synth.py) and are larger than L2, so no cache flush is needed.

    python bench.py --gpus N --steps K --warmup W          # the CUDA library
    python bench.py --impl reference ...                   # the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "eOptShrinkQ encode GB/s of fp16 KV"
UNIT = "GB/s"
WORKLOAD = "llama31_8b_T32768_n1024_d128_b2"
SEED = 1234
BITS = 2
G_PER_HEAD = 4
FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12   # 148 SMs x 64 FP64 FMA lanes x 2 flop x 1.965 GHz
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def oracle_sample_throughput(blocks_cpu, bits, seed):
    """Times the CPU oracle, as it stands, on the given blocks.  Returns (GB/s of fp16 in, seconds, threads)."""
    import oracle
    oracle.build()
    t0 = time.perf_counter()
    oracle.encode_blocks(blocks_cpu.double().numpy(), bits, seed)
    dt = time.perf_counter() - t0
    nbytes = blocks_cpu.numel() * 2
    return nbytes / dt / 1e9, dt, oracle.num_threads()


def run_reference(args):
    """The oracle on the machine's host cores, on a bounded sample of the same workload per step."""
    import torch
    from paper_2605_02905_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    threads = oracle.num_threads()
    sample = max(32, 4 * threads)
    w = synth.llama_32k(device="cpu", max_blocks=sample)
    blocks = w.blocks
    for _ in range(min(args.warmup, 1)):
        oracle_sample_throughput(blocks[: max(1, sample // 4)], BITS, SEED)
    times = []
    for _ in range(args.steps):
        gbs, dt, _ = oracle_sample_throughput(blocks, BITS, SEED)
        times.append(dt)
    dt = sum(times) / len(times)
    value = blocks.numel() * 2 / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": f"first {sample} blocks of the cache per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{sample} blocks of n=1024 d=128 per step, OpenMP over blocks"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def run_library(args):
    import torch
    import torch.distributed as dist
    import paper_2605_02905_b200 as eosq
    from paper_2605_02905_b200 import build as lib_build, shard, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lib_build.build()
    ctx = eosq.Context()
    peaks = measured_peaks()

    # every rank owns one whole cache of the same shape (independent blocks: no collective)
    layers, heads = 32, 8
    w = synth.llama_32k(device="cuda", seed=2 + rank, max_blocks=args.blocks)
    blocks = w.blocks
    B, n, d = blocks.shape
    bph = w.meta["blocks_per_stream"]
    num_heads = B // (2 * bph)            # (layer, kv head) streams that are complete
    cache = eosq.Cache.allocate(B, n, d, BITS, diagnostics=False)
    workspace = torch.empty(eosq.eosq_workspace_bytes(B, n, d), dtype=torch.uint8, device="cuda")
    q = synth.queries(max(num_heads, 1), G_PER_HEAD, seed=9).cuda()
    scores = torch.empty((max(num_heads, 1), G_PER_HEAD, bph * n), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        eosq.eosq_encode(ctx, blocks, BITS, SEED, out=cache, workspace=workspace)
        if num_heads > 0:
            eosq.eosq_scores(ctx, cache, q, num_heads, bph, 2 * bph, SEED, out=scores)

    ENC_STAGES = ("gram", "tridiag_a", "tridiag_b", "tridiag_c", "eigvals", "spectral", "quant", "redo")
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    # Untimed: two more steps with every launch bracketed by events give the per-stage breakdown and
    # name the dominant kernel.  The events cost about 9 % of an encode, so the timed region below
    # brackets the launches of that one kernel only.
    ctx.profile_enable(True)
    for _ in range(2):
        step()
    breakdown = ctx.profile_read()
    breakdown_ms = {k: v[0] / 2 for k, v in breakdown.items() if v[1]}
    dominant = max((k for k in ENC_STAGES if k != "redo"), key=lambda k: breakdown[k][0])
    ctx.profile_select([dominant])
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()

    enc_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    sc_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = ctx.launch_count
    with ClockSampler(local_rank) as clocks:
        t_all0 = torch.cuda.Event(enable_timing=True)
        t_all1 = torch.cuda.Event(enable_timing=True)
        t_all0.record()
        for i in range(args.steps):
            enc_ev[i][0].record()
            eosq.eosq_encode(ctx, blocks, BITS, SEED, out=cache, workspace=workspace)
            enc_ev[i][1].record()
            sc_ev[i][0].record()
            if num_heads > 0:
                eosq.eosq_scores(ctx, cache, q, num_heads, bph, 2 * bph, SEED, out=scores)
            sc_ev[i][1].record()
        t_all1.record()
        torch.cuda.synchronize()
    launches = ctx.launch_count - launches0
    stage = ctx.profile_read()
    ctx.profile_enable(False)
    total_ms = t_all0.elapsed_time(t_all1)
    enc_ms = sum(a.elapsed_time(b) for a, b in enc_ev) / args.steps
    sc_ms = sum(a.elapsed_time(b) for a, b in sc_ev) / args.steps
    total_ms, enc_ms, sc_ms = shard.max_over_ranks([total_ms, enc_ms, sc_ms], device="cuda")
    if world > 1:
        dist.barrier()
    in_bytes = B * n * d * 2
    enc_gbs = world * in_bytes / (enc_ms * 1e-3) / 1e9
    flagged = eosq.eosq_check_status(ctx, cache)
    ranks = cache.rank.float()
    mean_rank = float(ranks.mean())
    k_blocks = num_heads * bph
    # bytes the score pass has to read: codes + norms + kept factor rows of the key blocks
    key_idx = (torch.arange(num_heads, device="cuda")[:, None] * 2 * bph + torch.arange(bph, device="cuda")[None, :]).reshape(-1)
    key_rank_sum = float(cache.rank[key_idx].sum()) if k_blocks else 0.0
    score_bytes = k_blocks * (n * d * BITS // 8 + n * 2) + key_rank_sum * (n + d) * 2 + k_blocks * G_PER_HEAD * n * 4
    sc_gbs = world * score_bytes / (sc_ms * 1e-3) / 1e9 if k_blocks else 0.0

    # ---- roofline of the dominant kernel (timed live with events inside the library) -------------
    out_bytes_per_block = n * d * BITS // 8 + n * 2 + mean_rank * (n + d) * 2 + 64
    algo = {
        # stage: (bound, algorithmic units per block, peak, unit)
        "gram": ("tensor", 2.0 * n * d * d / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"),
        # Householder tridiagonalisation: 4/3 m^3 flops for order m; three kernels take d -> 3d/4 -> d/2 -> 0
        "tridiag_a": ("alu", (4.0 / 3.0) * (d ** 3 - (3 * d // 4) ** 3) / 1e12, FP64_PEAK_TFLOPS, "TFLOP/s"),
        "tridiag_b": ("alu", (4.0 / 3.0) * ((3 * d // 4) ** 3 - (d // 2) ** 3) / 1e12, FP64_PEAK_TFLOPS, "TFLOP/s"),
        "tridiag_c": ("alu", (4.0 / 3.0) * (d // 2) ** 3 / 1e12, FP64_PEAK_TFLOPS, "TFLOP/s"),
        "eigvals": ("alu", 32 * d * d * 6.0 / 1e12, FP64_PEAK_TFLOPS, "TFLOP/s"),   # ~32 Sturm counts x d steps x 3 fp64 ops per eigenvalue
        "spectral": ("alu", (4.0 * d * d * max(mean_rank, 1.0)) / 1e12, FP64_PEAK_TFLOPS, "TFLOP/s"),
        "quant": ("hbm", (n * d * 2 + out_bytes_per_block) / 1e9, peaks["hbm_gbs"], "GB/s"),
    }
    bound, units, peak, unit = algo[dominant]
    dom_launches = stage[dominant][1]
    dom_ms_per_launch = stage[dominant][0] / max(dom_launches, 1)
    blocks_per_launch = B * args.steps / max(dom_launches, 1)
    achieved = units * blocks_per_launch / (dom_ms_per_launch * 1e-3)
    # DRAM bytes per block from the committed ncu section capture (profiles/sections_per_kernel_*.txt),
    # scaled to the blocks of one launch; None for kernels changed since that capture
    ncu_traffic_per_block = {"gram": 187.4e6 / 592, "tridiag_a": 86.4e6 / 592, "tridiag_b": 44.4e6 / 592, "tridiag_c": 20.1e6 / 592,
                             "eigvals": 1.2e6 / 592, "spectral": 81.6e6 / 592, "quant": 177.9e6 / 592}
    traffic = ncu_traffic_per_block.get(dominant)
    roofline = {"kernel": dominant, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "traffic": (traffic * blocks_per_launch if traffic else None),
                "traffic_note": "dram__bytes (read+write) of one 592-block launch under ncu, scaled by blocks per launch",
                "peak_source": peaks["source"],
                "ms_per_launch": dom_ms_per_launch, "launches": dom_launches}
    # whole encode against the task's roofline: slower of bytes at HBM peak and Gram+rotation flops at tensor peak
    t_hbm = (in_bytes + B * out_bytes_per_block) / (peaks["hbm_gbs"] * 1e9)
    t_tensor = B * 4.0 * n * d * d / (peaks["bf16_tflops_sustained"] * 1e12)
    encode_roofline = {"t_roof_ms": max(t_hbm, t_tensor) * 1e3, "frac": max(t_hbm, t_tensor) * 1e3 / enc_ms,
                       "stage_ms_per_step": {k: round(v, 4) for k, v in breakdown_ms.items()},
                       "stage_note": "from two untimed steps with every launch bracketed by events (that costs about 9 %)"}
    t_sc_roof = score_bytes / (peaks["hbm_gbs"] * 1e9)
    scores_roofline = {"bound": "hbm", "achieved": sc_gbs / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": (t_sc_roof * 1e3 / sc_ms) if k_blocks else None}

    # ---- decode (Algorithm 1 DeQuant + low-rank part), timed on its own: it is not part of a step ----
    decode = None
    if not args.no_decode:
        dec_out = torch.empty((B, n, d), dtype=torch.float16, device="cuda")
        for _ in range(2):
            eosq.eosq_decode(ctx, cache, SEED, out=dec_out)
        torch.cuda.synchronize()
        reps = max(2, min(args.steps, 5))
        d0 = torch.cuda.Event(enable_timing=True)
        d1 = torch.cuda.Event(enable_timing=True)
        d0.record()
        for _ in range(reps):
            eosq.eosq_decode(ctx, cache, SEED, out=dec_out)
        d1.record()
        torch.cuda.synchronize()
        dec_ms = shard.max_over_ranks([d0.elapsed_time(d1) / reps], device="cuda")[0]
        dec_bytes = B * n * d * 2 + B * out_bytes_per_block   # fp16 out + compressed in
        decode = {"ms": dec_ms, "gbs": world * dec_bytes / (dec_ms * 1e-3) / 1e9, "bytes": dec_bytes,
                  "roofline": {"bound": "hbm", "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": dec_bytes / (dec_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}}
        del dec_out

    # ---- end to end through the host-buffer entry point ------------------------------------------
    e2e = None
    cpu_baseline = None
    if not args.no_e2e:
        eb = B if args.e2e_blocks is None else min(B, args.e2e_blocks)
        host_in = torch.empty((eb, n, d), dtype=torch.float16).pin_memory()
        host_in.copy_(blocks[:eb])
        host_out = eosq.Cache.allocate(eb, n, d, BITS, pinned=True, diagnostics=False)
        arena = torch.empty(eosq.eosq_encode_host_arena_bytes(eb, n, d, BITS, eosq.EOSQ_F16), dtype=torch.uint8, device="cuda")
        for _ in range(2):
            eosq.eosq_encode_host(ctx, host_in, BITS, SEED, host_out, arena)
        torch.cuda.synchronize()
        reps = max(2, min(args.steps, 5))
        t0 = time.perf_counter()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            eosq.eosq_encode_host(ctx, host_in, BITS, SEED, host_out, arena)
        e1.record()
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / reps
        e2e_ms = shard.max_over_ranks([e2e_ms], device="cuda")[0]
        h2d = eb * n * d * 2
        d2h = sum(getattr(host_out, k).numel() * getattr(host_out, k).element_size()
                  for k in ("codes", "norms", "rank", "sigma", "phi", "P", "V", "status"))
        e2e = {"value": world * h2d / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "blocks": eb, "ms": e2e_ms}
        del host_in, host_out, arena

    if rank == 0 and not args.no_cpu_baseline:
        import oracle
        threads = oracle.num_threads()
        sample = min(B, max(64, 16 * threads))   # a few seconds of wall time on all cores: tens of core-seconds
        sub = blocks[:sample].cpu()
        gbs, dt, threads = oracle_sample_throughput(sub, BITS, SEED)
        cpu_baseline = {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": f"first {sample} blocks (n=1024, d=128) of the same cache, {dt:.1f} s wall on {threads} threads, OpenMP over blocks"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": enc_gbs, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 x f16 -> f32 (tensor), f64 (spectral)", "data": "synthetic",
            "config": {"workload": WORKLOAD, "blocks_per_gpu": B, "n": n, "d": d, "bits": BITS, "G": G_PER_HEAD,
                       "l2": "inputs (4 GiB per GPU) larger than L2, no flush", "mean_rank": mean_rank,
                       "flagged_blocks": flagged},
            "encode": {"ms": enc_ms, "gbs_in": enc_gbs},
            "scores": {"ms": sc_ms, "gbs_compressed": sc_gbs, "bytes": score_bytes, "roofline": scores_roofline},
            "decode": decode,
            "roofline": roofline, "encode_roofline": encode_roofline,
            "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks.summary(),
        }
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    global BITS, WORKLOAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="eosq", choices=["eosq", "reference"])
    ap.add_argument("--blocks", type=int, default=None, help="encode only the first BLOCKS blocks (profiling captures)")
    ap.add_argument("--e2e-blocks", type=int, default=None, help="blocks per end-to-end host-buffer call (default: the whole cache)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--bits", type=int, default=BITS, choices=[1, 2, 3, 4],
                    help="code width b (the headline configuration is b = 2; b = 3 is its second variant)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    BITS = args.bits
    WORKLOAD = f"llama31_8b_T32768_n1024_d128_b{BITS}"
    if args.impl == "reference":
        run_reference(args)
    else:
        run_library(args)


if __name__ == "__main__":
    main()
