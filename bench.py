#!/usr/bin/env python
"""Benchmark of the eOptShrinkQ hot path on B200.

One step = one pass of the whole hot path over a KV cache of synthetic spiked blocks
(paper_2605_02905_b200/synth.py): ``eosq_encode`` of every block, then ``eosq_scores`` of the query
heads against the compressed keys.  The headline value is encode throughput in GB/s of fp16 KV
read; the score pass and a decode of the whole cache are reported beside it.  Inputs are larger than
L2, so no cache flush is needed.

    python bench.py --gpus N --steps K --warmup W          # the CUDA library (N > 1: starts N ranks itself)
    python bench.py --workload ministral64k                # Ministral-8B-shaped cache, G = 16
    python bench.py --workload sweep                       # block lengths 256..4096 x code widths 1..4
    python bench.py --impl reference ...                   # the CPU oracle on a bounded sample

The default workload is the Llama-3.1-8B-shaped 32k-token cache (32 layers x 8 KV heads x {K,V},
T = 32768, n = 1024, d = 128, fp16; 16384 blocks, 4 GiB per GPU) at b = 2 with G = 4 queries per KV head.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "eOptShrinkQ encode GB/s of fp16 KV"
UNIT = "GB/s"
SEED = 1234
# double-precision multiply-add rate of the CUDA cores: 148 SMs x 64 lanes x 2 flop x 1.965 GHz (a product of
# nominal figures, not a measurement)
FP64_NOMINAL_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12

WORKLOADS = {
    # name: (generator name in synth, workload label, queries per KV head, layers, kv heads)
    "llama32k": ("llama_32k", "llama31_8b_T32768_n1024_d128", 4, 32, 8),
    "ministral64k": ("ministral_64k", "ministral_8b_T65536_n1024_d128", 16, 36, 8),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def recorded_traffic(n: int, d: int, bits: int):
    """DRAM bytes per block of each kernel from the committed ncu capture (profiles/traffic.json).  The
    record names the kernel sources it was taken on (a hash over csrc/) and the block shape; when either
    differs from what runs now the counters no longer describe it and {} is returned (traffic: null)."""
    import glob
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        rec = json.load(f)
    h = hashlib.sha256()
    for src in sorted(glob.glob(os.path.join(ROOT, "paper_2605_02905_b200", "csrc", "*"))):
        h.update(os.path.basename(src).encode())
        with open(src, "rb") as f:
            h.update(f.read())
    if h.hexdigest() != rec.get("sources_sha256"):
        return {"note": "the kernels have changed since the recorded ncu capture"}
    if (n, d, bits) != (1024, 128, 2):
        return {"note": "the recorded ncu capture is of n = 1024, d = 128, b = 2"}
    return rec


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


def oracle_sample(blocks_cpu, bits, seed):
    """Times the CPU oracle, as it stands, on the given blocks.  Returns (GB/s of fp16 in, seconds, threads, result)."""
    import oracle
    oracle.build()
    t0 = time.perf_counter()
    enc = oracle.encode_blocks(blocks_cpu.double().numpy(), bits, seed)
    dt = time.perf_counter() - t0
    nbytes = blocks_cpu.numel() * 2
    return nbytes / dt / 1e9, dt, oracle.num_threads(), enc


def run_reference(args):
    """The oracle on the machine's host cores, on a bounded sample of the same workload per step."""
    from paper_2605_02905_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    gen_name, label, _, _, _ = WORKLOADS["llama32k" if args.workload == "sweep" else args.workload]
    threads = oracle.num_threads()
    sample = max(32, 4 * threads)
    w = getattr(synth, gen_name)(device="cpu", max_blocks=sample)
    blocks = w.blocks
    for _ in range(min(args.warmup, 1)):
        oracle_sample(blocks[: max(1, sample // 4)], args.bits, SEED)
    times = []
    for _ in range(args.steps):
        _, dt, _, _ = oracle_sample(blocks, args.bits, SEED)
        times.append(dt)
    dt = sum(times) / len(times)
    value = blocks.numel() * 2 / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{label}_b{args.bits}", "sample": f"first {sample} blocks of the cache per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{sample} blocks of n=1024 d=128 per step, OpenMP over blocks"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def parity_on_sample(eosq, ctx, blocks, bits, enc, count, heads_for_scores, bph, G):
    """Parity counts of the library against the oracle's result `enc` on the first `count` blocks (outside any
    timed region; the oracle only checks).  Violations of a tolerance are reported, not raised."""
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import parity
    from paper_2605_02905_b200 import synth
    B, n, d = blocks.shape
    count = min(count, B)
    sub_dev = blocks[:count].contiguous()
    sub_cache = eosq.Cache.allocate(count, n, d, bits, diagnostics="staged")
    eosq.eosq_encode(ctx, sub_dev, bits, SEED, out=sub_cache)
    torch.cuda.synchronize()
    out = {"blocks": count, "violation": None}
    try:
        rep, _ = parity.compare_encode(sub_dev.cpu(), sub_cache, bits, SEED, blocks_idx=range(count), enc=enc)
        for k in ("near_threshold_blocks", "rank_mismatch", "codes", "staged_mismatch_in_band", "staged_mismatch_out_band",
                  "e2e_mismatch_in_band", "e2e_mismatch_out_band", "max_sigma_rel", "max_phi_rel", "max_lowrank_rel", "flagged"):
            out[k] = rep[k]
        dec = eosq.eosq_decode(ctx, sub_cache, SEED)
        out["max_decode_rel"] = parity.compare_decode(sub_cache, dec, bits, SEED, blocks_idx=range(min(count, 4)))
        if heads_for_scores > 0 and count >= bph:
            # keys of the first head only: blocks [0, bph) of the sample
            q = synth.queries(1, G, seed=9).cuda()
            s = eosq.eosq_scores(ctx, sub_cache, q, 1, bph, bph, SEED)
            torch.cuda.synchronize()
            out["max_score_rel"] = parity.compare_scores(sub_cache, q, s, 1, bph, bph, bits, SEED, 1.0 / math.sqrt(d),
                                                         pairs=[(0, 0), (0, bph - 1)])
    except AssertionError as e:
        out["violation"] = str(e)[:200]
    return out


def encode_roofline_ms(peaks, in_bytes, out_bytes, B, n, d):
    """The whole-encode roofline: the slower of all bytes at HBM peak and Gram + rotation flops at tensor peak."""
    t_hbm = (in_bytes + out_bytes) / (peaks["hbm_gbs"] * 1e9)
    t_tensor = B * 4.0 * n * d * d / (peaks["bf16_tflops_sustained"] * 1e12)
    return max(t_hbm, t_tensor) * 1e3, ("hbm" if t_hbm >= t_tensor else "tensor")


def run_sweep(args, eosq, ctx, peaks):
    """Block lengths 256 .. 4096 x code widths 1 .. 4 on the sweep shape (1 layer x 8 KV heads, T = 131072, four
    spikes at {5, 1.5, 1.05, 0.9} x the detection threshold): GB/s and roofline fraction per point."""
    import torch
    from paper_2605_02905_b200 import synth
    points = []
    for n in (256, 512, 1024, 2048, 4096):
        w = synth.sweep_point(n, device="cuda")
        blocks = w.blocks
        B, _, d = blocks.shape
        workspace = torch.empty(eosq.eosq_workspace_bytes(B, n, d), dtype=torch.uint8, device="cuda")
        for bits in (1, 2, 3, 4):
            cache = eosq.Cache.allocate(B, n, d, bits, diagnostics=False)
            for _ in range(max(args.warmup, 3)):
                eosq.eosq_encode(ctx, blocks, bits, SEED, out=cache, workspace=workspace)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(args.steps, 5)
            e0.record()
            for _ in range(reps):
                eosq.eosq_encode(ctx, blocks, bits, SEED, out=cache, workspace=workspace)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
            ranks = cache.rank.cpu()
            mean_rank = float(ranks.float().mean())
            in_bytes = B * n * d * 2
            out_bytes = B * (n * d * bits // 8 + n * 2 + mean_rank * (n + d) * 2 + 64)
            roof_ms, bound = encode_roofline_ms(peaks, in_bytes, out_bytes, B, n, d)
            hist = torch.bincount(ranks, minlength=4).tolist()
            points.append({"n": n, "bits": bits, "blocks": B, "ms": ms, "gbs_in": in_bytes / (ms * 1e-3) / 1e9,
                           "roofline_frac": roof_ms / ms, "bound": bound, "selected_rank_histogram": hist,
                           "planted": "5, 1.5, 1.05, 0.9 x threshold", "flagged": eosq.eosq_check_status(ctx, cache)})
            del cache
        del blocks, workspace, w
        torch.cuda.empty_cache()
    head = next(p for p in points if p["n"] == 1024 and p["bits"] == 2)
    line = {"metric": METRIC, "value": head["gbs_in"], "unit": UNIT, "n_gpus": 1, "steps": max(args.steps, 5), "warmup": max(args.warmup, 3),
            "ms_per_step": head["ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 x f16 -> f32 (tensor), f64 (spectral)", "data": "synthetic",
            "config": {"workload": "sweep_T131072_d128 (value: the n=1024, b=2 point)", "l2": "inputs (512 MiB per point) larger than L2, no flush"},
            "points": points}
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
        os.environ.setdefault("NCCL_DEBUG", "INFO")          # the communicator's rank count goes to the log
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lib_build.build()
    ctx = eosq.Context()
    peaks = measured_peaks()
    BITS = args.bits
    if args.workload == "sweep":
        if rank == 0:
            run_sweep(args, eosq, ctx, peaks)
        ctx.close()
        return
    gen_name, label, G_PER_HEAD, layers, kv_heads = WORKLOADS[args.workload]

    # The job's cache is `world` times the named cache, [stream][K|V][block]; a rank owns the blocks of its
    # (layer, head) streams (no data-path collective: blocks are compressed independently) and draws them itself.
    w = getattr(synth, gen_name)(device="cuda", seed=2 + rank, max_blocks=args.blocks)
    blocks = w.blocks
    B, n, d = blocks.shape
    bph = w.meta["blocks_per_stream"]
    num_heads = B // (2 * bph)            # (layer, kv head) streams that are complete
    streams_per_rank = layers * kv_heads
    owned = shard.block_range(world * streams_per_rank, bph, rank, world)
    if args.blocks is None:
        assert len(owned) == B, (len(owned), B)
    cache = eosq.Cache.allocate(B, n, d, BITS, diagnostics=False)
    workspace = torch.empty(eosq.eosq_workspace_bytes(B, n, d), dtype=torch.uint8, device="cuda")
    q = synth.queries(max(num_heads, 1), G_PER_HEAD, seed=9).cuda()
    scores = torch.empty((max(num_heads, 1), G_PER_HEAD, bph * n), dtype=torch.float32, device="cuda")

    def step():
        eosq.eosq_encode(ctx, blocks, BITS, SEED, out=cache, workspace=workspace)
        if num_heads > 0:
            eosq.eosq_scores(ctx, cache, q, num_heads, bph, 2 * bph, SEED, out=scores)

    ENC_STAGES = ("gram", "tridiag_a", "tridiag_b", "tridiag_c", "eigvals", "spectral", "quant", "redo")
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    # Untimed: two more steps with every launch bracketed by events give the per-stage breakdown and
    # name the dominant kernel.  The events cost a few per cent of an encode, so the timed region below
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
    decode = None
    e2e = None
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

        ranks = cache.rank.float()
        mean_rank = float(ranks.mean())
        out_bytes_per_block = n * d * BITS // 8 + n * 2 + mean_rank * (n + d) * 2 + 64

        # ---- decode (Algorithm 1 DeQuant + low-rank part), timed on its own: it is not part of a step ----
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

    in_bytes = B * n * d * 2
    enc_gbs = world * in_bytes / (enc_ms * 1e-3) / 1e9
    flagged = eosq.eosq_check_status(ctx, cache)
    k_blocks = num_heads * bph
    # bytes the score pass has to read: codes + norms + kept factor rows of the key blocks
    key_idx = (torch.arange(num_heads, device="cuda")[:, None] * 2 * bph + torch.arange(bph, device="cuda")[None, :]).reshape(-1)
    key_rank_sum = float(cache.rank[key_idx].sum()) if k_blocks else 0.0
    score_bytes = k_blocks * (n * d * BITS // 8 + n * 2) + key_rank_sum * (n + d) * 2 + k_blocks * G_PER_HEAD * n * 4
    sc_gbs = world * score_bytes / (sc_ms * 1e-3) / 1e9 if k_blocks else 0.0
    rank_hist = torch.bincount(cache.rank.clamp(min=0), minlength=12).tolist()
    planted_hist = None
    if hasattr(w, "planted_rank"):
        import numpy as np
        planted_hist = np.bincount(np.asarray(w.planted_rank), minlength=1).tolist()

    # ---- rooflines --------------------------------------------------------------------------------
    # The whole encode against the roofline of the task: the slower of all its bytes at the HBM peak and the
    # Gram + rotation flops at the tensor peak.  The double-precision spectral stages are credited nothing.
    roof_ms, roof_bound = encode_roofline_ms(peaks, in_bytes, B * out_bytes_per_block, B, n, d)
    algo_bytes = in_bytes + B * out_bytes_per_block
    traffic_tab = recorded_traffic(n, d, args.bits)
    roofline = {"kernel": "eosq_encode (all stages of one pass)", "bound": roof_bound,
                "achieved": (algo_bytes / (enc_ms * 1e-3) / 1e9) if roof_bound == "hbm" else (B * 4.0 * n * d * d / (enc_ms * 1e-3) / 1e12),
                "peak": peaks["hbm_gbs"] if roof_bound == "hbm" else peaks["bf16_tflops_sustained"],
                "unit": "GB/s" if roof_bound == "hbm" else "TFLOP/s", "frac": roof_ms / enc_ms,
                "t_roof_ms": roof_ms, "peak_source": peaks["source"],
                "traffic": (sum(traffic_tab["per_block_bytes"].get(k, 0.0) for k in ENC_STAGES) * B
                            if traffic_tab.get("per_block_bytes") else None),
                "traffic_note": traffic_tab.get("note", "no ncu capture of the current kernels is recorded"),
                "stage_ms_per_step": {k: round(v, 4) for k, v in breakdown_ms.items()},
                "stage_note": "from two untimed steps with every launch bracketed by events"}
    # the kernel with the largest share, against the bound that holds for it
    algo = {
        "gram": ("tensor", 2.0 * n * d * d / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s", peaks["source"]),
        # Householder tridiagonalisation: 4/3 m^3 flops for order m; three kernels take d -> d/2 -> d/4 -> 0
        "tridiag_a": ("alu", (4.0 / 3.0) * (d ** 3 - (d // 2) ** 3) / 1e12, FP64_NOMINAL_TFLOPS, "TFLOP/s", "nominal (SMs x lanes x clock)"),
        "tridiag_b": ("alu", (4.0 / 3.0) * ((d // 2) ** 3 - (d // 4) ** 3) / 1e12, FP64_NOMINAL_TFLOPS, "TFLOP/s", "nominal (SMs x lanes x clock)"),
        "tridiag_c": ("alu", (4.0 / 3.0) * (d // 4) ** 3 / 1e12, FP64_NOMINAL_TFLOPS, "TFLOP/s", "nominal (SMs x lanes x clock)"),
        "eigvals": ("alu", 32 * 14 * d * 6.0 / 1e12, FP64_NOMINAL_TFLOPS, "TFLOP/s", "nominal (SMs x lanes x clock)"),
        "spectral": ("alu", (4.0 * d * d * max(mean_rank, 1.0)) / 1e12, FP64_NOMINAL_TFLOPS, "TFLOP/s", "nominal (SMs x lanes x clock)"),
        "quant": ("hbm", (n * d * 2 + out_bytes_per_block) / 1e9, peaks["hbm_gbs"], "GB/s", peaks["source"]),
    }
    bound, units, peak, unit, peak_source = algo[dominant]
    dom_launches = stage[dominant][1]
    dom_ms_per_launch = stage[dominant][0] / max(dom_launches, 1)
    blocks_per_launch = B * args.steps / max(dom_launches, 1)
    achieved = units * blocks_per_launch / (dom_ms_per_launch * 1e-3)
    dom_traffic = traffic_tab.get("per_block_bytes", {}).get(dominant)
    dominant_kernel = {"kernel": dominant, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                       "frac": achieved / peak, "peak_source": peak_source,
                       "traffic": (dom_traffic * blocks_per_launch if dom_traffic else None),
                       "ms_per_launch": dom_ms_per_launch, "launches": dom_launches}
    t_sc_roof = score_bytes / (peaks["hbm_gbs"] * 1e9)
    scores_roofline = {"bound": "hbm", "achieved": sc_gbs / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": (t_sc_roof * 1e3 / sc_ms) if k_blocks else None}

    # ---- the oracle beside it: timed on a bounded sample, and the same result checks the library's ----
    cpu_baseline = None
    parity = None
    if rank == 0 and not args.no_cpu_baseline:
        import oracle
        threads = oracle.num_threads()
        sample = min(B, max(64, 16 * threads))   # a few seconds of wall time on all cores: tens of core-seconds
        sub = blocks[:sample].cpu()
        gbs, dt, threads, enc = oracle_sample(sub, BITS, SEED)
        cpu_baseline = {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": f"first {sample} blocks (n={n}, d={d}) of the same cache, {dt:.1f} s wall on {threads} threads, OpenMP over blocks"}
        parity = parity_on_sample(eosq, ctx, blocks, BITS, enc, min(sample, 2 * bph), num_heads, bph, G_PER_HEAD)

    if rank == 0:
        line = {
            "metric": METRIC, "value": enc_gbs, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 x f16 -> f32 (tensor), f64 (spectral)", "data": "synthetic",
            "config": {"workload": f"{label}_b{BITS}", "blocks_per_gpu": B, "n": n, "d": d, "bits": BITS, "G": G_PER_HEAD,
                       "global_blocks": world * B, "block_range_rank0": [owned.start, owned.stop],
                       "l2": f"inputs ({in_bytes / 2 ** 30:.1f} GiB per GPU) larger than L2, no flush", "mean_rank": mean_rank,
                       "selected_rank_histogram": rank_hist, "planted_rank_histogram": planted_hist,
                       "flagged_blocks": flagged},
            "encode": {"ms": enc_ms, "gbs_in": enc_gbs},
            "scores": {"ms": sc_ms, "gbs_compressed": sc_gbs, "bytes": score_bytes, "roofline": scores_roofline},
            "decode": decode,
            "roofline": roofline, "dominant_kernel": dominant_kernel, "parity": parity,
            "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks.summary(),
        }
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def free_port():
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="eosq", choices=["eosq", "reference"])
    ap.add_argument("--workload", default="llama32k", choices=["llama32k", "ministral64k", "sweep"])
    ap.add_argument("--blocks", type=int, default=None, help="encode only the first BLOCKS blocks (profiling captures)")
    ap.add_argument("--e2e-blocks", type=int, default=None, help="blocks per end-to-end host-buffer call (default: the whole cache)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--bits", type=int, default=2, choices=[1, 2, 3, 4],
                    help="code width b (the headline configuration is b = 2; b = 3 is its second variant)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly with --gpus N: start the N ranks (one per GPU) and let rank 0 print the line
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        os.execv(sys.executable, cmd)
    run_library(args)


if __name__ == "__main__":
    main()
