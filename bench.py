#!/usr/bin/env python
"""Benchmark of the MoSKA decode-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

One step = one decode step of one attention layer over one batch of synthetic requests:
route -> group -> shared attention || unique attention -> merge, through the C ABI.  Prints ONE
JSON line (rank 0).

Without --config the headline is the largest workload (index 4: serving mix, batch 1024, 8
re-routed decode steps) and the same line carries a `per_config` record for workloads 1, 2 and 3,
each timed on blocks of its own.  The timed region is R blocks of K steps (R chosen so that the
blocks add up to at least half a second of device time); `ms_per_step` is the median block / K.

With N > 1 (torchrun) ONE batch is split by KV head: every rank holds Hkv / N heads of the shared
store and of every request's private store and computes those heads' outputs, no data-path
collective (strong scaling).  `--shard replicas` gives every rank its own batch and its own copy
of the shared store instead (weak scaling); `--shard disaggregated` runs rank 0 as the Shared-KV
rank and the others as Unique-KV ranks with one point-to-point exchange each way per step.

`--impl reference` times the fp64 CPU oracle on the host cores instead (bounded sample per step).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2511_06010_b200 import distributed as DD
from paper_2511_06010_b200 import workloads as W

METRIC = "decode_queries_per_s_per_layer"
UNIT = "queries/s"
L2_BYTES = 126e6
HEADLINE_CONFIG = 4            # the largest single-GPU workload
PER_CONFIG = (1, 2, 3)         # further workloads recorded on the same line

# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu captures (summaries under
# profiles/).  Keyed by (kernel, workload name); "ratio" entries are traffic / algorithmic bytes
# measured on a smaller launch of the same kernel and scaled by the units a full launch processes
# (the traffic of these streaming kernels grows in proportion to the tokens they read).
NCU_TRAFFIC_BYTES = {
    # profiles/unique_staged_kernel_cfg1.md: 1.0744 GB read + 7.3 MB written
    ("unique_staged_kernel", "cfg1_llama8b_b64"): 1.0817e9,
    # profiles/unique_fp8_kernel_cfg1.md: 554.3 MB read + 6.7 MB written
    ("unique_fp8_kernel", "cfg1_llama8b_b64"): 5.610e8,
    # profiles/shared_tc_kernel_cfg3.md: 568.2 MB read + 130.6 MB written
    ("shared_tc_kernel", "cfg3_dense_b512"): 6.987e8,
}
# DRAM bytes the per-request GEMV baseline really reads per launch (ncu), where captured
GEMV_DRAM_BYTES = {
    # profiles/gemv_baseline_dram_cfg1.md: 725.7 MB read + 7.3 MB written (algorithmic: 1073.7 MB)
    "cfg1_llama8b_b64": 7.33e8,
}
NCU_TRAFFIC_RATIO = {
    # profiles/unique_staged_kernel_cfg4_b64.md: 4.7050 GB measured for 4.7009 GB algorithmic on a
    # 64-request cut of workload 4 (the full workload is too large to capture with counters)
    "unique_staged_kernel": (4.7050e9 / 4.7009e9, "scaled by bytes from the capture of a 64-request cut of workload 4"),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while the timed region runs.

    Reads through NVML in a thread every 5 ms (read-only queries); falls back to an `nvidia-smi`
    loop when the NVML binding is missing."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []          # (sm_mhz, set of reason names)
        self.sm_max = None
        self.proc = None
        self.thread = None
        self.stop_flag = False
        self.source = None

    def _nvml_loop(self, nv, handle):
        names = {
            "hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown
            if hasattr(nv, "nvmlClocksEventReasonHwSlowdown") else nv.nvmlClocksThrottleReasonHwSlowdown,
            "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown
            if hasattr(nv, "nvmlClocksEventReasonHwThermalSlowdown") else nv.nvmlClocksThrottleReasonHwThermalSlowdown,
            "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown
            if hasattr(nv, "nvmlClocksEventReasonSwThermalSlowdown") else nv.nvmlClocksThrottleReasonSwThermalSlowdown,
            "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap
            if hasattr(nv, "nvmlClocksEventReasonSwPowerCap") else nv.nvmlClocksThrottleReasonSwPowerCap,
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)
                bits = get_reasons(handle)
                self.rows.append((float(mhz), {n for n, b in names.items() if bits & b}))
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        try:
            import pynvml as nv

            nv.nvmlInit()
            # NVML enumerates physical GPUs; honour CUDA_VISIBLE_DEVICES when it lists indices
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            ids = [v for v in vis.split(",") if v.strip().isdigit()]
            phys = int(ids[self.index]) if self.index < len(ids) else self.index
            handle = nv.nvmlDeviceGetHandleByIndex(phys)
            self.sm_max = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            self.source = "nvml"
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.source = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.source = "nvidia-smi"
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read_smi(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.proc.stdout:
            r = [x.strip() for x in line.split(",")]
            try:
                self.sm_max = float(r[1])
                self.rows.append((float(r[0]),
                                  {n for n, v in zip(names, r[3:7]) if v.lower().startswith("active")}))
            except Exception:
                continue

    def stop(self):
        if self.source is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source available"]}
        if self.source == "nvml":
            self.stop_flag = True
            self.thread.join(timeout=1)
        else:
            time.sleep(0.05)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        sm = [r[0] for r in self.rows]
        reasons = set().union(*[r[1] for r in self.rows]) if self.rows else set()
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_mhz_min": min(sm) if sm else None, "sm_max_mhz": self.sm_max,
                "samples": len(sm), "source": self.source, "reasons": sorted(reasons)}


def algorithmic_work(w: W.Workload, lens: np.ndarray, n_unique_splits: int, shared_slots: int,
                     touched_segments: int):
    """Bytes and flops the method must move/compute per step (no padding, no re-reads)."""
    rows = w.B * w.Hq
    P = w.B * w.Hkv * w.k
    unique_bytes = int(lens.sum()) * w.Hkv * 4 * w.D + rows * w.D * 2 + rows * n_unique_splits * (w.D + 1) * 4
    shared_flops = P * w.G * w.L * 4 * w.D
    shared_bytes = touched_segments * 4 * w.D * w.L + rows * w.D * 2 + rows * shared_slots * (w.D + 1) * 4
    gemv_bytes = P * 4 * w.D * w.L + rows * w.D * 2 + rows * shared_slots * (w.D + 1) * 4
    return dict(unique_bytes=unique_bytes, shared_flops=shared_flops, shared_bytes=shared_bytes,
                gemv_bytes=gemv_bytes)


def time_events(fn, iters: int, flush=None):
    """Average milliseconds of fn() on the current stream, CUDA events, optional L2 flush between."""
    total = 0.0
    for _ in range(iters):
        if flush is not None:
            flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        total += a.elapsed_time(b)
    return total / iters


def cpu_oracle_step(w, sh_host, un_host, q_host, kv_len, summ_ref, sample):
    """One oracle decode step (route + group + attention by definition) for the sampled requests."""
    from oracle import oracle as O

    qs = q_host[sample]
    scale = 1.0 / float(np.sqrt(w.D))
    if w.dense:
        topk = np.tile(np.arange(w.C, dtype=np.int32), (len(sample), w.Hkv, 1))
    else:
        topk, _ = O.route(qs, summ_ref, w.k)
        O.group_by_chunk(topk, w.C, fast=True)
    out, _ = O.attend_direct(qs, sh_host[0], sh_host[1], un_host[0], un_host[1],
                             un_host[2][sample], kv_len[sample], topk, scale)
    return out


def run_reference(args, w):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload."""
    rank, _, world = DD.env_world()
    if rank != 0:
        return
    from oracle import oracle as O

    O.build()
    n_sample = min(w.B, args.ref_sample)
    ws = W.scaled(w, B=n_sample)
    sh = W.make_shared_store(ws, "cpu")
    un = W.make_unique_store(ws, "cpu")
    q = W.make_queries(ws, sh, 0, "cpu")
    summ = None if w.dense else O.chunk_summaries(sh.k_shared)
    sample = np.arange(n_sample)
    kv_len = un.kv_len.numpy()
    host = ((sh.k_shared, sh.v_shared), (un.k_unique, un.v_unique, un.kv_start.numpy()))
    for _ in range(args.warmup):
        cpu_oracle_step(ws, host[0], host[1], q, kv_len, summ, sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        cpu_oracle_step(ws, host[0], host[1], q, kv_len, summ, sample)
    dt = (time.perf_counter() - t0) / args.steps
    value = n_sample / dt
    sample_txt = f"first {n_sample} of {w.B} requests per step, all heads, full context per request"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "batch": w.B, "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                         "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def timed_blocks(run_block, min_total_ms: float, dev, max_blocks: int = 200, min_blocks: int = 3):
    """Runs run_block() -> milliseconds (device-timed, this rank) repeatedly: the first block fixes
    the number of blocks R (same on every rank: derived from the slowest rank's first block) so
    that the blocks add up to min_total_ms; returns the per-block maxima over ranks."""
    first = DD.max_over_ranks(run_block(), dev)
    n = int(min(max_blocks, max(min_blocks, math.ceil(min_total_ms / max(first, 1e-3)))))
    blocks = [first]
    for _ in range(n - 1):
        blocks.append(DD.max_over_ranks(run_block(), dev))
    return blocks


def cpu_baseline(w, sh, un, q0, kv_len0, n_sample: int, seconds: float):
    """The oracle as it stands on the host cores: a bounded sample of the workload's requests
    (all heads, full context), repeated for about `seconds`."""
    from oracle import oracle as O

    O.build()
    n_s = min(w.B, n_sample)
    sample = np.arange(n_s)
    qh = q0.cpu()
    lens_s = kv_len0.cpu().numpy()
    end = int((un.kv_start[n_s - 1] + un.capacity[n_s - 1]).item())
    un_host = (un.k_unique[:end].cpu(), un.v_unique[:end].cpu(), un.kv_start.cpu().numpy())
    sh_host = (sh.k_shared.cpu(), sh.v_shared.cpu())
    summ = None if w.dense else O.chunk_summaries(sh_host[0])
    t0 = time.perf_counter()
    reps = 0
    while True:
        cpu_oracle_step(w, sh_host, un_host, qh, lens_s, summ, sample)
        reps += 1
        if time.perf_counter() - t0 > seconds or reps >= 500:
            break
    dt = (time.perf_counter() - t0) / reps
    return {"value": n_s / dt, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": f"first {n_s} of {w.B} requests (all heads, full context), {reps} repeats, "
                      f"{dt * reps:.1f} s"}


def measure(args, w_full, rank, world, dev, headline: bool):
    """Everything measured on one workload; returns the record (rank 0) or None."""
    from paper_2511_06010_b200 import binding as M
    from paper_2511_06010_b200.engine import MoskaLayer

    local_rank = dev.index
    # ---- what this rank holds
    if world > 1 and args.shard == "kv_head":
        if w_full.Hkv % world != 0:
            raise SystemExit(f"{w_full.name}: {w_full.Hkv} KV heads do not split over {world} ranks "
                             "(use --shard replicas)")
        w = W.kv_head_shard(w_full, rank, world)
        per_gpu = f"KV heads [{rank * w.Hkv}, {(rank + 1) * w.Hkv}) of one batch: 1/{world} of the shared and private stores"
        units_this_rank = w.B / world      # every request is served by all ranks together
        scaling = "strong"
    elif world > 1:
        w = W.scaled(w_full, seed=w_full.seed + 7919 * rank)
        per_gpu = "own request batch, own copy of the shared store"
        units_this_rank = w.B
        scaling = "weak"
    else:
        w = w_full
        per_gpu = "single GPU"
        units_this_rank = w.B
        scaling = "weak"
    free, _ = torch.cuda.mem_get_info()
    lens0 = W.unique_lengths(w)
    need = (2 * w.Hkv * w.C * w.L * w.D + 2 * int((lens0 + w.steps).sum()) * w.Hkv * w.D) * 2
    if need * 1.15 > free:
        raise SystemExit(f"workload {w.name} needs {need/1e9:.1f} GB, only {free/1e9:.1f} GB free")
    sh = W.make_shared_store(w, dev)
    un = W.make_unique_store(w, dev)
    # --q-len T: every request brings T query tokens (speculative decoding); the batch rows are
    # requests x T, token i of a request sees its context up to T - 1 - i tokens from the end
    T = max(1, args.q_len)
    if T > 1:
        if w.D != 128 or T * w.G > (8 if args.unique_kv == "fp8" else 16):
            raise SystemExit("--q-len needs head dimension 128 and q_len * G <= 16 (8 with --unique-kv fp8)")
        w = W.scaled(w, B=w.B * T)
        units_this_rank *= T
    fp8 = args.unique_kv == "fp8"
    f8 = None
    if fp8:
        # the private store in FP8 E4M3 with per-token scales; the bf16 copy is not kept
        if w.D != 128:
            raise SystemExit("--unique-kv fp8 needs head dimension 128")
        f8 = W.quantize_unique_store_fp8(un, release=True)
        torch.cuda.empty_cache()
    sfp8 = args.shared_kv == "fp8"
    if sfp8 and w.D != 128:
        raise SystemExit("--shared-kv fp8 needs head dimension 128")
    n_q = max(1, w.steps)
    qs = [W.make_queries(w, sh, s, dev) for s in range(n_q)]
    kv_lens = [(un.kv_len + s).to(torch.int32) for s in range(n_q)]
    max_len = int(lens0.max()) + w.steps
    layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, max_len, dense=w.dense,
                       n_unique_splits=args.unique_splits, fp8_unique=fp8, q_len=T)
    S = layer.shape
    if not w.dense:
        layer.build_summaries(sh.k_shared)
    sf8 = None
    if sfp8:
        # the shared store in FP8 E4M3 with one scale per (KV head, chunk); the chunk embeddings were
        # built from the bf16 keys (offline step); the bf16 copy is kept only for the per-request baseline
        sf8 = W.quantize_shared_store_fp8(sh)
    torch.cuda.synchronize()

    two_streams = (not args.one_stream) and layer.overlap_routing
    input_bytes = sh.k_shared.numel() * 4 + (f8.k8.numel() * 2 if fp8 else un.k_unique.numel() * 4)
    flush_buf = None
    if input_bytes < 2 * L2_BYTES:
        flush_buf = torch.empty(int(3 * L2_BYTES), dtype=torch.uint8, device=dev)
    flush = (lambda: flush_buf.fill_(1)) if flush_buf is not None else None

    # the host knows its batch: total private tokens per step, a scheduling hint for the library
    tokens = [int(k.sum().item()) for k in kv_lens]

    def step(i, prof=None):
        s = i % n_q
        if sfp8 and fp8:
            layer.step_fp8(qs[s], sf8, f8, un.kv_start, kv_lens[s], two_streams=two_streams, prof=prof,
                           unique_tokens=tokens[s])
        elif sfp8:
            layer.step_fp8shared(qs[s], sf8, un.k_unique, un.v_unique, un.kv_start, kv_lens[s],
                                 two_streams=two_streams, prof=prof, unique_tokens=tokens[s])
        elif fp8:
            layer.step_fp8kv(qs[s], sh.k_shared, sh.v_shared, f8, un.kv_start, kv_lens[s],
                             two_streams=two_streams, prof=prof, unique_tokens=tokens[s])
        else:
            layer.step(qs[s], sh.k_shared, sh.v_shared, un.k_unique, un.v_unique, un.kv_start,
                       kv_lens[s], two_streams=two_streams, prof=prof, unique_tokens=tokens[s])

    bound_host = {}

    def step_host(i):
        s = i % n_q
        if fp8 or sfp8:
            # one store in FP8: no host-buffer entry point, the same copies around the device call
            if sfp8 and fp8:
                # both stores in FP8: the host-buffer entry point of that step
                if s not in bound_host:
                    bound_host[s] = layer.bind_step_fp8_host(q_host[s], q_dev, out_host, sf8, f8, un.kv_start,
                                                             kv_lens[s], two_streams=two_streams,
                                                             unique_tokens=tokens[s])
                layer.shape.unique_tokens = tokens[s]
                bound_host[s]()
                return
            q_dev.copy_(q_host[s], non_blocking=True)
            if sfp8:
                out = layer.step_fp8shared(q_dev, sf8, un.k_unique, un.v_unique, un.kv_start, kv_lens[s],
                                           two_streams=two_streams, unique_tokens=tokens[s])
            else:
                out = layer.step_fp8kv(q_dev, sh.k_shared, sh.v_shared, f8, un.kv_start, kv_lens[s],
                                       two_streams=two_streams, unique_tokens=tokens[s])
            out_host.copy_(out, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        else:
            # the serving-loop form of the host-buffer call: arguments marshalled once per buffer set
            if s not in bound_host:
                bound_host[s] = layer.bind_step_host(
                    q_host[s], q_dev, out_host, sh.k_shared, sh.v_shared, un.k_unique, un.v_unique,
                    un.kv_start, kv_lens[s], two_streams=two_streams, unique_tokens=tokens[s])
            layer.shape.unique_tokens = tokens[s]
            bound_host[s]()

    def unique_alone():
        if fp8:
            layer.unique_fp8(qs[0], f8, un.kv_start, kv_lens[0])
        else:
            layer.unique(qs[0], un.k_unique, un.v_unique, un.kv_start, kv_lens[0])

    K = args.steps
    n_warm = max(3, args.warmup)
    for i in range(n_warm):
        step(i)
    torch.cuda.synchronize()

    # Per-stage device times of every stage from a short untimed pass (two event records per stage
    # and step cost about 3 us each); in the timed region only the dominant kernel's stage is
    # recorded, for the roofline.
    n_pre = min(16, max(8, K))
    prof_pre = M.profiler_create(n_pre)
    for i in range(n_pre):
        if flush is not None:
            flush()
        step(i, prof_pre)
    torch.cuda.synchronize()
    stage_ms_pre, n_rec = M.profiler_read(prof_pre)
    M.profiler_destroy(prof_pre)
    stage_ms_pre = {k: v / max(1, n_rec) for k, v in stage_ms_pre.items()}
    # The dominant kernel is the one with the longest roofline time for its algorithmic work (the
    # in-step durations do not say: a kernel that shares the SMs with another one is stretched).
    peaks = measured_peaks()
    lens = kv_lens[0].cpu().numpy().astype(np.int64)
    if w.dense:
        touched, P = w.Hkv * w.C, w.B * w.Hkv * w.C
    else:
        off = layer.seg_offsets.cpu().numpy()
        touched, P = int((np.diff(off) > 0).sum()), w.B * w.Hkv * w.k
    work = algorithmic_work(w, lens, S.n_unique_splits, S.shared_slots, touched)
    if fp8:  # one byte per element and two fp32 scales per (token, KV head) instead of bf16 K and V
        work["unique_bytes"] -= int(lens.sum()) * w.Hkv * (2 * w.D - 8)
    if sfp8:  # one byte per element of every touched chunk (the two scales per chunk are negligible)
        work["shared_bytes"] -= touched * 2 * w.D * w.L
    t_flops = work["shared_flops"] / (peaks["bf16_tflops_sustained"] * 1e12)
    t_bytes = work["shared_bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_unique = work["unique_bytes"] / (peaks["hbm_gbs"] * 1e9)
    dominant = "unique" if t_unique >= max(t_flops, t_bytes) else "shared"

    # ---- the timed region: R blocks of K steps, barrier + synchronize on both sides of a block
    prof = M.profiler_create(K)
    M.profiler_select(prof, [dominant])
    dom_ms = []

    def run_block():
        DD.barrier()
        torch.cuda.synchronize()
        if flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(K):
                step(i, prof)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
        else:
            ms = 0.0
            for i in range(K):
                flush()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                step(i, prof)
                e1.record()
                e1.synchronize()
                ms += e0.elapsed_time(e1)
        DD.barrier()
        t, n = M.profiler_read(prof)
        dom_ms.append(t[dominant] / max(1, n))
        return ms

    sampler = ClockSampler(local_rank)
    sampler.start()
    blocks = timed_blocks(run_block, args.min_timed_ms if headline else args.min_timed_ms / 2, dev)
    clocks = sampler.stop()
    M.profiler_destroy(prof)
    block_ms = statistics.median(blocks)
    ms_per_step = block_ms / K
    value = DD.sum_over_ranks(units_this_rank * K, dev) / (block_ms * 1e-3)
    stage_ms = dict(stage_ms_pre)
    stage_ms[dominant] = statistics.median(dom_ms)  # from the timed region itself

    # ---- end to end through the host-buffer entry point (pinned q in, out back, every step)
    q_host = [q.cpu().pin_memory() for q in qs]
    out_host = torch.empty(w.B, w.Hq, w.D, dtype=torch.bfloat16).pin_memory()
    q_dev = torch.empty_like(qs[0])
    for i in range(3):
        step_host(i)

    def run_block_host():
        DD.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if flush is None:
            e0.record()
            for i in range(K):
                step_host(i)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        ms = 0.0
        for i in range(K):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step_host(i)
            e1.record()
            e1.synchronize()
            ms += e0.elapsed_time(e1)
        return ms

    e2e_blocks = timed_blocks(run_block_host, args.min_timed_ms / 2 if headline else args.min_timed_ms / 4, dev)
    e2e_block_ms = statistics.median(e2e_blocks)
    e2e_value = DD.sum_over_ranks(units_this_rank * K, dev) / (e2e_block_ms * 1e-3)
    io_bytes = w.B * w.Hq * w.D * 2

    if rank != 0:
        return None

    # ---- per-kernel detail (rank 0, outside the timed region)
    iters = max(3, min(K, 10))
    gemv_ms = None
    if not args.no_baseline:
        big = w.dense and w.B * w.C > 20000   # 256 GiB of re-reads in the dense config: sample it
        if big:
            sub = MoskaLayer(8, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, max_len, dense=True,
                             dense_slots=S.shared_slots)
            qsub = qs[0][:8].contiguous()
            gemv_ms = time_events(lambda: sub.gemv_baseline(qsub, sh.k_shared, sh.v_shared), 3) * (w.B / 8)
        else:
            layer.gemv_baseline(qs[0], sh.k_shared, sh.v_shared)
            gemv_ms = time_events(lambda: layer.gemv_baseline(qs[0], sh.k_shared, sh.v_shared), iters, flush)
    gemv_step_ms = None
    if gemv_ms is not None:
        def baseline_step():
            if not w.dense:
                layer.route(qs[0])
                layer.group()
            unique_alone()
            layer.merge()
        # shared attention is the only stage that differs: time the other stages once, add the baseline
        gemv_step_ms = time_events(baseline_step, iters, flush) + gemv_ms
    # every kernel alone on the GPU (same inputs, after the timed region): separates a kernel's own
    # speed from the bandwidth and SM sharing of the two overlapped streams
    iso = {}
    if not w.dense:
        iso["route"] = time_events(lambda: layer.route(qs[0]), iters, flush)
        iso["group"] = time_events(lambda: layer.group(), iters, flush)
    if sfp8:
        iso["shared"] = time_events(lambda: layer.shared_fp8(qs[0], sf8), iters, flush)
    else:
        iso["shared"] = time_events(lambda: layer.shared(qs[0], sh.k_shared, sh.v_shared), iters, flush)
    iso["unique"] = time_events(unique_alone, iters, flush)
    iso["merge"] = time_events(lambda: layer.merge(), iters, flush)
    shared_ms, unique_ms = stage_ms["shared"], stage_ms["unique"]
    shared_tflops = work["shared_flops"] / (shared_ms * 1e-3) / 1e12 if shared_ms > 0 else None
    unique_gbs = work["unique_bytes"] / (unique_ms * 1e-3) / 1e9 if unique_ms > 0 else None
    shared_gbs = work["shared_bytes"] / (shared_ms * 1e-3) / 1e9 if shared_ms > 0 else None

    # dominant kernel and the roofline that bounds it
    if dominant == "unique":
        kernel = "unique_fp8_kernel" if fp8 else ("unique_staged_kernel" if w.D == 128 else "unique_attn_kernel")
        if T > 1 and not fp8:
            kernel = "unique_multi_kernel"
        roof = dict(bound="hbm", achieved=unique_gbs, peak=peaks["hbm_gbs"], unit="GB/s")
        algo = work["unique_bytes"]
    elif t_flops > t_bytes:
        kernel = "shared_tc_kernel"
        roof = dict(bound="tensor", achieved=shared_tflops, peak=peaks["bf16_tflops_sustained"],
                    unit="TFLOP/s")
        algo = None
    else:
        kernel = "shared_tc_kernel" if w.D == 128 else "shared_small_kernel"
        roof = dict(bound="hbm", achieved=shared_gbs, peak=peaks["hbm_gbs"], unit="GB/s")
        algo = work["shared_bytes"]
    roof["frac"] = roof["achieved"] / roof["peak"] if roof["achieved"] else None
    roof["traffic"] = NCU_TRAFFIC_BYTES.get((kernel, w.name))
    if roof["traffic"] is None and kernel in NCU_TRAFFIC_RATIO and algo is not None:
        ratio, how = NCU_TRAFFIC_RATIO[kernel]
        roof["traffic"] = ratio * algo
        roof["traffic_source"] = how
    roof["kernel"] = kernel
    roof["peak_source"] = "of " + peaks["source"]
    roof["avg_launch_ms"] = unique_ms if kernel.startswith("unique") else shared_ms
    roof["alone"] = {
        "avg_launch_ms": iso["unique"] if kernel.startswith("unique") else iso["shared"],
        "frac": ((work["unique_bytes"] / (iso["unique"] * 1e-3) / 1e9 / peaks["hbm_gbs"])
                 if kernel.startswith("unique") else
                 (work["shared_flops"] / (iso["shared"] * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"])
                 if roof["bound"] == "tensor" else
                 (work["shared_bytes"] / (iso["shared"] * 1e-3) / 1e9 / peaks["hbm_gbs"]))}

    # ---- CPU baseline: the oracle as it stands on the host cores, bounded sample (N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline and not fp8 and not sfp8 and T == 1:
        cpu = cpu_baseline(w, sh, un, qs[0], kv_lens[0], args.cpu_sample,
                           args.cpu_seconds if headline else args.cpu_seconds / 2)

    # the merge reads every partial once more and writes the bf16 result
    rows_merge_bytes = w.B * w.Hq * ((S.shared_slots + S.n_unique_splits) * (w.D + 1) * 4 + w.D * 2)
    # kernels of one step: route (scoring + selection beyond 256 chunks), 2-3 grouping passes, unique,
    # shared, merge
    # the tensor-core kernel and the 8-row streaming tiles (FP8 shared store: plus the query
    # conversion), or 16-row and 8-row tiles
    n_shared_launches = 3 if sfp8 else 2
    n_launch = (3 + (1 if sfp8 else 0)) if w.dense else \
        (1 + (w.C > 256)) + (3 if w.B > 64 else 2) + 1 + n_shared_launches + 1
    hbm_bytes = work["unique_bytes"] + work["shared_bytes"] + rows_merge_bytes
    amort = P / max(1, touched)
    rec = {
        "workload": w_full.name, "value": value, "ms_per_step": ms_per_step, "steps_per_block": K,
        "blocks": len(blocks), "block_ms": {"median": block_ms, "min": min(blocks), "max": max(blocks)},
        "timed_ms_total": sum(blocks), "scaling": scaling,
        "config": {
            "workload": w_full.name, "batch": w.B, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": w.D,
            "shared_tokens": w.C * w.L, "chunk_tokens": w.L, "top_k": None if w.dense else w.k,
            "unique_tokens_mean": float(lens.mean()), "n_unique_splits": S.n_unique_splits,
            "shared_slots": S.shared_slots, "streams": 2 if two_streams else 1,
            "unique_kv": "fp8_e4m3 + fp32 scale per (token, kv head)" if fp8 else "bf16",
            "shared_kv": "fp8_e4m3 + fp32 scale per (kv head, chunk)" if sfp8 else "bf16",
            "q_len": T, "requests": w.B // T,
            "l2": ("flushed between steps" if flush is not None
                   else f"inputs exceed L2 ({input_bytes / 2**20:.0f} MiB of K/V per step)"),
            "per_gpu": per_gpu,
            "timed_region": f"{len(blocks)} blocks of {K} steps, median block",
        },
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": io_bytes,
                "d2h_bytes_per_step": io_bytes, "ms_per_step": e2e_block_ms / K,
                "blocks": len(e2e_blocks)},
        "gpu_launches": n_launch * K * len(blocks),
        "gpu_launches_per_step": n_launch,
        "roofline": roof,
        "cpu_baseline": cpu,
        "stage_ms": stage_ms,
        "stage_ms_isolated": iso,
        "isolated": {
            "unique_gbs": work["unique_bytes"] / (iso["unique"] * 1e-3) / 1e9,
            "unique_frac_of_measured_hbm": work["unique_bytes"] / (iso["unique"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "shared_tflops": work["shared_flops"] / (iso["shared"] * 1e-3) / 1e12,
            "shared_frac_of_measured_sustained": work["shared_flops"] / (iso["shared"] * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
            "shared_frac_of_nominal_2250": work["shared_flops"] / (iso["shared"] * 1e-3) / 1e12 / 2250.0,
            "shared_gbs": work["shared_bytes"] / (iso["shared"] * 1e-3) / 1e9,
            "shared_frac_of_measured_hbm": work["shared_bytes"] / (iso["shared"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
        },
        "shared": {"tflops": shared_tflops, "frac_of_measured_sustained": (shared_tflops or 0) / peaks["bf16_tflops_sustained"],
                   "frac_of_nominal_2250": (shared_tflops or 0) / 2250.0, "gbs": shared_gbs,
                   "frac_of_measured_hbm": (shared_gbs or 0) / peaks["hbm_gbs"],
                   "touched_segments": touched, "pairs": P,
                   "amortisation_factor": amort},
        "unique": {"gbs": unique_gbs, "frac_of_measured_hbm": (unique_gbs or 0) / peaks["hbm_gbs"],
                   "frac_of_nominal_8000": (unique_gbs or 0) / 8000.0},
        # all HBM-bound work of the step against the step time: the two streams share the bandwidth,
        # so a kernel's own in-step rate (roofline.achieved) understates how busy HBM is
        "step_hbm": {"bytes": hbm_bytes, "gbs": hbm_bytes / (ms_per_step * 1e-3) / 1e9,
                     "frac_of_measured_hbm": hbm_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "gemv_baseline": None if gemv_ms is None else {
            "ms": gemv_ms,
            # algorithmic bytes of the baseline (every routed chunk once per request and KV head);
            # where they fit the 126 MB L2 part of them never reaches DRAM
            "algorithmic_gbs": work["gemv_bytes"] / (gemv_ms * 1e-3) / 1e9,
            "algorithmic_bytes": work["gemv_bytes"],
            "dram_bytes_ncu": GEMV_DRAM_BYTES.get(w_full.name),
            "shared_attention_bytes": work["shared_bytes"],
            # both kernels alone on the GPU (in the step part of shared attention overlaps unique)
            "shared_speedup": gemv_ms / iso["shared"] if iso["shared"] > 0 else None,
            "amortisation_factor": amort,
            "shared_speedup_over_amortisation": (gemv_ms / iso["shared"] / amort) if iso["shared"] > 0 else None,
            # the step with the per-request baseline in the place of shared attention, stages
            # back to back on one stream, against the real step
            "step_ms_with_baseline": gemv_step_ms,
            "step_speedup": None if gemv_step_ms is None else gemv_step_ms / ms_per_step},
    }
    return rec


def measure_disaggregated(args, w, rank, world, dev):
    """Rank 0 as the Shared-KV rank, the others as Unique-KV ranks (Section III-C in miniature): per
    step the unique ranks send their queries, run Unique KV Attention, receive the shared result of
    their requests and merge.  Point-to-point over the process group; no kernel reads a peer."""
    from paper_2511_06010_b200 import disaggregated as DG
    from paper_2511_06010_b200.engine import MoskaLayer

    if world < 2:
        raise SystemExit("--shard disaggregated needs at least 2 ranks")
    unique_ranks = list(range(1, world))
    blocks = DG.request_blocks(w.B, unique_ranks)
    lens_all = W.unique_lengths(w)
    K = args.steps
    if rank == 0:
        sh = W.make_shared_store(w, dev)
        layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, 1, dense=w.dense, n_unique_splits=1)
        role = DG.SharedRank(layer, sh.k_shared, sh.v_shared)
        q_all = torch.empty(w.B, w.Hq, w.D, dtype=torch.bfloat16, device=dev)
        q_local = kv_len = None
    else:
        _, b0, b1 = [b for b in blocks if b[0] == rank][0]
        wl = W.scaled(w, B=b1 - b0, shard=rank)
        un = W.make_unique_store(wl, dev, lens_all[b0:b1])
        mu = W.shared_centres(w, dev)
        q_local = W.make_queries(w, W.SharedStore(None, None, mu), 0, dev)[b0:b1].contiguous()
        kv_len = un.kv_len
        layer = MoskaLayer(b1 - b0, w.Hq, w.Hkv, w.D, 1, w.L, 1, int(lens_all.max()) + w.steps)
        role = DG.UniqueRank(layer, un.k_unique, un.v_unique, un.kv_start)
        q_all = None

    def one():
        DG.step(role, q_local, kv_len, 0, blocks, q_all=q_all)

    for _ in range(max(3, args.warmup)):
        one()

    def run_block():
        DD.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(K):
            one()
        e1.record()
        torch.cuda.synchronize()
        DD.barrier()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(dev.index)
    sampler.start()
    blocks_ms = timed_blocks(run_block, args.min_timed_ms, dev)
    clocks = sampler.stop()
    if rank != 0:
        return None
    block_ms = statistics.median(blocks_ms)
    rows = w.B * w.Hq
    return {
        "workload": w.name, "value": w.B * K / (block_ms * 1e-3), "ms_per_step": block_ms / K,
        "steps_per_block": K, "blocks": len(blocks_ms), "scaling": "strong",
        "config": {"workload": w.name, "batch": w.B,
                   "per_gpu": f"rank 0: shared store, routing, grouping, Shared KV Attention for all {w.B} requests; "
                              f"ranks 1..{world - 1}: private KV and Unique KV Attention of {w.B // (world - 1)} requests each",
                   "exchange_bytes_per_step": {"queries_up": rows * w.D * 2, "shared_partials_down": rows * (w.D + 1) * 4},
                   "timed_region": f"{len(blocks_ms)} blocks of {K} steps, median block"},
        "clocks": clocks, "e2e": None, "gpu_launches": None, "roofline": None, "cpu_baseline": None,
    }


def run_cuda(args):
    rank, local_rank, world = DD.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    from paper_2511_06010_b200 import build as B

    if rank == 0:
        B.build()
    DD.barrier()

    def pick(i):
        w = W.CONFIGS[i]
        if args.batch:
            w = W.scaled(w, name=f"{w.name}@B{args.batch}", B=args.batch)
        return w

    headline_idx = HEADLINE_CONFIG if args.config is None else args.config
    if world > 1 and args.shard == "disaggregated":
        rec = measure_disaggregated(args, pick(headline_idx), rank, world, dev)
        per = {}
    else:
        per = {}
        if args.config is None and not args.no_per_config and world == 1:
            for i in PER_CONFIG:
                r = measure(args, pick(i), rank, world, dev, headline=False)
                torch.cuda.empty_cache()
                if r is not None:
                    per[r["workload"]] = {
                        k: r[k] for k in ("value", "ms_per_step", "blocks", "timed_ms_total", "roofline",
                                          "gemv_baseline", "cpu_baseline", "stage_ms",
                                          "stage_ms_isolated", "isolated", "shared", "unique", "step_hbm",
                                          "e2e", "clocks")}
        rec = measure(args, pick(headline_idx), rank, world, dev, headline=True)
    if rank == 0:
        line = {
            "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": rec["ms_per_step"], "higher_is_better": True,
            "scaling": rec["scaling"], "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        }
        for k, v in rec.items():
            if k not in ("workload", "value", "ms_per_step", "scaling"):
                line[k] = v
        if per:
            line["per_config"] = per
        print(json.dumps(line), flush=True)
    DD.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="K: steps per timed block")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=None,
                    help="workload index 0..4; default: 4 as the headline plus per_config records of 1, 2, 3")
    ap.add_argument("--no-per-config", action="store_true", help="headline workload only")
    ap.add_argument("--min-timed-ms", type=float, default=500.0,
                    help="blocks of K steps are repeated until they add up to this much device time")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (sweeps)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--shard", default="kv_head", choices=["kv_head", "replicas", "disaggregated"],
                    help="what N > 1 ranks hold: KV heads of one batch (default), own batches, or the "
                         "Shared-KV / Unique-KV roles")
    ap.add_argument("--one-stream", action="store_true", help="run unique attention on the main stream")
    ap.add_argument("--unique-splits", type=int, default=None, help="override the split-K count of unique attention")
    ap.add_argument("--unique-kv", default="bf16", choices=["bf16", "fp8"],
                    help="storage of the private KV (fp8: E4M3 codes with per-token scales; no CPU baseline)")
    ap.add_argument("--shared-kv", default="bf16", choices=["bf16", "fp8"],
                    help="storage of the shared KV (fp8: E4M3 codes with one scale per (KV head, chunk); routed "
                         "workloads; no CPU baseline)")
    ap.add_argument("--q-len", type=int, default=1,
                    help="query tokens per request (batch rows = requests x q_len; queries/s counts rows; no CPU baseline)")
    ap.add_argument("--no-baseline", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample", type=int, default=16, help="requests in the CPU-oracle sample")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--ref-sample", type=int, default=8, help="requests per step of --impl reference")
    args = ap.parse_args()
    if args.impl == "reference":
        w = W.CONFIGS[HEADLINE_CONFIG if args.config is None else args.config]
        if args.batch:
            w = W.scaled(w, name=f"{w.name}@B{args.batch}", B=args.batch)
        run_reference(args, w)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
