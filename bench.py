#!/usr/bin/env python
"""Benchmark of the fused attention forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic input: for the default
workload ``c2`` (B=4, H=16, Sq=Sk=4096, D=128, bf16) one non-causal and one causal call, as
the configuration is stated.  The metric is effective attention-forward TFLOP/s counting only
unmasked FLOPs (4*D per visible query/key pair).  Inputs are resident in HBM for ``value``;
``e2e`` repeats the measurement through ``attn_fwd_host`` with pinned host buffers, copies
inside the timed region.  Rank 0 prints one JSON line.

With N > 1 (under torchrun) every rank runs the same workload on its own GPU: the problems
are independent batches, there is no data-path collective, scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from synth_inputs import benchmark_workloads, gemm_case_study_workloads, make_ab, make_qkv

METRIC = "effective attention-fwd TFLOP/s (unmasked FLOPs)"
UNIT = "TFLOP/s"

# name -> list of workload variants that make one step
STEP_SETS = {
    "c2": ["c2_noncausal", "c2_causal"],
    "c2_noncausal": ["c2_noncausal"],
    "c2_causal": ["c2_causal"],
    "c3": ["c3_gqa_window_alibi"],
    "c4": ["c4a_softcap", "c4b_sigmoid"],
    "c4a": ["c4a_softcap"],
    "c4b": ["c4b_sigmoid"],
    "c5": ["c5_packed_doc_causal"],
    "c1": ["c1_fp32_causal"],
}

# DRAM bytes per launch of the dominant kernel, per variant, from the ncu captures summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum of one launch); a step set reports the mean
# over its launches; None where no capture exists.
NCU_TRAFFIC_BYTES_PER_VARIANT = {
    "c2_noncausal": 314.3e6, "c2_causal": 344.6e6, "c3_gqa_window_alibi": 309.9e6,
    "c4a_softcap": 344.3e6, "c4b_sigmoid": 395.2e6, "c5_packed_doc_causal": 1182.3e6,
}


# The same for the GEMM + row-sum kernel, per workload.
GEMM_NCU_TRAFFIC_BYTES = {"g_4k_4k_4k": 75.4e6}


def ncu_traffic(workload_key):
    per = [NCU_TRAFFIC_BYTES_PER_VARIANT.get(n) for n in STEP_SETS[workload_key]]
    return None if any(x is None for x in per) else float(sum(per) / len(per))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return {"bf16_tflops": float(m["bf16_tflops"]), "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", 0.0)),
                "hbm_gbs": float(m["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML from a background thread.  The thread is started ahead
    of the timed region (its first queries are slow) and keeps sampling; ``begin()`` / ``end()`` mark the region,
    and the summary covers the samples taken between the two marks."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.samples, self.max_mhz = [], None          # (time, MHz, reason mask)
        self.period_s = period_s
        self._stop = threading.Event()
        self._thread = None
        self._t0 = self._t1 = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            pynvml.nvmlDeviceGetClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _reason_names(self):
        nv = self._nv
        return {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.samples.append((time.perf_counter(), mhz, mask))
            except Exception:
                pass
            time.sleep(self.period_s)

    def start(self):
        if self._nv is not None and self._thread is None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
            time.sleep(0.02)                    # let the first (slow) queries pass before anything is timed
        return self

    def begin(self):
        self._t0 = time.perf_counter()

    def end(self):
        self._t1 = time.perf_counter()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    # context-manager form: the whole block is the region
    def __enter__(self):
        self.start()
        self.begin()
        return self

    def __exit__(self, *exc):
        self.end()
        self.stop()

    def summary(self):
        t0 = self._t0 if self._t0 is not None else 0.0
        t1 = self._t1 if self._t1 is not None else float("inf")
        inside = [(m, r) for t, m, r in self.samples if t0 <= t <= t1]
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        mask = 0
        for _, r in inside:
            mask |= r
        reasons = sorted(name for bit, name in self._reason_names().items() if mask & bit)
        return {"sm_mhz": float(np.median([m for m, _ in inside])), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(inside)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def config_block(workload_key, workloads):
    """The ``config`` object of the JSON line: the same for the CUDA arm and for the reference (oracle) arm."""
    from workload_flops import algorithmic_bytes
    step_bytes = sum(algorithmic_bytes(w) for w in workloads)
    flushed = step_bytes < (256 << 20)
    return {"workload": workload_key, "variants": STEP_SETS[workload_key],
            "shape": {k: getattr(workloads[0], k) for k in ("B", "Hq", "Hkv", "Sq", "Sk", "D")},
            "l2": (f"inputs and outputs of a step ({step_bytes / 1e6:.0f} MB) are larger than the 126 MB L2; no flush"
                   if not flushed else
                   f"a step touches {step_bytes / 1e6:.1f} MB: L2 flushed (256 MB overwritten) before every launch; "
                   "time = sum of the per-launch event intervals"),
            "per_rank": "same workload on every GPU, different seeds, no collective"}, flushed


# Multiply-adds (rows x keys x head dimension, summed over the step's variants) of one oracle sample: about 20 s on
# the 16 host cores of this pool's GPU machines.
ORACLE_SAMPLE_WORK = 2.0e11


def oracle_sample(workloads, target_rows):
    """Times the float64 oracle, as it stands, on evenly spaced rows of each variant.
    Returns (TFLOP/s over the unmasked FLOPs of those rows, threads, description, seconds)."""
    import oracle
    from oracle.attn_oracle import NORM_RELU, NORM_SIGMOID, NORM_SOFTMAX, OracleVariant
    from workload_flops import row_visibility

    flops, secs, desc = 0.0, 0.0, []
    for w in workloads:
        q, k, v = make_qkv(w)
        var = OracleVariant(normalizer={"softmax": NORM_SOFTMAX, "sigmoid": NORM_SIGMOID, "relu": NORM_RELU}[w.normalizer],
                            causal=w.causal, window_left=w.window_left, window_right=w.window_right,
                            scale=w.scale, softcap=w.softcap, slopes=w.slopes, sigmoid_bias=w.sigmoid_bias,
                            out_scale=w.out_scale, cu_seqlens=w.cu_seqlens, prefix_len=w.prefix_len,
                            test_query_start=w.test_query_start, global_len=w.global_len)
        total = w.B * w.Hq * w.Sq
        # the oracle computes every score of a row (all Sk keys): bound the sample's work, not only its row count
        n = max(64, min(total, target_rows, int(ORACLE_SAMPLE_WORK / (w.Sk * w.D * len(workloads)))))
        rows = np.unique(np.linspace(0, total - 1, n).astype(np.int64))
        oracle.attn_fwd_rows(q, k, v, var, rows[:8])            # page the library and inputs in
        t0 = time.perf_counter()
        oracle.attn_fwd_rows(q, k, v, var, rows)
        secs += time.perf_counter() - t0
        pre, lo, hi = row_visibility(w.Sq, w.Sk, causal=w.causal, window_left=w.window_left,
                                     window_right=w.window_right, cu_seqlens=w.cu_seqlens, prefix_len=w.prefix_len,
                                     test_query_start=w.test_query_start, global_len=w.global_len)
        vis = (np.maximum(hi - lo + 1, 0) + pre)[rows % w.Sq]
        flops += 4.0 * w.D * float(vis.sum())
        desc.append(f"{w.name}: {len(rows)} of {total} rows, evenly spaced")
    return flops / secs / 1e12, oracle.num_threads(), "; ".join(desc), secs


def run_reference(args, rank):
    if rank != 0:
        return
    wl = benchmark_workloads()
    workloads = [wl[n] for n in STEP_SETS[args.workload]]
    per_step_rows = max(64, args.ref_rows // max(1, len(workloads)))
    vals, secs = [], []
    for _ in range(args.warmup):
        oracle_sample(workloads, 64)
    cores, sample = 0, ""
    for _ in range(args.steps):
        v, cores, sample, s = oracle_sample(workloads, per_step_rows)
        vals.append(v)
        secs.append(s)
    value = float(np.sum([v * s for v, s in zip(vals, secs)]) / np.sum(secs))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_block(args.workload, workloads)[0],
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GEMM + row sum (the paper's GEMM case study): --workload g_<M>_<N>_<K>
# ------------------------------------------------------------------------------------------------
GEMM_METRIC = "GEMM + row ReduceSum TFLOP/s (2*M*N*K)"
# TFLOPS of the paper's generated kernel on H100 (Table "GEMM+ReduceSum"), by workload name: other hardware, context only.
GEMM_PAPER_H100_TFLOPS = {"g_4k_4k_4k": 566.76, "g_1k_1k_1k": 87.65, "g_4k_4k_1k": 592.41, "g_2k_4k_1k": 386.06,
                          "g_4k_2k_1k": 447.39}


def gemm_oracle_sample(w, target_rows):
    """Times the float64 oracle, as it stands, on evenly spaced rows of A.  Returns (TFLOP/s, threads, description, s)."""
    import oracle
    a, b = make_ab(w)
    rows = np.unique(np.linspace(0, w.M - 1, min(w.M, target_rows)).astype(np.int64))
    oracle.gemm_rowsum(a, b, rows=rows[:4])
    t0 = time.perf_counter()
    oracle.gemm_rowsum(a, b, rows=rows)
    secs = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    except Exception:
        cores = len(os.sched_getaffinity(0))
    return 2.0 * len(rows) * w.N * w.K / secs / 1e12, cores, f"{w.name}: {len(rows)} of {w.M} rows of A, evenly spaced", secs


def run_gemm_reference(args, rank):
    if rank != 0:
        return
    w = gemm_case_study_workloads()[args.workload]
    for _ in range(args.warmup):
        gemm_oracle_sample(w, 8)
    vals, secs, cores, sample = [], [], 0, ""
    for _ in range(args.steps):
        v, cores, sample, sec = gemm_oracle_sample(w, max(8, args.ref_rows // 64))
        vals.append(v)
        secs.append(sec)
    value = float(np.sum([v * t for v, t in zip(vals, secs)]) / np.sum(secs))
    print(json.dumps({
        "impl": "reference", "metric": GEMM_METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": args.workload},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}), flush=True)


def run_gemm(args, rank, world, local):
    """One step = one gemm_rowsum call (C and the row sums).  Every rank multiplies its own matrices: no collective."""
    args.warmup = max(args.warmup, 3)
    import torch.distributed as dist
    import paper_2605_05023_b200 as pk
    from paper_2605_05023_b200.ranks import max_over_ranks, rank_seed, whole_job_throughput
    from dataclasses import replace

    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = gemm_case_study_workloads()[args.workload]
    w = replace(w, seed=rank_seed(w.seed, rank))
    a, b = make_ab(w)
    stream = torch.cuda.current_stream(dev)
    set_bytes = 2 * (w.M * w.K + w.K * w.N + w.M * w.N) + 4 * w.M
    # Copies of the operands that together exceed L2 three times over: a launch meets inputs that were last touched
    # n_sets launches ago, i.e. evicted (no flush between launches, the kernels run back to back).
    n_sets = max(2, -(-(384 << 20) // set_bytes))
    sets = [{"a": a.to(dev), "b": b.to(dev), "c": torch.empty((w.M, w.N), device=dev, dtype=torch.bfloat16),
             "r": torch.empty((w.M,), device=dev, dtype=torch.float32)} for _ in range(n_sets)]
    status = torch.zeros(64, dtype=torch.int32, device=dev)
    flops = 2.0 * w.M * w.N * w.K
    count = [0]

    def step(events=None):
        s = sets[count[0] % n_sets]
        count[0] += 1
        if events is not None:
            e0 = torch.cuda.Event(enable_timing=True)
            e0.record(stream)
        pk.gemm_rowsum(s["a"], s["b"], c=s["c"], rowsum=s["r"], status_word=status, stream=stream)
        if events is not None:
            e1 = torch.cuda.Event(enable_timing=True)
            e1.record(stream)
            events.append((e0, e1))

    for _ in range(args.warmup):
        step()
    barrier()
    launches0 = pk.gemm_rowsum_launch_count()
    events = []
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(physical_gpu_index(local)) as clocks:
        t_start.record(stream)
        for _ in range(args.steps):
            step(events)
        t_stop.record(stream)
        barrier()
    launches = pk.gemm_rowsum_launch_count() - launches0
    word = int(status[0].item())
    if word != 0:
        raise RuntimeError(f"{w.name}: kernel reported status {word} ({pk.status_string(word)})")
    ms_total = max_over_ranks(t_start.elapsed_time(t_stop), dev)
    value = whole_job_throughput(flops * args.steps, ms_total * 1e-3, world) / 1e12
    per_launch = [e0.elapsed_time(e1) for e0, e1 in events]
    ms_per_launch = float(np.mean(per_launch))
    peaks = measured_peaks()
    achieved = flops / (ms_per_launch * 1e-3) / 1e12
    roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"], "traffic": GEMM_NCU_TRAFFIC_BYTES.get(args.workload),
                "peak_kind": f"bf16 dense burst, of {peaks['source']}",
                "frac_of_sustained_peak": (achieved / peaks["bf16_tflops_sustained"]) if peaks["bf16_tflops_sustained"] else None,
                "kernel": "gemm_rowsum_pair_kernel (CTA pairs; 256 x 512 tiles for K >= 2048 with enough tiles, else 256 x 256; each interval also holds the 4*M-byte clear of the row sums)",
                "launches": len(per_launch), "ms_per_launch": ms_per_launch, "median_ms_per_launch": float(np.median(per_launch)),
                "algorithmic_bytes": set_bytes}

    e2e = None
    if not args.no_e2e:
        e2e_steps = max(3, min(args.steps, 10))
        ah, bh = a.contiguous().pin_memory(), b.contiguous().pin_memory()
        ch = torch.empty((w.M, w.N), dtype=torch.bfloat16).pin_memory()
        rh = torch.empty((w.M,), dtype=torch.float32).pin_memory()
        ws = torch.empty(pk.gemm_rowsum_host_workspace_bytes(w.M, w.N, w.K), device=dev, dtype=torch.uint8)
        for _ in range(3):
            pk.gemm_rowsum_host(ah, bh, ch, rh, ws, status_word=status, stream=stream)
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(e2e_steps):
            pk.gemm_rowsum_host(ah, bh, ch, rh, ws, status_word=status, stream=stream)
        s1.record(stream)
        barrier()
        ms_e2e = max_over_ranks(s0.elapsed_time(s1), dev)
        e2e = {"value": whole_job_throughput(flops * e2e_steps, ms_e2e * 1e-3, world) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": int(2 * (w.M * w.K + w.K * w.N)), "d2h_bytes_per_step": int(2 * w.M * w.N + 4 * w.M),
               "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps,
               "api": "gemm_rowsum_host (pinned host buffers, copies in the timed region)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample, secs = gemm_oracle_sample(w, 1024)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": secs}

    if rank == 0:
        paper = GEMM_PAPER_H100_TFLOPS.get(args.workload)
        print(json.dumps({
            "metric": GEMM_METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": (value / world / paper) if paper else None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "shape": {"M": w.M, "N": w.N, "K": w.K},
                       "l2": f"{n_sets} copies of the operands and outputs ({n_sets * set_bytes / 1e6:.0f} MB, L2 is 126 MB) used in "
                             "turn: every launch reads inputs that have been evicted; no flush",
                       "vs_baseline_note": "against the paper's generated kernel on H100 (other hardware: context)",
                       "per_rank": "same shape on every GPU, different seeds, no collective"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks.summary(), "rejected_runs": [],
            "pct_of_nominal_dense_bf16_peak": 100.0 * value / world / 2250.0}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Context numbers: the paper's sweep shapes (three models x four sequence lengths at 16k tokens) for the
    Appendix A variants this library builds.  Inputs are drawn on the device from a seeded generator; every
    point moves more than L2 (>= 270 MB); 3 warm-up and 20 timed launches per point, CUDA events."""
    import paper_2605_05023_b200 as pk
    from workload_flops import unmasked_flops
    from synth_inputs import paper_sweep_workloads
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev).manual_seed(9000)
    bufs = {}
    rows = []
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for w in paper_sweep_workloads():
        if args.sweep_filter and not any(f in w.name for f in args.sweep_filter.split(",")):
            continue
        key = (w.Hq, w.Hkv, w.D)
        if key not in bufs:
            bufs.clear()
            torch.cuda.empty_cache()
            bufs[key] = tuple(torch.randn(16384 * h * w.D, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
                              for h in (w.Hq, w.Hkv, w.Hkv))
        qf, kf, vf = bufs[key]
        q = qf[: w.B * w.Sq * w.Hq * w.D].view(w.B, w.Sq, w.Hq, w.D).transpose(1, 2).contiguous()
        k = kf[: w.B * w.Sk * w.Hkv * w.D].view(w.B, w.Sk, w.Hkv, w.D).transpose(1, 2).contiguous()
        v = vf[: w.B * w.Sk * w.Hkv * w.D].view(w.B, w.Sk, w.Hkv, w.D).transpose(1, 2).contiguous()
        o = torch.empty((w.B, w.Hq, w.Sq, w.D), device=dev, dtype=torch.bfloat16)
        kw = pk.variant_kwargs(w, dev)
        for _ in range(3):
            pk.attn_fwd(q, k, v, o=o, status_word=status, **kw)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            pk.attn_fwd(q, k, v, o=o, status_word=status, **kw)
        e1.record()
        torch.cuda.synchronize()
        if int(status.item()) != 0:
            raise RuntimeError(f"{w.name}: kernel reported status {int(status.item())}")
        ms = e0.elapsed_time(e1) / 20
        variant, model, s = w.name.split("|")
        rows.append({"variant": variant, "model": model, "heads": f"{w.Hq}/{w.Hkv}/{w.D}", "S": int(s), "B": w.B,
                     "ms": ms, "tflops": unmasked_flops(w) / (ms * 1e-3) / 1e12})
    print(json.dumps({"sweep": "paper", "unit": "TFLOP/s (unmasked FLOPs)", "dtype": "bf16", "data": "synthetic",
                      "timing": "3 warm-up + 20 launches per point, CUDA events, inputs > L2", "rows": rows}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c2", choices=sorted(STEP_SETS) + sorted(gemm_case_study_workloads()),
                    help="c1..c5: attention configurations; g_<M>_<N>_<K>: GEMM + row sum shapes of the paper's case study")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ref-rows", type=int, default=16384, help="oracle rows per reference step")
    ap.add_argument("--cpu-rows", type=int, default=393216, help="oracle rows of the cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 1.5 s steady-state run")
    ap.add_argument("--no-per-config", action="store_true", help="skip the per-configuration roofline block")
    ap.add_argument("--per-config-launches", type=int, default=60)
    ap.add_argument("--sweep", choices=["paper"], help="time the paper-shaped sweep instead (one JSON object; 1 GPU)")
    ap.add_argument("--sweep-filter", default="", help="comma-separated substrings: only sweep points whose name holds one of them")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.workload in gemm_case_study_workloads():
        if args.impl == "reference":
            run_gemm_reference(args, rank)
        else:
            run_gemm(args, rank, world, local)
        return
    if args.impl == "reference":
        run_reference(args, rank)
        return

    run_attention(args, rank, world, local)


# Variants whose kernel-only throughput the default line reports one by one (``roofline.per_config``): every large
# bf16 configuration, each timed alone over back-to-back launches.
PER_CONFIG_VARIANTS = ["c2_noncausal", "c2_causal", "c3_gqa_window_alibi", "c4a_softcap", "c4b_sigmoid", "c5_packed_doc_causal"]


def kernel_name(w):
    if w.dtype != "bf16":
        return "attn_fwd_fp32_kernel"
    if w.global_len is not None:
        return "attn_fwd_split_kernel (one tile per CTA)"
    return "attn_fwd_pair_kernel (CTA pairs)" if w.D == 256 else "attn_fwd_tc_kernel (two-tile ping-pong)"


def run_attention(args, rank, world, local):
    args.warmup = max(args.warmup, 3)
    import torch.distributed as dist
    import paper_2605_05023_b200 as pk
    from workload_flops import algorithmic_bytes, unmasked_flops
    from paper_2605_05023_b200.ranks import max_over_ranks, rank_seed, whole_job_throughput

    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl = benchmark_workloads()
    names = STEP_SETS[args.workload]
    workloads = [wl[n] for n in names]
    stream = torch.cuda.current_stream(dev)
    peaks = measured_peaks()
    gpu_index = physical_gpu_index(local)

    def make_case(w):
        q, k, v = make_qkv(w.with_(seed=rank_seed(w.seed, rank)))   # every rank its own batch
        odt = torch.float32 if w.o_dtype == "fp32" else torch.bfloat16
        return {"w": w, "host": (q, k, v), "q": q.to(dev), "k": k.to(dev), "v": v.to(dev),
                "o": torch.empty((w.B, w.Hq, w.Sq, w.D), device=dev, dtype=odt),
                "lse": None if w.normalizer != "softmax" else torch.empty((w.B, w.Hq, w.Sq), device=dev, dtype=torch.float32),
                "kw": pk.variant_kwargs(w, dev), "flops": unmasked_flops(w), "bytes": algorithmic_bytes(w),
                "status": torch.zeros(1, dtype=torch.int32, device=dev)}

    def launch(c):
        pk.attn_fwd(c["q"], c["k"], c["v"], o=c["o"], lse=c["lse"], stream=stream, status_word=c["status"], **c["kw"])

    def status_error(cs):
        bad = None
        for c in cs:
            word = int(c["status"].item())
            if word != 0:
                bad = f"{c['w'].name}: kernel reported status {word} ({pk.status_string(word)})"
                c["status"].zero_()
        return bad

    # ---- resident inputs ----------------------------------------------------------------------
    cases = [make_case(w) for w in workloads]
    step_flops = float(sum(c["flops"] for c in cases))
    # A step whose inputs and outputs fit in L2 (126 MB) gets the L2 flushed before every launch (a 256 MB
    # buffer is overwritten); its time is then the sum of the per-launch CUDA-event intervals.
    config, flushed = config_block(args.workload, workloads)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if flushed else None

    def step(events=None):
        for c in cases:
            if flush_buf is not None:
                flush_buf.zero_()
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            launch(c)
            if events is not None:
                e1 = torch.cuda.Event(enable_timing=True)
                e1.record(stream)
                events.append((c["w"].name, e0, e1))

    for _ in range(args.warmup):
        step()
    barrier()
    # A timed region in which a kernel reported an error (a bounded device-side wait that gave up) is no
    # measurement: it is rejected and taken once more; the JSON line says so ("rejected_runs").
    rejected = []
    for attempt in range(2):
        launches0 = pk.launch_count()
        kernel_events = []
        t_start = torch.cuda.Event(enable_timing=True)
        t_stop = torch.cuda.Event(enable_timing=True)
        clocks = ClockSampler(gpu_index, period_s=0.0005).start()
        barrier()
        clocks.begin()
        t_start.record(stream)
        for _ in range(args.steps):
            step(kernel_events)
        t_stop.record(stream)
        barrier()
        clocks.end()
        clocks.stop()
        launches = pk.launch_count() - launches0
        bad = status_error(cases)
        if world > 1:   # every rank repeats if any rank has to
            flag = torch.tensor([1 if bad else 0], device=dev)
            dist.all_reduce(flag, op=dist.ReduceOp.MAX)
            if int(flag.item()) and bad is None:
                bad = "another rank reported a kernel error"
        if bad is None:
            break
        rejected.append(bad)
        print(f"bench: timed region rejected ({bad})", file=sys.stderr, flush=True)
    else:
        raise RuntimeError("; ".join(rejected))
    ms_total = t_start.elapsed_time(t_stop)
    if flush_buf is not None:
        ms_total = float(sum(e0.elapsed_time(e1) for _, e0, e1 in kernel_events))
    ms_total = max_over_ranks(ms_total, dev)
    value = whole_job_throughput(step_flops * args.steps, ms_total * 1e-3, world) / 1e12
    clock_summary = clocks.summary()

    # per-kernel durations (CUDA events on the launching stream), for the roofline
    per_variant = {}
    for name, e0, e1 in kernel_events:
        per_variant.setdefault(name, []).append(e0.elapsed_time(e1))
    kernel_ms = sum(float(np.sum(v)) for v in per_variant.values())
    n_launch = sum(len(v) for v in per_variant.values())
    flops_per_launch = step_flops * args.steps / n_launch
    ms_per_launch = kernel_ms / n_launch
    compute_bound = workloads[0].dtype == "bf16"
    traffic_note = "stored figure: dram__bytes_read.sum + dram__bytes_write.sum of one launch from the ncu captures under profiles/, not measured in this run"
    if compute_bound:
        achieved = flops_per_launch / (ms_per_launch * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops"], "traffic": ncu_traffic(args.workload), "traffic_note": traffic_note,
                    "peak_kind": f"bf16 dense burst, of {peaks['source']}",
                    "kernel": kernel_name(workloads[0]),
                    "launches": n_launch, "ms_per_launch": ms_per_launch,
                    "ms_x_sm_mhz": (ms_per_launch * clock_summary["sm_mhz"]) if clock_summary["sm_mhz"] else None,
                    "median_ms_per_launch": {n: float(np.median(v)) for n, v in per_variant.items()},
                    "per_variant_tflops": {n: float(unmasked_flops(wl[n]) / (np.mean(v) * 1e-3) / 1e12)
                                           for n, v in per_variant.items()}}
    else:
        gbs = sum(c["bytes"] for c in cases) * args.steps / n_launch / (ms_per_launch * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": gbs / peaks["hbm_gbs"], "traffic": ncu_traffic(args.workload), "traffic_note": traffic_note,
                    "peak_kind": f"copy bandwidth, of {peaks['source']}; this workload (17 MFLOP, 0.5 MB) is launch-latency bound",
                    "kernel": "attn_fwd_fp32_kernel", "launches": n_launch, "ms_per_launch": ms_per_launch,
                    "median_ms_per_launch": {n: float(np.median(v)) for n, v in per_variant.items()}}
        if flush_buf is not None:
            # the same launches with a warm L2 (no flush in between), for comparison with the cold figure above
            warm = []
            for _ in range(50):
                for c in cases:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    launch(c)
                    e1.record(stream)
                    warm.append((e0, e1))
            torch.cuda.synchronize()
            roofline["warm_l2_median_ms_per_launch"] = float(np.median([a.elapsed_time(b) for a, b in warm]))

    # ---- the same step repeated for at least 1.5 s: the power-capped steady state ------------------
    # (A short timed region runs at the boost clock; a long one settles at the clock the 1000 W limit allows.  The
    # contract value above is the K steps asked for; this block says what a long-running job sees.)
    sustained = None
    if compute_bound and world == 1 and not args.no_sustained:
        n_sus = max(args.steps, int(np.ceil(1500.0 / max(ms_total / args.steps, 1e-3))))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(gpu_index, period_s=0.01) as sus_clocks:
            s0.record(stream)
            for _ in range(n_sus):
                step()
            s1.record(stream)
            torch.cuda.synchronize()
        bad = status_error(cases)
        if bad is not None:
            raise RuntimeError(bad)
        ms_sus = s0.elapsed_time(s1)
        v_sus = step_flops * n_sus / (ms_sus * 1e-3) / 1e12
        sc = sus_clocks.summary()
        sustained = {"value": v_sus, "unit": UNIT, "steps": n_sus, "seconds": ms_sus * 1e-3, "ms_per_step": ms_sus / n_sus,
                     "clocks": sc, "ms_per_step_x_sm_mhz": (ms_sus / n_sus * sc["sm_mhz"]) if sc["sm_mhz"] else None,
                     "frac_of_burst_peak": v_sus / peaks["bf16_tflops"],
                     "frac_of_sustained_peak": (v_sus / peaks["bf16_tflops_sustained"]) if peaks["bf16_tflops_sustained"] else None}

    # ---- end to end: pinned host buffers through attn_fwd_host ------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(3, min(args.steps, 10))
        h2d = d2h = 0
        hcases = []
        for c in cases:
            w = c["w"]
            qh, kh, vh = (t.contiguous().pin_memory() for t in c["host"])
            oh = torch.empty_like(c["o"], device="cpu").pin_memory()
            lh = None if c["lse"] is None else torch.empty_like(c["lse"], device="cpu").pin_memory()
            desc = pk.make_desc(c["q"], c["k"], c["v"], c["o"], **c["kw"])
            ws = torch.empty(pk.host_workspace_bytes(w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.D, desc), device=dev, dtype=torch.uint8)
            hcases.append((qh, kh, vh, oh, lh, ws, c["kw"]))
            h2d += sum(t.numel() * t.element_size() for t in (qh, kh, vh))
            d2h += oh.numel() * oh.element_size() + (0 if lh is None else lh.numel() * 4)

        # One side stream per case: the device-to-host copy of one call's output overlaps the host-to-device copy of
        # the next call's inputs (separate copy engines).  The timed interval is taken on the launching stream, which
        # the side streams wait for at the start and which waits for them at the end.
        side = [torch.cuda.Stream(device=dev) for _ in hcases]

        def e2e_step():
            for (qh, kh, vh, oh, lh, ws, kw), st in zip(hcases, side):
                pk.attn_fwd_host(qh, kh, vh, oh, lh, ws, stream=st, **kw)

        def fork():
            ev = torch.cuda.Event()
            ev.record(stream)
            for st in side:
                st.wait_event(ev)

        def join():
            for st in side:
                ev = torch.cuda.Event()
                ev.record(st)
                stream.wait_event(ev)

        fork()
        for _ in range(3):
            e2e_step()
        join()
        barrier()
        s0 = torch.cuda.Event(enable_timing=True)
        s1 = torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        fork()
        for _ in range(e2e_steps):
            e2e_step()
        join()
        s1.record(stream)
        barrier()
        ms_e2e = s0.elapsed_time(s1)
        ms_e2e = max_over_ranks(ms_e2e, dev)
        e2e = {"value": whole_job_throughput(step_flops * e2e_steps, ms_e2e * 1e-3, world) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
               "ms_per_step": ms_e2e / e2e_steps,
               "api": "attn_fwd_host (pinned host buffers, copies in the timed region; one stream per call of the step)"}
        del hcases

    # ---- every large configuration on its own (rank 0, N = 1 only) ---------------------------------
    per_config = None
    if compute_bound and rank == 0 and world == 1 and not args.no_per_config:
        per_config = {}
        by_name = {c["w"].name: c for c in cases}
        n_pc = max(50, args.per_config_launches)
        for name in PER_CONFIG_VARIANTS:
            c = by_name.get(name) or make_case(wl[name])
            for _ in range(5):
                launch(c)
            torch.cuda.synchronize()
            evs = []
            with ClockSampler(gpu_index) as pc_clocks:
                for _ in range(n_pc):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    launch(c)
                    e1.record(stream)
                    evs.append((e0, e1))
                torch.cuda.synchronize()
            bad = status_error([c])
            if bad is not None:
                raise RuntimeError(bad)
            ms = np.array([a.elapsed_time(b) for a, b in evs])
            pc = pc_clocks.summary()
            tf = c["flops"] / (float(ms.mean()) * 1e-3) / 1e12
            per_config[name] = {
                "flops_per_launch": float(c["flops"]), "launches": n_pc, "mean_ms": float(ms.mean()), "median_ms": float(np.median(ms)),
                "tflops": tf, "tflops_at_median": c["flops"] / (float(np.median(ms)) * 1e-3) / 1e12,
                "frac_of_burst_peak": tf / peaks["bf16_tflops"], "algorithmic_bytes": int(c["bytes"]),
                "traffic": NCU_TRAFFIC_BYTES_PER_VARIANT.get(name), "kernel": kernel_name(c["w"]),
                "sm_mhz": pc["sm_mhz"], "clock_samples": pc["samples"], "reasons": pc["reasons"],
                "mean_ms_x_sm_mhz": (float(ms.mean()) * pc["sm_mhz"]) if pc["sm_mhz"] else None}
            if name not in by_name:
                del c
                torch.cuda.empty_cache()
        roofline["per_config"] = per_config
        roofline["per_config_note"] = (f"each configuration alone, {n_pc} back-to-back launches after 5 warm-up launches, CUDA events per launch; "
                                       "inputs and outputs of every configuration exceed L2; traffic = stored ncu figures")

    # ---- oracle on the host cores (rank 0, N = 1 only) -------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample, secs = oracle_sample(workloads, max(64, args.cpu_rows // len(workloads)))
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": secs}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if compute_bound else "f32", "data": "synthetic",
            "config": config,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clock_summary, "sustained": sustained, "rejected_runs": rejected,
            "pct_of_nominal_dense_bf16_peak": 100.0 * value / world / 2250.0,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
