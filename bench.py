#!/usr/bin/env python
"""Benchmark of the A2SF hot path: one "step" = prefill (attention + scores +
selection) + cache build + T fused decode steps over one synthetic batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line.  `value` is the decode-step throughput in algorithmic GB/s
(inputs resident in HBM); `prefill` carries the prefill-scoring TFLOP/s; `e2e` is
the same decode metric through the host-buffer entry points (copies timed);
`roofline` is the decode kernel against the measured HBM copy bandwidth;
`cpu_baseline` is the fp64 oracle timed on the host cores on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import torch  # noqa: E402

from paper_2407_20485_b200 import dist as a2dist  # noqa: E402
from paper_2407_20485_b200 import workloads as wl  # noqa: E402

METRIC = "a2sf_decode_step_hbm_gbps"
UNIT = "GB/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
# The ncu DRAM traffic of one decode launch is kept as a data line beside the launch-list summary,
# together with a hash of the kernel's sources at the time of the capture.
TRAFFIC_RECORD = ROOT / "profiles" / "launch_list_llama2_13b.md"


def ncu_decode_traffic(workload: str, batch: int):
    """dram__bytes_read.sum + dram__bytes_write.sum of one decode_step_stream_kernel launch from
    the committed ncu capture -- or None when there is no capture of this workload, or when any
    source of the kernel has changed since it was taken (a stale figure is not a measurement)."""
    import hashlib

    try:
        for line in TRAFFIC_RECORD.read_text().splitlines():
            if not line.startswith("bench-data:"):
                continue
            rec = json.loads(line[len("bench-data:"):])
            if rec.get("workload") != workload or rec.get("batch") != batch:
                continue
            for rel, digest in rec["sources"].items():
                if hashlib.sha256((ROOT / rel).read_bytes()).hexdigest() != digest:
                    return None
            return int(rec["dram_bytes_per_launch"])
    except (OSError, ValueError, KeyError):
        pass
    return None


def load_peaks():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        d = json.loads(f.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def __enter__(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0=None, t1=None):
        """Median SM clock and throttle reasons of the samples taken between the wall-clock
        instants t0 and t1 (datetime, local time; None = no bound)."""
        from datetime import datetime

        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.path or not os.path.exists(self.path):
            return out
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 10:
                continue
            try:
                ts = datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                if (t0 and ts < t0) or (t1 and ts > t1):
                    continue
                sm_v, mx_v = float(parts[2]), float(parts[3])
            except ValueError:
                continue
            sm.append(sm_v)
            mx.append(mx_v)
            for name, val in zip(names, parts[6:10]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            # the region is busy throughout: the median describes the clocks under load
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def cuda_events(n):
    return [torch.cuda.Event(enable_timing=True) for _ in range(n)]


def run_ours(args):
    from paper_2407_20485_b200 import binding as a2sf   # raises if the CUDA library is missing

    rank, local_rank, world = a2dist.init("nccl")
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    w = wl.WORKLOADS[args.workload]
    if args.batch:
        w = w.scaled(B=args.batch)
    T = args.decode_steps or w.steps
    # weak scaling: every rank owns a full per-GPU batch of a job world x as large
    wg = w.scaled(B=w.B * world, steps=T)
    b_range = a2dist.rank_batch_range(w.B, rank)
    q, k, v = wl.make_prompt_chunked(wg, dev, b_range=b_range)
    dq, dk, dv = wl.make_decode(wg, dev, t_range=(0, T), b_range=b_range)
    U, n, d = w.units, w.n, w.d
    p = a2sf.make_params(w.B, w.H, d, w.torch_dtype, w.budget, w.recent, w.alpha)
    m = min(n, w.budget)
    out = torch.empty_like(q)
    scores = torch.empty((w.B, w.H, n), dtype=torch.float32, device=dev)
    kept = torch.empty((w.B, w.H, m), dtype=torch.int32, device=dev)
    lse = torch.empty((w.B, w.H, n), dtype=torch.float32, device=dev)
    ws = torch.empty((max(256, a2sf.a2sf_prefill_workspace_bytes(p, n)),), dtype=torch.uint8, device=dev)
    cache = a2sf.Cache(p, dev)
    o_t = torch.empty((T, w.B, w.H, d), dtype=w.torch_dtype, device=dev)
    e_t = torch.empty((T, w.B, w.H), dtype=torch.int32, device=dev)

    # The T generation steps of a benchmark step are captured once in a CUDA graph (the calls hold
    # no host-side state; counts and lengths live on the device) and replayed: the same T launches
    # of the same kernel, without T round trips through the Python binding.
    decode_graph = None
    if not args.no_graph:
        a2sf.a2sf_prefill(p, q, k, v, out=out, scores=scores, kept_idx=kept, lse=lse, workspace=ws)
        cache.a2sf_cache_load(k, v, scores, kept)
        cache.a2sf_decode_step(w.alpha, dq[0], dk[0], dv[0], o_t[0], e_t[0])     # set-up outside the capture
        torch.cuda.synchronize()
        decode_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(decode_graph):
            for t in range(T):
                cache.a2sf_decode_step(w.alpha, dq[t], dk[t], dv[t], o_t[t], e_t[t])

    def step(ev=None):
        if ev: ev[0].record()
        a2sf.a2sf_prefill(p, q, k, v, out=out, scores=scores, kept_idx=kept, lse=lse, workspace=ws)
        if ev: ev[1].record()
        cache.a2sf_cache_load(k, v, scores, kept)
        if ev: ev[2].record()
        if decode_graph is not None:
            decode_graph.replay()
        else:
            for t in range(T):
                cache.a2sf_decode_step(w.alpha, dq[t], dk[t], dv[t], o_t[t], e_t[t])
        if ev: ev[3].record()

    from datetime import datetime

    # the sampler starts before the warm-up (nvidia-smi needs a moment to come up); only the
    # samples that fall inside the timed region are reported
    with ClockSampler(local_rank) as clk:
        for _ in range(args.warmup):
            step()
        torch.cuda.synchronize()
        a2dist.barrier()
        evs = [cuda_events(4) for _ in range(args.steps)]
        launches0 = a2sf.a2sf_kernel_launch_count()
        t_start = cuda_events(1)[0]
        t_end = cuda_events(1)[0]
        wall0 = datetime.now()
        t_start.record()
        for i in range(args.steps):
            step(evs[i])
        t_end.record()
        torch.cuda.synchronize()
        wall1 = datetime.now()
    a2dist.barrier()
    launches = a2sf.a2sf_kernel_launch_count() - launches0
    if decode_graph is not None:
        launches += args.steps * T          # the replayed launches do not pass through the library's counter
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK
    total_ms = t_start.elapsed_time(t_end)
    prefill_ms = sum(e[0].elapsed_time(e[1]) for e in evs)
    load_ms = sum(e[1].elapsed_time(e[2]) for e in evs)
    decode_ms = sum(e[2].elapsed_time(e[3]) for e in evs)
    clocks = clk.summary(wall0, wall1)

    # ---- the two prefill passes apart: the scoring pass + selection run alone from the saved lse
    # (a2sf_rescore); the attention pass is the rest of the prefill time measured above
    er = cuda_events(3)
    a2sf.a2sf_rescore(p, q, k, lse, scores=scores, kept_idx=kept)
    reps_r = 5
    er[0].record()
    for _ in range(reps_r):
        a2sf.a2sf_rescore(p, q, k, lse, scores=scores, kept_idx=kept)
    er[1].record()
    for _ in range(reps_r):       # the whole prefill under the same (short-run) clocks
        a2sf.a2sf_prefill(p, q, k, v, out=out, scores=scores, kept_idx=kept, lse=lse, workspace=ws)
    er[2].record()
    es_ = cuda_events(2)
    es_[0].record()
    for _ in range(reps_r):       # the selection (K3) alone, from the scores just written
        a2sf.a2sf_select(p, scores, kept_idx=kept)
    es_[1].record()
    torch.cuda.synchronize()
    rescore_ms = er[0].elapsed_time(er[1]) / reps_r
    prefill_short_ms = er[1].elapsed_time(er[2]) / reps_r
    select_ms = es_[0].elapsed_time(es_[1]) / reps_r

    # ---- separate line: the scoring pass without the rows whose forgetting weight is exactly
    # zero in fp32 (bit-identical scores, less work; NOT part of the headline step above)
    windowed = None
    if 0.0 < w.alpha < 1.0:
        import math
        pw = a2sf.make_params(w.B, w.H, d, w.torch_dtype, w.budget, w.recent, w.alpha,
                              flags=a2sf.A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS)
        s_ref = scores.clone()
        sw = torch.empty_like(scores)
        kw_ = torch.empty_like(kept)
        for _ in range(2):
            a2sf.a2sf_prefill(pw, q, k, v, out=out, scores=sw, kept_idx=kw_, lse=lse, workspace=ws)
        ew = cuda_events(2)
        reps = 5
        ew[0].record()
        for _ in range(reps):
            a2sf.a2sf_prefill(pw, q, k, v, out=out, scores=sw, kept_idx=kw_, lse=lse, workspace=ws)
        ew[1].record()
        torch.cuda.synchronize()
        span = math.ceil(127.0 / -math.log2(w.alpha))
        i_min = max(0, n - span)
        rows = sum(n - max(j, i_min) for j in range(n))          # (i, j) pairs with a non-zero weight
        windowed = {"ms_per_prefill": ew[0].elapsed_time(ew[1]) / reps,
                    "scores_bit_identical": bool(torch.equal(sw, s_ref)),
                    "window_rows": span,
                    "flops_per_prefill": U * (w.prefill_flops_per_unit()["pass1"] + 2 * d * rows)}
        del s_ref, sw, kw_

    # ---- separate line: the prompt pruned row by row (n launches of the step kernel) instead of
    # dense prefill + one selection; a different reading of the method, never part of the headline
    streamed = None
    if not args.no_streamed:
        sc_cache = a2sf.Cache(p, dev)
        ev_s = torch.empty((n, w.B, w.H), dtype=torch.int32, device=dev)
        sc_cache.a2sf_prefill_streaming(w.alpha, q, k, v, out=out, evicted=ev_s)      # warm-up
        es = cuda_events(2)
        es[0].record()
        sc_cache.a2sf_prefill_streaming(w.alpha, q, k, v, out=out, evicted=ev_s)
        es[1].record()
        torch.cuda.synchronize()
        ms = es[0].elapsed_time(es[1])
        # rows 0..M-1 read i slots, the rest M: bytes follow the step's formula with that row count
        eb = w.elem_bytes
        row_bytes = sum(U * (2 * min(i, w.budget) * d * eb + 12 * min(i, w.budget) + 6 * d * eb + 16)
                        for i in range(n))
        streamed = {"ms_per_prompt": ms, "rows": n, "us_per_row": ms * 1e3 / n,
                    "gbps": row_bytes / (ms * 1e-3) / 1e9,
                    "evictions_per_unit": int((ev_s[:, 0, 0] >= 0).sum().item())}
        sc_cache.close()
        del ev_s

    # ---- end to end through the host-buffer entry points (copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
        hout = torch.empty_like(hq).pin_memory()
        hs = torch.empty((w.B, w.H, n), dtype=torch.float32).pin_memory()
        hkept = torch.empty((w.B, w.H, m), dtype=torch.int32).pin_memory()
        hdq, hdk, hdv = (t.cpu().pin_memory() for t in (dq, dk, dv))
        ho = torch.empty((w.B, w.H, d), dtype=w.torch_dtype).pin_memory()
        he = torch.empty((w.B, w.H), dtype=torch.int32).pin_memory()
        del out
        hws = torch.empty((a2sf.a2sf_prefill_host_workspace_bytes(p, n),), dtype=torch.uint8, device=dev)
        strides = (w.H * n * d, n * d, d)

        def e2e_step():
            t0 = time.perf_counter()
            addr = a2sf.a2sf_prefill_host(p, n, hq, hk, hv, hout, hs, hkept, hws)
            cache.a2sf_cache_load(addr[0], addr[1], addr[2], addr[3], n=n, strides=strides)
            torch.cuda.synchronize()
            t1 = time.perf_counter()
            for t in range(T):
                cache.a2sf_decode_step_host(w.alpha, hdq[t], hdk[t], hdv[t], ho, he)
            t2 = time.perf_counter()
            return (t1 - t0) * 1e3, (t2 - t1) * 1e3

        ke = max(1, min(args.steps, args.e2e_steps))
        e2e_step()
        a2dist.barrier()
        res = [e2e_step() for _ in range(ke)]
        a2dist.barrier()
        e_pre = sum(r[0] for r in res) / ke
        e_dec = sum(r[1] for r in res) / ke
        eb = w.elem_bytes
        h2d = 3 * U * n * d * eb + T * 3 * U * d * eb
        d2h = U * n * d * eb + U * n * 4 + U * m * 4 + T * (U * d * eb + U * 4)
        e2e = {"pre_ms": e_pre, "dec_ms": e_dec, "h2d": h2d, "d2h": d2h, "steps": ke}

    # ---- combine over ranks ------------------------------------------------------------
    bytes_per_launch = U * w.decode_bytes_per_unit_step()
    flops = w.prefill_flops_per_unit()
    prefill_flops = U * (flops["pass1"] + flops["pass2"])
    total_units, max_total_ms = a2dist.job_throughput(U, total_ms, dev)
    max_decode_ms = a2dist.max_over_ranks(decode_ms, dev)
    max_prefill_ms = a2dist.max_over_ranks(prefill_ms, dev)
    max_load_ms = a2dist.max_over_ranks(load_ms, dev)
    scale_units = total_units / U                      # = world size
    K = args.steps
    value = scale_units * bytes_per_launch * T * K / (max_decode_ms * 1e-3) / 1e9
    prefill_tflops = scale_units * prefill_flops * K / (max_prefill_ms * 1e-3) / 1e12
    peaks = load_peaks()
    launch_us = decode_ms / (K * T) * 1e3
    achieved = bytes_per_launch / (launch_us * 1e-6) / 1e9
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": max_total_ms / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": {"bf16": "bf16", "fp16": "f16", "fp32": "f32"}[w.dtype],
        "data": "synthetic",
        "config": {"workload": f"{w.name} (config {w.index}): B{w.B} H{w.H} d{d} n{n} alpha{w.alpha} "
                               f"budget{w.budget} recent{w.recent} decode_steps{T} per GPU",
                   "l2": "inputs_larger_than_l2" if bytes_per_launch > 126e6 else "l2_resident_working_set",
                   "units_per_gpu": U, "step": "prefill+select+cache_load+decode_steps",
                   "decode_launches": "cuda_graph_replay" if decode_graph is not None else "one_call_per_step"},
        "phases_ms_per_step": {"prefill": max_prefill_ms / K, "cache_load": max_load_ms / K,
                               "decode": max_decode_ms / K},
        "prefill": {"metric": "prefill_scoring_tflops", "value": prefill_tflops, "unit": "TFLOP/s",
                    "flops_per_step": prefill_flops, "frac_of_measured_bf16_sustained":
                        prefill_tflops / scale_units / peaks["bf16_tflops_sustained"],
                    "frac_of_nominal_bf16": prefill_tflops / scale_units / NOMINAL["bf16_tflops"],
                    "passes": {
                        "scores_and_selection_ms": rescore_ms,
                        "scores_ms": rescore_ms - select_ms,
                        "selection_ms": select_ms,
                        "scores_tflops": U * flops["pass2"] / ((rescore_ms - select_ms) * 1e-3) / 1e12,
                        "prefill_ms": prefill_short_ms,
                        "attention_ms": prefill_short_ms - rescore_ms,
                        "attention_tflops": U * flops["pass1"] / ((prefill_short_ms - rescore_ms) * 1e-3) / 1e12,
                        "note": "this rank, 5 back-to-back repetitions after the timed region (shorter "
                                "run, higher clocks than inside it); K1 attention = prefill - (scores + "
                                "selection), includes the fp16 copy of V for bf16 storage; K2 scores = "
                                "a2sf_rescore - a2sf_select; K3 selection = a2sf_select; K4 = "
                                "phases_ms_per_step.cache_load"},
                    "roofline": prefill_roofline(w, U, prefill_tflops / scale_units, max_prefill_ms / K, peaks,
                                                 clocks.get("sm_mhz"))},
        "roofline": {"kernel": "decode_step_stream_kernel", "bound": "hbm", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "frac_of_nominal_8TBps": achieved / NOMINAL["hbm_gbs"],
                     "traffic": ncu_decode_traffic(w.name, w.B), "bytes_per_launch": bytes_per_launch, "launch_us": launch_us},
        "prefill_zero_weight_rows_skipped": windowed,
        "prefill_streamed_row_by_row": streamed,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if e2e is not None:
        e_dec = a2dist.max_over_ranks(e2e["dec_ms"], dev)
        e_pre = a2dist.max_over_ranks(e2e["pre_ms"], dev)
        result["e2e"] = {"value": scale_units * bytes_per_launch * T / (e_dec * 1e-3) / 1e9, "unit": UNIT,
                         "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                         "ms_per_step": e_pre + e_dec, "prefill_ms": e_pre, "decode_ms": e_dec,
                         "steps": e2e["steps"]}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(w, T, q, k, v, dq, dk, dv)
    cache.close()
    if rank == 0 and world == 1 and not args.no_rotation:
        # the other stated workloads: their one-layer caches fit in L2, so they are also
        # stepped as a rotation over the named model's layer count (not part of the headline)
        result["decode_layer_rotation"] = [
            decode_layer_rotation(a2sf, dev, name, layers, args.rotation_steps, args.rotation_reps)
            for name, layers in (("llama2_7b", 32), ("opt_6p7b", 32), ("long_context", 32),
                                 ("llama2_13b", 1))]          # the headline workload, graph-replayed
    if rank == 0 and world == 1 and not args.no_grouped:
        # grouped query heads (not part of the headline): the same policy on 8 K/V heads per row
        result["decode_grouped"] = [decode_grouped(a2sf, dev, G, 8, args.rotation_steps, args.rotation_reps)
                                    for G in (4, 8)]
        # the same step at five times the batch: 1280 units, 345 MB per launch, several rounds of CTAs
        result["decode_grouped"] += [decode_grouped(a2sf, dev, G, 1, args.rotation_steps, args.rotation_reps, B=160)
                                     for G in (4, 8)]
    if rank == 0:
        print(json.dumps(result))
    a2dist.finalize()


def prefill_roofline(w, U, tflops, ms, peaks, sm_mhz):
    """The prefill against its two ceilings.  Tensor: the causal flops at the measured sustained
    and the nominal dense bf16 rate.  Special-function unit: the two passes evaluate one exp2 per
    logit of every 128x128 tile they touch (diagonal tiles in full), and an SM retires 16 of them
    per clock (measured: 15.8 per clock with the multiply-add and add of the scoring loop around
    them).  The kernels overlap the two only partly, so the time is compared with each and with
    their sum."""
    T = (w.n + 127) // 128
    tiles = U * T * (T + 1) // 2
    exps = 2 * tiles * 128 * 128
    mhz = sm_mhz or 1800.0
    sfu_ms = exps / (16.0 * 148 * mhz * 1e6) * 1e3
    fl = w.prefill_flops_per_unit()
    tensor_ms = U * (fl["pass1"] + fl["pass2"]) / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    return {"bound": "tensor", "achieved": tflops, "unit": "TFLOP/s",
            "peak": peaks["bf16_tflops_sustained"], "peak_source": peaks["source"] + " (sustained bf16)",
            "frac": tflops / peaks["bf16_tflops_sustained"],
            "peak_nominal": NOMINAL["bf16_tflops"], "frac_of_nominal": tflops / NOMINAL["bf16_tflops"],
            "ms": ms, "tensor_ms_at_measured_sustained": tensor_ms,
            "sfu_exp2_count": exps, "sfu_ms_at_16_per_clk_per_sm": sfu_ms, "sfu_clock_mhz": mhz,
            "tensor_plus_sfu_ms": tensor_ms + sfu_ms}


def decode_grouped(a2sf, dev, G, layers, steps, reps, B=None):
    """Grouped-query decode step (G query heads per K/V head, one pruned cache per K/V head) on the
    headline workload's policy with 8 K/V heads per batch row: 256 units x 512 slots, 69 MB per
    launch.  Timed like `decode_layer_rotation`: one layer (fits in L2) and `layers` caches stepped
    round-robin (larger than L2), `steps` x layers launches replayed from a CUDA graph."""
    w = wl.WORKLOADS["llama2_13b"].scaled(H=8, n=1024, **({"B": B} if B else {}))
    wq = w.scaled(H=w.H * G)
    q = wl.make_prompt(wq, dev)[0]
    _, k, v = wl.make_prompt(w, dev)
    dq = wl.make_decode(wq, dev, t_range=(0, steps))[0]
    _, dk, dv = wl.make_decode(w, dev, t_range=(0, steps))
    p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha)
    _, S, kept, _ = a2sf.a2sf_prefill_group(p, G, q, k, v)
    del q
    # K and V once per unit, whatever the group size; the G query and output rows on top
    bytes_per_launch = w.units * (w.decode_bytes_per_unit_step() + (G - 1) * 2 * w.d * 2)
    res = {"workload": f"B{w.B} Hkv{w.H} group{G} d{w.d} alpha{w.alpha} budget{w.budget} recent{w.recent} bf16",
           "bytes_per_launch": bytes_per_launch, "steps_per_replay": steps, "repetitions": reps}
    for L in sorted({1, layers}):
        caches = [a2sf.Cache(p, dev) for _ in range(L)]
        o = torch.empty((L, w.B, w.H * G, w.d), dtype=w.torch_dtype, device=dev)
        e = torch.empty((L, w.B, w.H), dtype=torch.int32, device=dev)

        def restore():
            for c in caches:
                c.a2sf_cache_load(k, v, S, kept)

        def run():
            for t in range(steps):
                for l, c in enumerate(caches):
                    c.a2sf_decode_step_group(G, w.alpha, dq[t], dk[t], dv[t], o[l], e[l])

        restore(); run()                        # kernel attributes are set outside the capture
        torch.cuda.synchronize()
        restore()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            run()
        times = []
        for _ in range(reps):
            restore()
            ev = cuda_events(2)
            ev[0].record(); g.replay(); ev[1].record()
            torch.cuda.synchronize()
            times.append(ev[0].elapsed_time(ev[1]) * 1e3 / (steps * L))      # us per launch
        assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK
        med, best = statistics.median(times), min(times)
        res["layers_%d" % L] = {
            "working_set_mb": L * bytes_per_launch / 1e6,
            "l2": "larger_than_l2" if L * bytes_per_launch > 126e6 else "l2_resident",
            "us_per_launch_median": med, "us_per_launch_min": best,
            "gbps_median": bytes_per_launch / med / 1e3, "gbps_max": bytes_per_launch / best / 1e3}
        del g
        for c in caches:
            c.close()
    return res


def decode_layer_rotation(a2sf, dev, name, layers, steps, reps):
    """Decode-step timing for a workload whose single-layer cache fits in L2: `layers`
    independent cache instances (the layer count of the named model) are stepped round-robin, so
    the working set is what one generation step of the whole model touches.  `steps` x `layers`
    launches are captured once in a CUDA graph; each repetition restores every cache (untimed)
    and times one replay with CUDA events.  Also run with one layer (L2-resident) for contrast."""
    w = wl.WORKLOADS[name]
    q, k, v = wl.make_prompt_chunked(w, dev)
    dq, dk, dv = wl.make_decode(w, dev, t_range=(0, steps))
    p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha)
    _, S, kept, _ = a2sf.a2sf_prefill(p, q, k, v)
    del q
    bytes_per_launch = w.units * w.decode_bytes_per_unit_step()
    res = {"workload": f"{w.name} (config {w.index}): B{w.B} H{w.H} d{w.d} n{w.n} alpha{w.alpha} "
                       f"budget{w.budget} recent{w.recent}",
           "bytes_per_launch": bytes_per_launch, "steps_per_replay": steps, "repetitions": reps,
           "timing": "one CUDA-graph replay of steps x layers launches between two events"}
    for L in sorted({1, layers}):
        caches = [a2sf.Cache(p, dev) for _ in range(L)]
        o = torch.empty((L, w.B, w.H, w.d), dtype=w.torch_dtype, device=dev)
        e = torch.empty((L, w.B, w.H), dtype=torch.int32, device=dev)

        def restore():
            for c in caches:
                c.a2sf_cache_load(k, v, S, kept)

        def run():
            for t in range(steps):
                for l, c in enumerate(caches):
                    c.a2sf_decode_step(w.alpha, dq[t], dk[t], dv[t], o[l], e[l])

        restore(); run()                        # lazy initialisation happens outside the capture
        torch.cuda.synchronize()
        restore()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            run()
        times = []
        for _ in range(reps):
            restore()
            ev = cuda_events(2)
            ev[0].record(); g.replay(); ev[1].record()
            torch.cuda.synchronize()
            times.append(ev[0].elapsed_time(ev[1]) * 1e3 / (steps * L))      # us per launch
        assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK
        med, best = statistics.median(times), min(times)
        res["layers_%d" % L] = {
            "working_set_mb": L * bytes_per_launch / 1e6,
            "l2": "larger_than_l2" if L * bytes_per_launch > 126e6 else "l2_resident",
            "us_per_launch_median": med, "us_per_launch_min": best,
            "gbps_median": bytes_per_launch / med / 1e3, "gbps_max": bytes_per_launch / best / 1e3}
        del g
        for c in caches:
            c.close()
    return res


def oracle_sample(w, units_sel, dsteps, q, k, v, dq, dk, dv, threads):
    """Times the oracle, as it stands, on the listed units: prefill + `dsteps` decode steps."""
    import numpy as np

    import oracle

    ub = [(u // w.H, u % w.H) for u in units_sel]
    f64 = lambda t: t.detach().cpu().to(torch.float64).numpy()
    Q = np.stack([f64(q[b, h]) for b, h in ub])
    K = np.stack([f64(k[b, h]) for b, h in ub])
    V = np.stack([f64(v[b, h]) for b, h in ub])
    t0 = time.perf_counter()
    ref = oracle.prefill(Q, K, V, w.scale, [w.alpha], w.budget, w.recent, nthreads=threads)
    t1 = time.perf_counter()
    oc = oracle.Cache(len(ub), w.d, w.budget, w.recent, w.scale)
    oc.load(K, V, ref["S"][:, 0], ref["kept"])
    ins = [[np.stack([f64(x[t, b, h]) for b, h in ub]) for x in (dq, dk, dv)] for t in range(dsteps)]
    t2 = time.perf_counter()
    for t in range(dsteps):
        oc.step(*ins[t], w.alpha, nthreads=threads)
    t3 = time.perf_counter()
    return t1 - t0, t3 - t2, ref["threads"]


def cpu_baseline(w, T, q, k, v, dq, dk, dv):
    import oracle

    threads = oracle.host_threads()
    # bounded sample: one unit per host thread; decode steps capped
    n_units = min(w.units, threads)
    dsteps = min(T, 64)
    units_sel = [int(i * (w.units - 1) / max(1, n_units - 1)) for i in range(n_units)] if n_units > 1 else [0]
    pre_s, dec_s, used = oracle_sample(w, units_sel, dsteps, q, k, v, dq, dk, dv, threads)
    flops = w.prefill_flops_per_unit()
    return {"value": n_units * dsteps * w.decode_bytes_per_unit_step() / dec_s / 1e9, "unit": UNIT,
            "cores": int(used), "kind": "oracle",
            "sample": f"{n_units} of {w.units} units: prefill n={w.n} ({pre_s:.2f} s) + {dsteps} decode steps "
                      f"({dec_s:.3f} s), fp64",
            "prefill_tflops": n_units * (flops["pass1"] + flops["pass2"]) / pre_s / 1e12,
            "prefill_units_per_s": n_units / pre_s, "decode_unit_steps_per_s": n_units * dsteps / dec_s}


def run_reference(args):
    """The reference arm: the fp64 oracle on the host cores, a bounded sample per step."""
    rank, _, world = a2dist.env_world()
    if rank != 0:
        return
    import oracle

    w = wl.WORKLOADS[args.workload]
    if args.batch:
        w = w.scaled(B=args.batch)
    T = args.decode_steps or w.steps
    threads = oracle.host_threads()
    n_units = min(w.units, threads)
    dsteps = min(T, 32)
    units_sel = [int(i * (w.units - 1) / max(1, n_units - 1)) for i in range(n_units)] if n_units > 1 else [0]
    bsel = sorted({u // w.H for u in units_sel})
    # generate only the sampled units' inputs (coordinate-addressed generator)
    qs, ks, vs, dqs, dks, dvs = {}, {}, {}, {}, {}, {}
    for u in units_sel:
        b, h = u // w.H, u % w.H
        a, b_, c = wl.make_prompt(w, "cpu", (b, b + 1), (h, h + 1))
        qs[u], ks[u], vs[u] = a[0, 0], b_[0, 0], c[0, 0]
        a, b_, c = wl.make_decode(w, "cpu", (0, dsteps), (b, b + 1), (h, h + 1))
        dqs[u], dks[u], dvs[u] = a[:, 0, 0], b_[:, 0, 0], c[:, 0, 0]
    w1 = w.scaled(B=1, H=n_units)
    q = torch.stack([qs[u] for u in units_sel])[None]
    k = torch.stack([ks[u] for u in units_sel])[None]
    v = torch.stack([vs[u] for u in units_sel])[None]
    dq = torch.stack([dqs[u] for u in units_sel], 1)[:, None]
    dk = torch.stack([dks[u] for u in units_sel], 1)[:, None]
    dv = torch.stack([dvs[u] for u in units_sel], 1)[:, None]
    sel = list(range(n_units))
    pre, dec, used = [], [], threads
    for i in range(args.warmup + args.steps):
        ps, ds, used = oracle_sample(w1, sel, dsteps, q, k, v, dq, dk, dv, threads)
        if i >= args.warmup:
            pre.append(ps)
            dec.append(ds)
    K = args.steps
    value = n_units * dsteps * K * w.decode_bytes_per_unit_step() / sum(dec) / 1e9
    sample = (f"{n_units} of {w.units} units per step: prefill n={w.n} + {dsteps} of {T} decode steps, fp64 "
              f"oracle, {used} threads")
    flops = w.prefill_flops_per_unit()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": args.warmup, "ms_per_step": (sum(pre) + sum(dec)) / K * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name} (config {w.index}): B{w.B} H{w.H} d{w.d} n{w.n} alpha{w.alpha} "
                               f"budget{w.budget} recent{w.recent} decode_steps{T} per GPU",
                   "sample": sample},
        "prefill": {"metric": "prefill_scoring_tflops", "unit": "TFLOP/s",
                    "value": n_units * K * (flops["pass1"] + flops["pass2"]) / sum(pre) / 1e12},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(used), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_13b", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--decode-steps", type=int, default=0, help="override T (0 = the workload's)")
    ap.add_argument("--batch", type=int, default=0, help="override the per-GPU batch (0 = the workload's); "
                    "smaller cases for profiler captures")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch the generation steps one call at a time instead of replaying a CUDA graph")
    ap.add_argument("--no-streamed", action="store_true",
                    help="skip the separate timing of the row-by-row streamed prompt")
    ap.add_argument("--no-rotation", action="store_true",
                    help="skip the layer-rotation decode timing of the L2-resident workloads")
    ap.add_argument("--no-grouped", action="store_true", help="skip the grouped-query decode timing")
    ap.add_argument("--rotation-steps", type=int, default=16, help="decode steps per graph replay")
    ap.add_argument("--rotation-reps", type=int, default=10)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
