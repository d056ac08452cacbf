#!/usr/bin/env python
"""Benchmark of the SJD hot path: committed image tokens per second.

One "step" = one SJD iteration (window forward pass against the KV cache, fused verify-and-resample,
window slide) of the 7B-shaped decoder (32 layers, d 4096, 32 heads, SwiGLU 11008, vocab 65536, bf16,
random init), batch 1, W = 32, top-k 2000, prompt 64.  Inputs are synthetic and seeded.

  python bench.py --gpus N --steps K --warmup W            # this library (N > 1: under torchrun)
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle on the host cores

Prints ONE JSON line.  `value` is device-timed with everything resident in HBM (median of at least five
blocks of K steps); `e2e` goes through the C-ABI with pinned host buffers for the prompt (copied in) and
the step results (written out) and a host read of the results every step; `roofline` is the
weight-streaming GEMM (the dominant kernel) against the measured HBM copy bandwidth; `kernels` holds the
isolated verification kernel and the window attention against the same bandwidth; `cpu_baseline` is the
oracle timed on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "committed_image_tokens_per_sec"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# DRAM traffic of the dominant kernel (gemm_tc_kernel) from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum) of the four projection launches of one decoder layer inside a step: 409.76 MB read +
# written for 404.75 MB of weights.  Traffic grows in proportion to the weight bytes of a launch, so a step's
# launches scale by that ratio.  Valid only for the kernel source the counters were taken with.
GEMM_TRAFFIC = {"source_sha256_16": "7a7d0504b4d33207", "dram_bytes_per_weight_byte": 409.76 / 404.75}


def gemm_traffic_per_launch(algorithmic_bytes_per_launch):
    import hashlib
    path = os.path.join(ROOT, "paper_2410_01699_b200", "csrc", "gemm_tc.cu")
    try:
        with open(path, "rb") as f:
            same = hashlib.sha256(f.read()).hexdigest()[:16] == GEMM_TRAFFIC["source_sha256_16"]
    except OSError:
        same = False
    return algorithmic_bytes_per_launch * GEMM_TRAFFIC["dram_bytes_per_weight_byte"] if same else None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["source"] = "measured"
        d.setdefault("bf16_tflops_sustained", d.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
        return d
    return dict(FALLBACK_PEAKS)


# ------------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            parts = [p.strip() for p in s.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# the oracle on the host cores (reference arm and cpu_baseline leg)
# ------------------------------------------------------------------------------------------------
def oracle_sample(wl, steps: int, warmup: int, tokens_per_step: float | None):
    """Times oracle SJD iterations on a bounded sample of the workload: the same window (W rows
    against the pre-filled prompt) through ONE of the n_layers decoder layers plus the lm_head and
    the full verification, then scales the time by streamed-parameter count to the full depth."""
    import numpy as np
    import torch

    from oracle.model import OracleModel
    from oracle.sjd import CachedModel, SampleCfg, sjd_begin, sjd_step
    from paper_2410_01699_b200.inputs import make_prompt, make_weights
    from tests.parity_util import oracle_model_cfg

    cores = len(os.sched_getaffinity(0))
    torch.set_num_threads(cores)
    sample_wl = wl.with_(n_layers=1)
    weights = make_weights(sample_wl)
    model = CachedModel(OracleModel(oracle_model_cfg(sample_wl), weights), wl.prompt_len + wl.n_generate + 1,
                        kv_storage=wl.dtype)
    scfg = SampleCfg(wl.temperature, wl.top_k, wl.philox_seed, wl.window, 0, wl.grid_stride, wl.n_generate, wl.dtype)
    prompt = [int(t) for t in make_prompt(wl, 1)[0]]
    model.prefill(prompt)
    st = sjd_begin(prompt, scfg, wl.vocab)
    times, committed = [], 0
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        rec = sjd_step(st, model, scfg, wl.vocab)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
            committed += len(rec.committed)
    t_sample = float(np.mean(times))
    # the part that does not scale with depth (embedding, lm_head, verification): the same
    # iteration on a zero-layer model
    head_wl = wl.with_(n_layers=0)
    head = CachedModel(OracleModel(oracle_model_cfg(head_wl), dict(weights, layers=[])), wl.prompt_len + wl.n_generate + 1,
                       kv_storage=wl.dtype)
    head.prefill(prompt)
    st0 = sjd_begin(prompt, scfg, wl.vocab)
    t0 = time.perf_counter()
    sjd_step(st0, head, scfg, wl.vocab)
    t_head = time.perf_counter() - t0
    t_layer = max(t_sample - t_head, 0.0)
    t_full = t_layer * wl.n_layers + t_head
    tps = tokens_per_step if tokens_per_step else committed / max(1, len(times))
    return {"value": tps / t_full, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": ("%d oracle SJD iterations (W=%d rows, prompt %d) of 1 of %d layers + lm_head + verification: "
                       "%.2f s each; layer part scaled x%d to full depth => %.1f s per iteration (extrapolated); "
                       "%.3f committed tokens per iteration" %
                       (len(times), wl.window, wl.prompt_len, wl.n_layers, t_sample, wl.n_layers, t_full, tps)),
            "seconds_per_step_full_depth": t_full}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 8))
    warm = max(0, min(args.warmup, 1))
    t0 = time.perf_counter()
    res = oracle_sample(wl, steps, warm, None)
    line = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["seconds_per_step_full_depth"] * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, 1), "gpu_launches": 0,
            "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "note": "CPU oracle (fp64, numpy); timed steps capped at %d; wall %.0f s" % (steps, time.perf_counter() - t0)}
    print(json.dumps(line), flush=True)


def workload_config(wl, batch_per_gpu):
    return {"workload": "7B-shaped decoder, one SJD iteration per step (7B Llama-style decoder, W=32, top-k 2000, batch 1)", "name": wl.name,
            "n_layers": wl.n_layers, "d_model": wl.d_model, "n_heads": wl.n_heads, "n_kv_heads": wl.n_kv_heads,
            "ffn_hidden": wl.ffn_hidden, "vocab": wl.vocab, "prompt_len": wl.prompt_len, "n_generate": wl.n_generate,
            "window": wl.window, "top_k": wl.top_k, "temperature": wl.temperature, "init": "random",
            "batch_per_gpu": batch_per_gpu, "parallelism": "independent sequences per GPU, no collective",
            "l2": "inputs (13.5 GB of weights per step) exceed L2; no flush needed"}


# ------------------------------------------------------------------------------------------------
# this library
# ------------------------------------------------------------------------------------------------
def kernel_points(peaks):
    """The isolated verification kernel and the window attention on the workloads their roofline bars are
    stated on, timed through the C-ABI in this same run (CUDA events on the launching stream, buffers
    rotating through more than the L2 cache): algorithmic bytes, microseconds, GB/s and the fraction of
    the measured HBM copy bandwidth."""
    from paper_2410_01699_b200 import microbench as mb
    pts = {}

    def put(name, res, gbs_key, nbytes):
        pts[name] = {"algorithmic_bytes": nbytes, "us": res["us"], "GBps": res[gbs_key],
                     "frac": res[gbs_key] / peaks["hbm_gbs"], "peak_source": "of " + peaks["source"]}

    for b in (32, 16):
        r = mb.bench_verify(b, 32, 16384, 2000, iters=60)
        put("verify_b%d_w32_v16384_k2000" % b, r, "logits_GBps", 2 * b * 32 * 16384 * 2)
    for b, prefix in ((8, 4000), (1, 2300)):
        r = mb.bench_attention(b, 32, prefix, 32, 32, 128, iters=60)
        put("attention_b%d_w32_n%d_h32x128" % (b, prefix + 32), r, "kv_GBps", b * 2 * 32 * (prefix + 32) * 128 * 2)
    return pts


def run_library(args, wl):
    import statistics

    import torch
    import torch.distributed as dist

    from paper_2410_01699_b200 import binding as B
    from paper_2410_01699_b200.inputs import make_prompt, make_weights
    from paper_2410_01699_b200.sharding import shard_sequences

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    batch = args.batch                                   # images per GPU
    streams = 2 if args.guidance != 0.0 else 1           # classifier-free guidance: two sequences per image
    seq_base, _ = shard_sequences(batch * world, world, rank)

    weights = make_weights(wl, device=dev)
    max_seq = wl.prompt_len + wl.n_generate + 8
    kv_pages = batch * streams * (-(-(wl.prompt_len + wl.n_generate) // 64)) if args.paged_kv else 0
    ctx = B.Context(B.make_model_cfg(wl, batch * streams, max_seq, wl.window, kv_pages=kv_pages), weights, device=dev)
    sample = B.make_sample_cfg(wl.temperature, wl.top_k, wl.philox_seed, wl.window, B.SJD_INIT_RANDOM,
                               wl.grid_stride, wl.n_generate, seq_base=seq_base, guidance=args.guidance)
    prompt_host = torch.from_numpy(make_prompt(wl, batch * streams * world)[seq_base * streams:(seq_base + batch) * streams]
                                   .copy()).pin_memory()
    prompt_dev = prompt_host.to(dev)
    out_dev = B.StepOut(batch, wl.window, device=dev)
    stream = torch.cuda.current_stream()
    total_tokens = wl.prompt_len + wl.n_generate

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def all_max(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def all_sum(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.int64, device=dev)
        dist.all_reduce(t)
        return int(t.item())

    # ---- warm-up: the requested steps, then more until at least WARM_SECONDS have gone by in total (the
    # first replays of the two step graphs and the clock ramp are slower than the steady state)
    WARM_SECONDS = 0.3
    ctx.prefill(prompt_dev, sample)
    info = ctx.info()
    t_warm = time.perf_counter()
    warm_run = 0
    while warm_run < max(3, args.warmup) or time.perf_counter() - t_warm < WARM_SECONDS:
        ctx.step(out_dev)
        warm_run += 1
        if warm_run % 4 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    warm_seconds = time.perf_counter() - t_warm

    # ---- device-resident timing: blocks of K steps enqueued back to back with no host round trip, each
    # block bracketed by a barrier + synchronize and timed with CUDA events; at least 5 blocks and at
    # least about a second in total.  ms_per_step is the median block (min and max beside it).
    clocks = ClockSampler(local)
    clocks.start()
    launches0 = B.sjd_launch_count()
    committed_acc = torch.zeros(batch, dtype=torch.int64, device=dev)
    block_ms, blocks_wanted, steps_timed = [], 5, 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    while len(block_ms) < blocks_wanted:
        # enough of the image left for this block even if every draft of every step were accepted?  else start over
        n_now = int(out_dev.total_committed.max().item())
        if n_now + args.steps * wl.window >= total_tokens and n_now + 2 * args.steps >= total_tokens:
            ctx.prefill(prompt_dev, sample)
            for _ in range(4):
                ctx.step(out_dev)
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            ctx.step(out_dev)
            committed_acc += out_dev.n_committed  # device-side add of the step's result, no sync
        e1.record(stream)
        barrier()
        block_ms.append(all_max(e0.elapsed_time(e1)))
        steps_timed += args.steps
        if len(block_ms) == blocks_wanted and sum(block_ms) < 1000.0 and blocks_wanted < 50:
            blocks_wanted += 1
    launches = B.sjd_launch_count() - launches0
    clk = clocks.stop()
    tokens = all_sum(int(committed_acc.sum().item()))
    assert ctx.device_status() == B.SJD_OK
    # tokens fixed per step and sequence over every timed step (a property of the seeded run, not of its
    # speed); throughput = that rate over the median block's time per step
    tokens_per_step = tokens / (steps_timed * batch * world)
    ms_per_step = statistics.median(block_ms) / args.steps
    value = tokens_per_step * batch * world / (ms_per_step * 1e-3)

    # ---- per-kernel-class device time (separate traced steps, CUDA events on the launching stream)
    trace_steps = max(3, min(10, args.steps))
    ctx.trace(True)
    for _ in range(trace_steps):
        ctx.step(out_dev)
    tr = ctx.trace_read()
    ctx.trace(False)
    peaks = measured_peaks()
    gemm_ms_per_launch = tr["ms"]["gemm"] / max(1, tr["launches"]["gemm"])
    achieved = tr["gemm_weight_bytes"] / (tr["ms"]["gemm"] * 1e-3) / 1e9 if tr["ms"]["gemm"] > 0 else 0.0
    rows = batch * streams * wl.window
    roofline = {"bound": "hbm", "kernel": "projection GEMMs (weight streaming, M = %d rows)" % rows,
                "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                "peak_source": "of " + peaks["source"], "nominal_peak": 8000.0, "frac_of_nominal": achieved / 8000.0,
                "traffic": gemm_traffic_per_launch(tr["gemm_weight_bytes"] / max(1, tr["launches"]["gemm"])),
                "algorithmic_bytes_per_launch": tr["gemm_weight_bytes"] / max(1, tr["launches"]["gemm"]),
                "algorithmic_bytes_per_step": tr["gemm_weight_bytes"] / trace_steps,
                "launches_per_step": tr["launches"]["gemm"] / trace_steps, "avg_launch_ms": gemm_ms_per_launch,
                "step_ms_by_class": {k: v / trace_steps for k, v in tr["ms"].items()},
                "whole_step_frac": wl.step_weight_bytes() / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    if rows > 128:
        # many rows: the projections are bound by the tensor pipe.  Useful flops = 2 * rows * weights;
        # the kernel multiplies both bf16 planes of the activations, i.e. issues twice that.
        flops = 2.0 * rows * (tr["gemm_weight_bytes"] / 2.0)
        tf = flops / (tr["ms"]["gemm"] * 1e-3) / 1e12 if tr["ms"]["gemm"] > 0 else 0.0
        roofline.update({"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": tf / peaks["bf16_tflops_sustained"], "issued_frac": 2.0 * tf / peaks["bf16_tflops_sustained"],
                         "nominal_peak": 2250.0, "frac_of_nominal": tf / 2250.0,
                         "weight_GBps": achieved,
                         "note": "achieved counts each product once; the tensor pipe runs two MMAs per product "
                                 "(hi and lo plane of the fp32 activations): issued_frac is its utilisation"})

    # ---- end to end through the C-ABI with host buffers: every step the host hands the library pinned
    # host buffers for the results, waits for the step and reads them; the prompt is copied in from pinned
    # host memory and pre-filled inside the timed region.  Same number of steps per block as above; the
    # rate of tokens per step is the one measured above (it does not depend on which leg runs).
    out_host = B.StepOut(batch, wl.window, pinned=True)
    e2e_steps = args.steps
    e2e_blocks = []
    for _ in range(3):
        barrier()
        t0 = time.perf_counter()
        prompt_dev.copy_(prompt_host, non_blocking=True)
        ctx.prefill(prompt_dev, sample)
        seen = 0
        for _ in range(e2e_steps):
            ctx.step(out_host)
            stream.synchronize()
            seen += int(out_host.n_committed.sum())
        torch.cuda.synchronize()
        e2e_blocks.append(all_max(time.perf_counter() - t0))
    e2e_s = statistics.median(e2e_blocks)
    out_bytes = sum(getattr(out_host, n).numel() * 4 for n in ("n_accepted", "n_committed", "committed", "draft",
                                                                "q_kind", "q_draft", "total_committed", "flags"))
    e2e = {"value": tokens_per_step * batch * world * e2e_steps / e2e_s, "unit": UNIT,
           "h2d_bytes_per_step": prompt_host.numel() * 4 / e2e_steps, "d2h_bytes_per_step": out_bytes,
           "ms_per_step": e2e_s / e2e_steps * 1e3,
           "note": "median of 3 blocks of %d steps, each with the copy and pre-fill of the %d-token prompt inside; "
                   "the host waits for and reads every step's results" % (e2e_steps, wl.prompt_len)}

    kernels = None
    if rank == 0 and world == 1 and not args.no_kernel_points:
        kernels = kernel_points(peaks)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_sample(wl, 2, 1, tokens_per_step)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": dict(workload_config(wl, batch), guidance=args.guidance, rows_per_step=rows, kv_cache="paged-64" if args.paged_kv else "contiguous"),
                "clocks": clk, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "kernels": kernels,
                "cpu_baseline": cpu,
                "timing": {"blocks": len(block_ms), "steps_per_block": args.steps,
                           "ms_per_step_min": min(block_ms) / args.steps, "ms_per_step_max": max(block_ms) / args.steps,
                           "warmup_steps_run": warm_run, "warmup_seconds": warm_seconds},
                "pipeline": info,
                "sjd": {"committed_tokens_per_step": tokens_per_step,
                        "steps_per_image_est": wl.n_generate / tokens_per_step if tokens_per_step else None,
                        "step_floor_ms_at_measured_hbm": wl.step_weight_bytes() / (peaks["hbm_gbs"] * 1e9) * 1e3}}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_table(args, wl):
    """The structure of the paper's Table 1 (rows A-D) and of its no-refinement ablation on this library's
    kernels: whole images generated by next-token sampling (A: window 1), Jacobi decoding with the
    deterministic criterion (B), SJD with random initialisation (C), SJD with the spatial prior (D: token
    one grid row above) and SJD without refinement; forward passes per image, latency, ratios against A.
    Random-init weights accept almost nothing, so the ratios say nothing about trained models."""
    import torch

    from paper_2410_01699_b200 import binding as B
    from paper_2410_01699_b200.inputs import make_prompt, make_weights

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    weights = make_weights(wl, device=dev)
    n_gen = args.n_generate or wl.n_generate
    max_seq = wl.prompt_len + n_gen + 8
    prompt = torch.from_numpy(make_prompt(wl, 1)).to(dev)
    ctx = B.Context(B.make_model_cfg(wl, 1, max_seq, wl.window), weights, device=dev)
    rows = [("A", "next-token sampling (window 1)", 1, B.SJD_SCHEDULE_SJD, B.SJD_INIT_RANDOM),
            ("B", "Jacobi decoding, unchanged-token criterion", wl.window, B.SJD_SCHEDULE_JACOBI, B.SJD_INIT_RANDOM),
            ("C", "SJD, random initialisation", wl.window, B.SJD_SCHEDULE_SJD, B.SJD_INIT_RANDOM),
            ("D", "SJD, token one grid row above", wl.window, B.SJD_SCHEDULE_SJD, B.SJD_INIT_COPY_ABOVE),
            ("no-refinement", "SJD without Eq. 3", wl.window, B.SJD_SCHEDULE_NO_REFINE, B.SJD_INIT_RANDOM)]
    table, chunk = [], 64
    for tag, name, window, schedule, init in rows:
        sample = B.make_sample_cfg(wl.temperature, wl.top_k, wl.philox_seed, window, init, wl.grid_stride, n_gen,
                                   schedule=schedule)
        out = B.StepOut(1, window, device=dev)
        ctx.prefill(prompt, sample)
        for _ in range(4):   # first replays of freshly captured step graphs
            ctx.step(out)
        ctx.prefill(prompt, sample)
        busy = torch.zeros(1, dtype=torch.int64, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        run = 0
        while True:
            for _ in range(chunk):
                ctx.step(out)
                busy += (out.n_committed > 0).to(torch.int64)   # device-side count of passes that fixed a token
            run += chunk
            if int(out.total_committed.item()) >= wl.prompt_len + n_gen:
                break
        e1.record()
        torch.cuda.synchronize()
        steps = int(busy.item())
        ms = e0.elapsed_time(e1) * steps / run     # passes after the image is complete are not counted
        table.append({"row": tag, "config": name, "window": window, "steps_per_image": steps,
                      "tokens_per_step": n_gen / steps, "latency_s": ms * 1e-3, "ms_per_step": ms / steps})
    base = table[0]
    for r in table:
        r["step_ratio_vs_A"] = base["steps_per_image"] / r["steps_per_image"]
        r["latency_ratio_vs_A"] = base["latency_s"] / r["latency_s"]
    print(json.dumps({"table": table, "workload": wl.name, "n_generate": n_gen, "data": "synthetic",
                      "note": "random-init weights: acceptance statistics are not those of a trained model"}), flush=True)


def _spawned_rank(local_rank, args, wl, port):
    os.environ.update({"RANK": str(local_rank), "LOCAL_RANK": str(local_rank), "WORLD_SIZE": str(args.gpus),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    run_library(args, wl)


def launch_ranks(args, wl):
    """`python bench.py --gpus N` without a launcher: start the N ranks here, one process per GPU."""
    import socket

    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_spawned_rank, args=(args, wl, port), nprocs=args.gpus, join=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b")
    ap.add_argument("--batch", type=int, default=1, help="sequences per GPU")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-points", action="store_true", help="skip the isolated verify / attention timings")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the prompt length (longer KV prefix)")
    ap.add_argument("--window", type=int, default=0, help="override the Jacobi window W (at most 64)")
    ap.add_argument("--table", action="store_true",
                    help="whole-image generation under the baseline schedules and SJD (rows A-D and no-refinement)")
    ap.add_argument("--n-generate", type=int, default=0, help="image tokens per image for --table (default: the workload's)")
    ap.add_argument("--temperature", type=float, default=0.0, help="override the sampling temperature (default: the workload's, 1.0)")
    ap.add_argument("--paged-kv", action="store_true", help="keep the KV cache in 64-position pages (same results)")
    ap.add_argument("--guidance", type=float, default=0.0,
                    help="classifier-free guidance weight (the paper runs 3.0): two streams per image, 2 x batch x W rows")
    args = ap.parse_args()
    from paper_2410_01699_b200.inputs import WORKLOADS
    wl = WORKLOADS[args.workload]
    if args.prompt_len:
        wl = wl.with_(prompt_len=args.prompt_len)
    if args.window:
        wl = wl.with_(window=args.window)
    if args.temperature > 0:
        wl = wl.with_(temperature=args.temperature)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.table:
        run_table(args, wl)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        launch_ranks(args, wl)
    else:
        run_library(args, wl)


if __name__ == "__main__":
    main()
