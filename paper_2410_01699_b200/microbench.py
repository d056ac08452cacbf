"""Single-kernel timings through the C-ABI (CUDA events on the launching stream).

    python -m paper_2410_01699_b200.microbench gemm M N K [--iters I]
    python -m paper_2410_01699_b200.microbench verify BATCH [--window W --vocab V --top-k K --iters I]

gemm    the weight-streaming projection (sjd_gemm): fp32 x[M][K], bf16 w[N][K]; reports the achieved
        weight-streaming rate N*K*2 bytes / time.  The weights rotate through enough copies to exceed
        the L2 cache, so every launch streams from HBM.
attention BATCH PREFIX [--window W --heads H --kv-heads KVH --head-dim D]: the window attention
        (sjd_attention) of W queries over PREFIX + W cached positions; reports K/V bytes / time.
verify  the isolated verify-and-resample kernel (sjd_verify) on the synthetic verification workload;
        reports 2*B*W*V*2 bytes / time (current and previous logits read once each).

Each call is small enough (a few launches of one kernel, buffers of a few hundred MB) to be captured under ncu.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import binding as B
from .inputs import make_verify_case


def _peak():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return json.load(open(path))["hbm_gbs"], "measured"
    return 6650.0, "fallback"


NOMINAL_HBM_GBPS = 8000.0   # the data-sheet figure, printed beside the measured copy bandwidth


def _time(fn, iters, warmup=20, graph=False):
    """Seconds per call.  graph=True records the `iters` calls into one CUDA graph and times replays of
    it, so that a kernel of a few microseconds is not timed by the speed of the Python loop."""
    for _ in range(warmup):
        fn(0)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(iters):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(5):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (5 * iters) * 1e-3
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e-3


def bench_gemm(m, n, k, iters):
    g = torch.Generator(device="cuda").manual_seed(0)
    x = torch.randn(m, k, generator=g, device="cuda")
    wbytes = n * k * 2
    copies = max(1, min(16, (192 << 20) // wbytes + 1))        # > L2 in total
    ws = [(torch.randn(n, k, generator=g, device="cuda") * 0.05).to(torch.bfloat16) for _ in range(copies)]
    out = torch.zeros(m, n, device="cuda")
    status = [None]

    def run(i):
        _, status[0] = B.sjd_gemm(x, ws[i % copies], out=out)

    sec = _time(run, iters)
    assert int(status[0].item()) == 0, "a device-side wait ran out"
    peak, src = _peak()
    gbs = wbytes / sec / 1e9
    return {"kernel": "sjd_gemm", "M": m, "N": n, "K": k, "us": sec * 1e6, "weight_GBps": gbs, "frac_of_hbm": gbs / peak, "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBPS,
            "peak_GBps": peak, "peak_source": src, "TFLOPs": 2.0 * m * n * k / sec / 1e12,
            "note": "time includes the hi/lo split and plane-sum launches of sjd_gemm"}


def bench_verify(batch, window, vocab, top_k, iters):
    case = make_verify_case(batch, window=window, vocab=vocab, top_k=top_k)
    copies = max(1, min(8, (192 << 20) // (2 * batch * window * vocab * 2) + 1))
    cur = [torch.from_numpy(case.logits_cur).cuda().to(torch.bfloat16).clone() for _ in range(copies)]
    prev = [torch.from_numpy(case.logits_prev).cuda().to(torch.bfloat16).clone() for _ in range(copies)]
    draft, kind, base = (torch.from_numpy(a).cuda() for a in (case.draft, case.q_kind, case.base_pos))
    out = B.StepOut(batch, window)
    sample = B.make_sample_cfg(temperature=case.temperature, top_k=case.top_k, seed=case.seed, window=window)
    ws = torch.empty(B.sjd_verify_workspace_bytes(batch, window), dtype=torch.uint8, device="cuda")

    def run(i):
        B.sjd_verify(cur[i % copies], prev[i % copies], draft, kind, base, sample, case.step, out, ws=ws)

    sec = _time(run, iters)
    peak, src = _peak()
    nbytes = 2 * batch * window * vocab * 2
    gbs = nbytes / sec / 1e9
    return {"kernel": "sjd_verify", "batch": batch, "window": window, "vocab": vocab, "top_k": top_k, "us": sec * 1e6,
            "logits_GBps": gbs, "frac_of_hbm": gbs / peak, "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBPS, "peak_GBps": peak, "peak_source": src,
            "rows_per_s": batch * window / sec, "mean_accepted": float(out.host()["n_accepted"].mean())}


def bench_attention(batch, window, prefix, n_heads, n_kv_heads, head_dim, iters, graph=True):
    g = torch.Generator(device="cuda").manual_seed(0)
    max_seq = prefix + window
    q = torch.randn(batch * window, n_heads, head_dim, generator=g, device="cuda")
    kv_bytes = batch * 2 * n_kv_heads * max_seq * head_dim * 2
    copies = max(1, min(8, (192 << 20) // kv_bytes + 1))
    kvs = [torch.randn(batch, 2, n_kv_heads, max_seq, head_dim, generator=g, device="cuda").to(torch.bfloat16)
           for _ in range(copies)]
    pos = (prefix - 1 + torch.arange(window, dtype=torch.int32, device="cuda")).repeat(batch).contiguous()
    out = torch.empty_like(q)
    ws = torch.empty(int(B.lib().sjd_attention_workspace_bytes(batch, window, n_heads, head_dim)), dtype=torch.uint8,
                     device="cuda")
    status = [None]

    def run(i):
        _, status[0] = B.sjd_attention(q, kvs[i % copies], pos, window, n_kv_heads, out=out, ws=ws)

    sec = _time(run, iters, graph=graph)
    assert int(status[0].item()) == 0
    peak, src = _peak()
    gbs = kv_bytes / sec / 1e9
    return {"kernel": "sjd_attention", "batch": batch, "window": window, "prefix": prefix, "n_heads": n_heads,
            "n_kv_heads": n_kv_heads, "head_dim": head_dim, "us": sec * 1e6, "kv_GBps": gbs, "frac_of_hbm": gbs / peak, "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBPS,
            "peak_GBps": peak, "peak_source": src, "note": "time includes the merge of the split-KV partials"}


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("M", type=int)
    g.add_argument("N", type=int)
    g.add_argument("K", type=int)
    g.add_argument("--iters", type=int, default=100)
    v = sub.add_parser("verify")
    v.add_argument("batch", type=int)
    v.add_argument("--window", type=int, default=32)
    v.add_argument("--vocab", type=int, default=16384)
    v.add_argument("--top-k", type=int, default=2000)
    v.add_argument("--iters", type=int, default=100)
    t = sub.add_parser("attention")
    t.add_argument("batch", type=int)
    t.add_argument("prefix", type=int)
    t.add_argument("--window", type=int, default=32)
    t.add_argument("--heads", type=int, default=32)
    t.add_argument("--kv-heads", type=int, default=32)
    t.add_argument("--head-dim", type=int, default=128)
    t.add_argument("--iters", type=int, default=100)
    t.add_argument("--no-graph", action="store_true", help="time a plain Python loop of calls (for captures under ncu)")
    a = ap.parse_args()
    if a.cmd == "attention":
        print(json.dumps(bench_attention(a.batch, a.window, a.prefix, a.heads, a.kv_heads, a.head_dim, a.iters, not a.no_graph)))
    elif a.cmd == "gemm":
        print(json.dumps(bench_gemm(a.M, a.N, a.K, a.iters)))
    else:
        print(json.dumps(bench_verify(a.batch, a.window, a.vocab, a.top_k, a.iters)))


if __name__ == "__main__":
    main()
