"""Device timeline of one overlapped SJD step (diagnostic).

    python -m paper_2410_01699_b200.timeline [--workload 7b] [--layer 10]

Builds a copy of the library with -DSJD_TIMELINE (block 0 of every kernel of the tensor-core pipeline
stamps %globaltimer at its entry, when its grid dependency has resolved, i.e. when the previous grid
has completed, and at its end), replays a few steps as CUDA graphs and prints, for one decoder layer
and for the end of the step, the time from each kernel's dependency resolution to the next one's: the
contribution of every link of the chain to the step as it really runs, with programmatic dependent
launch and weight prefetch overlapped.  CUDA events cannot show this: an event between two launches
breaks the overlap.  The instrumented library lives beside the normal one (libsjd_tl.so) and is never
loaded by anything else.
"""
from __future__ import annotations

import argparse
import ctypes as C
import os
import subprocess

import numpy as np
import torch

from . import binding as B
from . import build as bld
from .inputs import WORKLOADS, make_prompt, make_weights

LIB_TL = os.path.join(bld.HERE, "libsjd_tl.so")
NAMES = {0: "embed", 1: "resid_gain", 2: "gemm", 3: "qkv_finish", 4: "attention", 5: "combine", 6: "swiglu", 7: "verify"}


def build_instrumented() -> str:
    obj_dir = os.path.join(bld.OBJ, "tl")
    os.makedirs(obj_dir, exist_ok=True)
    sources = sorted(f for f in os.listdir(bld.CSRC) if f.endswith(".cu"))
    procs, objs = [], []
    for src in sources:
        obj = os.path.join(obj_dir, src[:-3] + ".o")
        objs.append(obj)
        procs.append(subprocess.Popen([bld._nvcc()] + bld.NVCC_FLAGS + ["-DSJD_TIMELINE", "-c", os.path.join(bld.CSRC, src),
                                                                         "-o", obj]))
    for p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed")
    subprocess.check_call([bld._nvcc(), "-shared", "-o", LIB_TL] + objs)
    return LIB_TL


def capture(wl, steps: int = 3):
    """[(ns since the first record, kernel class, phase)] of `steps` consecutive steps."""
    B.LIB_PATH = LIB_TL
    lib = B.lib()
    lib.sjd_timeline_bytes.restype = C.c_size_t
    buf = torch.zeros(lib.sjd_timeline_bytes(), dtype=torch.uint8, device="cuda")
    weights = make_weights(wl, device="cuda")
    ctx = B.Context(B.make_model_cfg(wl, 1, wl.prompt_len + wl.n_generate + 8, wl.window), weights)
    sample = B.make_sample_cfg(wl.temperature, wl.top_k, wl.philox_seed, wl.window, 0, wl.grid_stride, wl.n_generate)
    ctx.prefill(torch.from_numpy(make_prompt(wl, 1)).cuda(), sample)
    out = B.StepOut(1, wl.window)
    for _ in range(20):
        ctx.step(out)
    torch.cuda.synchronize()
    lib.sjd_timeline_attach(C.c_void_p(buf.data_ptr()))
    torch.cuda.synchronize()
    for _ in range(steps):
        ctx.step(out)
    torch.cuda.synchronize()
    raw = buf.cpu().numpy()
    n = min(int(raw[:4].view(np.uint32)[0]), 1 << 16)
    rec = raw[8:8 + 16 * n].view(np.dtype([("t", "<u8"), ("tag", "<i4"), ("phase", "<i4")]))
    order = np.argsort(rec["t"], kind="stable")
    t0 = int(rec["t"].min())
    return [(int(rec["t"][i]) - t0, NAMES.get(int(rec["tag"][i]), "?"), int(rec["phase"][i])) for i in order]


def links(rows):
    """Dependency-resolution records (phase 1) of the middle step: [(us, kernel)]."""
    ver = [k for k, r in enumerate(rows) if r[1] == "verify" and r[2] == 1]
    s, e = ver[0], ver[1]
    return [(r[0] / 1e3, r[1]) for r in rows[s:e + 1] if r[2] == 1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="7b")
    ap.add_argument("--layer", type=int, default=10)
    a = ap.parse_args()
    build_instrumented()
    wl = WORKLOADS[a.workload]
    ln = links(capture(wl))
    # ln[0] is the verification of the previous step; then per layer: resid, gemm, qkv, attention(, combine), gemm,
    # resid, gemm(, swiglu), gemm
    per_layer = (len(ln) - 3) // wl.n_layers
    print("step: %.1f us from one verification to the next; %d links per layer" % (ln[-1][0] - ln[0][0], per_layer))
    i0 = 1 + a.layer * per_layer
    for k in range(i0, i0 + per_layer):
        print("  %-11s %7.2f us" % (ln[k][1], ln[k + 1][0] - ln[k][0]))
    print("  layer       %7.2f us" % (ln[i0 + per_layer][0] - ln[i0][0]))
    print("end of step: final resid_gain %.2f us, logits projection %.2f us; verification to the next step's "
          "first dependency %.2f us" % (ln[-2][0] - ln[-3][0], ln[-1][0] - ln[-2][0], ln[1][0] - ln[0][0]))


if __name__ == "__main__":
    main()
