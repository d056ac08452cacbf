"""sjd_verify_static: the verification entry point for callers that cannot allocate device memory
(no cudaMalloc inside a latency-bound serving loop, no allocator in the calling thread, a plug-in
that only receives input and output buffers).  It must give exactly what sjd_verify gives, call after
call, although every call reuses the same built-in scratch array and finds the previous call's
leftovers in it.  Collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2410_01699_b200 import binding as B
from paper_2410_01699_b200.inputs import make_verify_case
from tests.parity_util import compare_window, oracle_verify_case

pytestmark = pytest.mark.gpu

FIELDS = ("n_accepted", "n_committed", "committed", "draft", "q_kind", "q_draft", "total_committed", "flags")


def _device_inputs(case):
    dt = torch.bfloat16 if case.dtype == "bf16" else torch.float32
    return (torch.from_numpy(case.logits_cur).cuda().to(dt), torch.from_numpy(case.logits_prev).cuda().to(dt),
            torch.from_numpy(case.draft).cuda(), torch.from_numpy(case.q_kind.astype(np.int32)).cuda(),
            torch.from_numpy(case.base_pos).cuda())


def _both(case):
    cur, prev, draft, kind, base = _device_inputs(case)
    sample = B.make_sample_cfg(temperature=case.temperature, top_k=case.top_k, seed=case.seed, window=case.window)
    ref, got = B.StepOut(case.batch, case.window), B.StepOut(case.batch, case.window)
    B.sjd_verify(cur, prev, draft, kind, base, sample, case.step, ref)
    B.sjd_verify_static(cur, prev, draft, kind, base, sample, case.step, got)
    return ref.host(), got.host()


def test_static_scratch_entry_point_matches_sjd_verify_on_consecutive_calls():
    # two different problems back to back, the second smaller than the first so that it runs on
    # scratch still holding the first call's records and (zeroed-on-exit) counters
    cases = [make_verify_case(6, window=32, vocab=16384, seed=41, mixed_kinds=True),
             make_verify_case(3, window=9, vocab=5001, dtype="f32", top_k=100, seed=42),
             make_verify_case(6, window=32, vocab=16384, seed=43)]
    for i, case in enumerate(cases):
        ref, got = _both(case)
        for f in FIELDS:
            assert np.array_equal(ref[f], got[f]), "call %d: %s differs" % (i, f)
        assert np.all(got["n_committed"] >= 1)
        # and against the CPU checker, like every other verification test
        prob_tol = 1e-5
        for b in range(case.batch):
            vr, qdescs = oracle_verify_case(case, b)
            compare_window(vr, dict(n_accepted=got["n_accepted"][b], committed=got["committed"][b],
                                    draft=got["draft"][b], q_draft=got["q_draft"][b]),
                           case.logits_cur[b].astype(np.float64), case.draft[b], qdescs, case.temperature,
                           case.top_k, prob_tol, where="call %d, seq %d" % (i, b))


def test_static_scratch_entry_point_allocates_nothing():
    """Free device memory, as the driver reports it, is the same before and after calls of the entry point
    (inputs and outputs are created before the first reading; the first call, which makes the runtime
    load the library's device code, comes before it too)."""
    case = make_verify_case(4, window=16, vocab=8192, top_k=300, seed=44)
    cur, prev, draft, kind, base = _device_inputs(case)
    sample = B.make_sample_cfg(temperature=case.temperature, top_k=case.top_k, seed=case.seed, window=case.window)
    got = B.StepOut(case.batch, case.window)
    B.sjd_verify_static(cur, prev, draft, kind, base, sample, case.step, got)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    reserved_before = torch.cuda.memory_reserved()
    for _ in range(3):
        B.sjd_verify_static(cur, prev, draft, kind, base, sample, case.step, got)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before
    assert torch.cuda.memory_reserved() == reserved_before


def test_static_scratch_entry_point_rejects_oversized_problems():
    lib = B.lib()
    s = B.make_sample_cfg(top_k=10, window=64)
    out = B.StepOut(1, 1)
    x = torch.zeros(16, device="cuda")
    p = C.c_void_p(x.data_ptr())
    too_many_rows = B.SJD_VERIFY_STATIC_MAX_ROWS // 64 + 1
    assert lib.sjd_verify_static(too_many_rows, 64, 4, 0, p, p, p, None, None, C.byref(s), 0, C.byref(out.c), None) \
        == B.SJD_ERR_CAPACITY
    assert lib.sjd_verify_static(B.SJD_VERIFY_STATIC_MAX_BATCH + 1, 1, 4, 0, p, p, p, None, None, C.byref(s), 0,
                                 C.byref(out.c), None) == B.SJD_ERR_CAPACITY
    assert lib.sjd_verify_static(1, 65, 4, 0, p, p, p, None, None, C.byref(s), 0, C.byref(out.c), None) \
        == B.SJD_ERR_CAPACITY
    assert lib.sjd_verify_static(0, 4, 4, 0, p, p, p, None, None, C.byref(s), 0, C.byref(out.c), None) \
        == B.SJD_ERR_BAD_ARG
    torch.cuda.synchronize()
