"""GPU parity of the fused verify-and-resample kernel (sjd_verify through the C-ABI) against the
CPU checker, element by element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2410_01699_b200 import binding as B
from paper_2410_01699_b200.inputs import make_verify_case, round_bf16
from tests.parity_util import ParityStats, compare_window, oracle_verify_case

pytestmark = pytest.mark.gpu


def _run_gpu(case, logits_prev=True):
    dt = torch.bfloat16 if case.dtype == "bf16" else torch.float32
    cur = torch.from_numpy(case.logits_cur).to("cuda").to(dt)
    prev = torch.from_numpy(case.logits_prev).to("cuda").to(dt) if logits_prev else None
    draft = torch.from_numpy(case.draft).cuda()
    kind = torch.from_numpy(case.q_kind.astype(np.int32)).cuda()
    base = torch.from_numpy(case.base_pos).cuda()
    out = B.StepOut(case.batch, case.window)
    sample = B.make_sample_cfg(temperature=case.temperature, top_k=case.top_k, seed=case.seed, window=case.window)
    B.sjd_verify(cur, prev, draft, kind, base, sample, case.step, out)
    return out.host()


def _check_case(case, prob_tol=1e-5, max_flag_frac=0.03):
    got = _run_gpu(case)
    stats = ParityStats()
    for b in range(case.batch):
        vr, qdescs = oracle_verify_case(case, b)
        gpu = dict(n_accepted=got["n_accepted"][b], committed=got["committed"][b], draft=got["draft"][b],
                   q_draft=got["q_draft"][b])
        st = compare_window(vr, gpu, case.logits_cur[b].astype(np.float64), case.draft[b], qdescs, case.temperature,
                            case.top_k, prob_tol, where=f"seq {b}")
        stats.merge(st)
        if st.skipped_sequences == 0:
            assert got["n_committed"][b] == len(vr.committed)
            assert got["total_committed"][b] == case.base_pos[b] + len(vr.committed)
            kept = len(vr.redraft)
            assert list(got["q_kind"][b][:kept]) == [B.SJD_Q_ROW] * kept
            assert all(x == -1 for x in got["draft"][b][kept:]) and all(x == -1 for x in got["q_kind"][b][kept:])
    assert stats.flagged <= max(2, max_flag_frac * stats.decisions), f"too many near-ties: {stats}"
    return stats


@pytest.mark.parametrize("batch", [1, 4])
def test_verify_workload_shape(batch):
    """The isolated-verification workload: W = 32 rows over a 16384 vocabulary, bf16, top-k 2000."""
    _check_case(make_verify_case(batch))


def test_verify_full_batch():
    """Largest batch of the workload in the launch configuration the benchmark times (32 sequences of
    32 rows): every sequence is re-computed by the checker."""
    stats = _check_case(make_verify_case(32))
    assert stats.sequences == 32


def test_verify_ratio_corner_cases():
    """Eq. 1 where q(d) or p(d) vanishes (drafts whose law is a logits row, top-k 200 of 4096):
    q(d) = 0 < p(d) accepts for any uniform, p(d) = 0 < q(d) rejects, p(d) = q(d) = 0 rejects.  Rows
    around the corner rows have identical current and previous logits (ratio exactly 1: accepted), so the
    scan reaches each corner row and the number of accepted drafts is known without any checker."""
    case = make_verify_case(3, window=6, vocab=4096, top_k=200, seed=77)
    case.logits_prev = case.logits_cur.copy()
    order = np.argsort(-case.logits_cur, axis=-1, kind="stable")   # tokens of each row, largest logit first

    def put(b, k, p_in, q_in):
        """Draft of row k of sequence b: a token of p's top-k set (or not), q's entry raised / lowered."""
        d = int(order[b, k, 50 if p_in else 3000])
        case.draft[b, k] = d
        if p_in and not q_in:
            case.logits_prev[b, k, d] = np.float32(-30.0)     # out of q's set; q's set takes the 201st entry in
        if q_in and not p_in:
            case.logits_prev[b, k, d] = np.float32(12.0)      # in q's set only
        return d

    for b in range(3):
        for k in range(6):
            case.draft[b, k] = int(order[b, k, 20])           # p == q on the draft: always accepted
    put(0, 2, True, False)     # q(d) = 0 < p(d): accepted, the scan goes on
    put(0, 4, False, False)    # 0 / 0: rejected
    put(1, 0, True, False)     # accepted
    put(1, 1, False, True)     # p(d) = 0 < q(d): rejected
    put(2, 0, False, False)    # 0 / 0 on the very first row
    got = _run_gpu(case)
    assert list(got["n_accepted"]) == [4, 1, 0]
    assert list(got["n_committed"]) == [5, 2, 1]
    stats = _check_case(case)
    assert stats.flagged == 0


@pytest.mark.parametrize("dtype,vocab,window,top_k", [
    ("bf16", 16001, 29, 2000),   # ragged: rows not 16-byte aligned, odd window
    ("f32", 1024, 16, 64),       # the tiny end-to-end model's head
    ("f32", 1000, 7, 1000),      # top_k == V: no filtering
    ("bf16", 4099, 5, 1),        # top-1
    ("bf16", 65536, 4, 2000),    # 128 KB rows (the 7B head)
    ("bf16", 184320, 2, 2048),   # rows longer than a block's registers: streamed in three segments (the 8B head)
    ("bf16", 100000, 5, 2000),   # two segments, the second partial (12500 vectors against 8192)
    ("bf16", 184320, 3, 184320), # streamed rows, top_k == V: no threshold
    ("bf16", 262000, 2, 4000),   # the longest row the chunk table covers: four segments
    ("f32", 50000, 3, 500),      # fp32 rows beyond the staging buffer
])
def test_verify_shapes(dtype, vocab, window, top_k):
    case = make_verify_case(2, window=window, vocab=vocab, dtype=dtype, top_k=top_k, seed=7 + vocab)
    _check_case(case, max_flag_frac=0.06)


def test_verify_mixed_laws():
    """Slots whose draft came from a uniform initialisation (q = 1/V) or a copy (point mass)."""
    case = make_verify_case(6, window=16, vocab=4096, top_k=300, seed=11, mixed_kinds=True)
    _check_case(case)


def test_verify_mixed_laws_on_streamed_rows():
    """The same on rows too long for the registers (drift 3: most drafts are rejected, so Eq. 2 runs on streamed
    rows against uniform, copied and predicted drafts)."""
    case = make_verify_case(3, window=6, vocab=100000, top_k=2000, seed=12, mixed_kinds=True, drift=3.0)
    _check_case(case, max_flag_frac=0.06)


def test_verify_streamed_rows_in_a_grid_of_several_waves():
    """160 streamed rows on 148 SMs: the rejected rows leave Eq. 2 to their sequence's last block, which streams
    the two rows again."""
    case = make_verify_case(10, window=16, vocab=70000, top_k=2000, seed=13, drift=2.0)
    _check_case(case, max_flag_frac=0.06)


def test_verify_temperature_and_ties():
    case = make_verify_case(3, window=8, vocab=8192, top_k=500, temperature=0.7, seed=5)
    _check_case(case)
    # coarse logits: many exact ties at the top-k threshold (all must be kept)
    case = make_verify_case(3, window=8, vocab=8192, top_k=500, seed=6)
    case.logits_cur = round_bf16(np.round(case.logits_cur * 2) / 2)
    case.logits_prev = round_bf16(np.round(case.logits_prev * 2) / 2)
    _check_case(case)


@pytest.mark.parametrize("shift,top_k", [
    (-9.0, 2000),    # positive maximum, negative threshold: more than 4095 bf16 codes apart (general route)
    (-30.0, 2000),   # every logit negative: maximum and threshold within a few binades (register route)
    (0.0, 8000),     # half the row kept: threshold around zero
    (0.0, 16384),    # top_k == V: no filtering on the register route
])
def test_verify_threshold_far_from_the_maximum(shift, top_k):
    """The register-resident route counts entries by their distance below the row maximum and hands rows
    whose threshold is out of that reach to the general route; both must agree with the checker."""
    case = make_verify_case(2, window=6, vocab=16384, top_k=top_k, seed=31)
    case.logits_cur = round_bf16(case.logits_cur + np.float32(shift))
    case.logits_prev = round_bf16(case.logits_prev + np.float32(shift))
    _check_case(case, max_flag_frac=0.06)


def test_verify_zeros_at_the_threshold():
    """Exact zeros of both signs around the top-k threshold (bf16 comparison cannot order +0 and -0, the
    order-preserving keys can): such rows take the general route."""
    case = make_verify_case(2, window=4, vocab=8192, top_k=3000, seed=33)
    for arr in (case.logits_cur, case.logits_prev):
        small = np.abs(arr) < 0.35
        arr[small] = np.where(arr[small] < 0, np.float32(-0.0), np.float32(0.0))
    _check_case(case, max_flag_frac=0.06)


def test_verify_identical_rows_accept_everything():
    """p == q bit for bit: every ratio is 1 and every draft is accepted for any uniform."""
    case = make_verify_case(2, window=12, vocab=4096, top_k=100, seed=3)
    case.logits_prev = case.logits_cur.copy()
    got = _run_gpu(case)
    assert list(got["n_accepted"]) == [12, 12] and list(got["n_committed"]) == [12, 12]
    assert np.array_equal(got["committed"], case.draft)
    assert np.all(got["draft"] == -1)


def test_verify_nonfinite_rows_are_flagged():
    case = make_verify_case(2, window=4, vocab=2048, top_k=50, seed=9)
    case.logits_cur[0, 1, 5] = np.nan
    case.logits_cur[0, 1, 9] = np.inf
    got = _check_and_flags(case)
    assert got["flags"][0] & B.SJD_FLAG_NONFINITE
    assert not (got["flags"][1] & B.SJD_FLAG_NONFINITE)


def _check_and_flags(case):
    _check_case(case)
    return _run_gpu(case)


def test_verify_is_deterministic():
    case = make_verify_case(4, window=16, vocab=16384, seed=21)
    a, b = _run_gpu(case), _run_gpu(case)
    for k in a:
        assert np.array_equal(a[k], b[k]), k


def test_verify_argument_errors():
    out = B.StepOut(1, 4)
    s = B.make_sample_cfg(top_k=10, window=4)
    cur = torch.zeros(1, 4, 128, device="cuda")
    d = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.sjd_verify_workspace_bytes(1, 4), dtype=torch.uint8, device="cuda")
    L = B.lib()
    import ctypes as C
    args = lambda **kw: [kw.get("b", 1), kw.get("w", 4), 128, kw.get("dt", 0), C.c_void_p(cur.data_ptr()),
                         C.c_void_p(cur.data_ptr()), C.c_void_p(d.data_ptr()), None, None, C.byref(kw.get("s", s)), 0,
                         C.byref(out.c), C.c_void_p(ws.data_ptr()), kw.get("n", ws.numel()), None]
    assert L.sjd_verify(*args()) == B.SJD_OK
    assert L.sjd_verify(*args(b=0)) == B.SJD_ERR_BAD_ARG
    assert L.sjd_verify(*args(dt=5)) == B.SJD_ERR_UNSUPPORTED
    assert L.sjd_verify(*args(n=16)) == B.SJD_ERR_CAPACITY
    assert L.sjd_verify(*args(s=B.make_sample_cfg(temperature=0.0, top_k=10))) == B.SJD_ERR_BAD_ARG
    assert L.sjd_verify(*args(s=B.make_sample_cfg(top_k=0))) == B.SJD_ERR_BAD_ARG
    torch.cuda.synchronize()
