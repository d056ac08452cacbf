"""Pins for the CPU checker's random numbers, logit warp, sampler and
verification scan: known answers, closed forms, library routines and the
identities of the paper's Appendix A.  No GPU."""
import os

import numpy as np
import pytest
from scipy import special, stats

from oracle import philox
from oracle.sampling import (FLAG_RESIDUAL_EMPTY, Q_ONEHOT, Q_ROW, Q_UNIFORM, QDesc, icdf,
                             verify_window, warp)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- Philox (Salmon et al., SC'11)
def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([int(x, 16) for x in line.split()])
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for r in rows:
        assert list(philox.philox4x32_10(r[0:4], r[4:6])) == r[6:10]


def test_philox_vectorised_matches_scalar():
    rng = np.random.default_rng(0)
    c = rng.integers(0, 2 ** 32, size=(4, 50), dtype=np.uint64)
    k0, k1 = 0x12345678, 0x9ABCDEF0
    out = philox.philox4x32_10_np(c[0], c[1], c[2], c[3], k0, k1)
    for i in range(50):
        ref = philox.philox4x32_10(tuple(int(c[j, i]) for j in range(4)), (k0, k1))
        assert tuple(int(o[i]) for o in out) == ref
    for r in _kat_rows():
        out = philox.philox4x32_10_np(*[np.array([x]) for x in r[0:4]], r[4], r[5])
        assert [int(o[0]) for o in out] == r[6:10]


def test_uniform_range_and_moments():
    c0 = np.arange(200000)
    w = philox.philox4x32_10_np(c0, 7, 3, 0, *philox.split_seed(99))
    u = (w[0] >> np.uint64(8)).astype(np.float64) / 2 ** 24
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / u.size)
    # u24 is exactly representable in fp32
    assert np.all(u.astype(np.float32).astype(np.float64) == u)
    assert philox.u24(0xFFFFFFFF) == (2 ** 24 - 1) / 2 ** 24
    # uniformity over 64 bins
    chi = stats.chisquare(np.bincount((u * 64).astype(int), minlength=64))
    assert chi.pvalue > 1e-4


def test_init_token_uniform_over_vocab():
    vocab = 37
    w = philox.philox4x32_10_np(np.arange(100000), 5, 0, philox.STREAM_INIT, *philox.split_seed(3))
    tok = (w[0] * np.uint64(vocab)) >> np.uint64(32)
    assert tok.max() == vocab - 1 and tok.min() == 0
    assert stats.chisquare(np.bincount(tok.astype(int), minlength=vocab)).pvalue > 1e-4
    assert philox.init_token(3, 17, 5, 0, vocab) == int(tok[17])


# ---------------------------------------------------------------- warp (top-K sampling, Sec. 3.1)
def test_warp_no_filter_is_softmax():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 3, size=500)
    for t in (1.0, 0.5, 2.5):
        np.testing.assert_allclose(warp(x, t, 500), special.softmax(x / t), rtol=1e-13, atol=0)
        np.testing.assert_allclose(warp(x, t, 10 ** 6), special.softmax(x / t), rtol=1e-13, atol=0)


def test_warp_topk_matches_partition_and_renormalises():
    rng = np.random.default_rng(2)
    x = rng.normal(0, 3, size=1000)
    k = 50
    p = warp(x, 1.0, k)
    kth = np.partition(x, 1000 - k)[1000 - k]
    keep = x >= kth
    assert keep.sum() == k
    assert np.all((p > 0) == keep)
    assert abs(p.sum() - 1) < 1e-14
    np.testing.assert_allclose(p[keep], special.softmax(x[keep]), rtol=1e-13)


def test_warp_top1_is_argmax_and_ties_are_kept():
    x = np.array([0.1, 2.0, -1.0, 1.5])
    np.testing.assert_array_equal(warp(x, 1.0, 1), [0, 1, 0, 0])
    # tiny temperature with no top-k filter also collapses onto the arg-max
    assert warp(x, 1e-3, 4)[1] > 1 - 1e-12
    # ties at the threshold: all kept, kept set exceeds K
    y = np.array([1.0, 3.0, 3.0, 0.0, 3.0])
    np.testing.assert_allclose(warp(y, 1.0, 1), [0, 1 / 3, 1 / 3, 0, 1 / 3])
    np.testing.assert_allclose(warp(y, 1.0, 2), [0, 1 / 3, 1 / 3, 0, 1 / 3])
    z = np.array([1.0, 3.0, 2.0, 2.0, 0.0])
    p = warp(z, 1.0, 2)
    assert np.all((p > 0) == np.array([False, True, True, True, False]))


def test_warp_nonfinite_rows():
    x = np.array([0.0, np.nan, 1.0, np.inf, -np.inf])
    p = warp(x, 1.0, 5)
    np.testing.assert_allclose(p, special.softmax(np.array([0.0, -np.inf, 1.0, -np.inf, -np.inf])))
    np.testing.assert_array_equal(warp(np.array([np.nan, -np.inf]), 1.0, 2), [1.0, 0.0])


def test_warp_rejects_bad_arguments():
    with pytest.raises(ValueError):
        warp(np.zeros(4), 0.0, 2)
    with pytest.raises(ValueError):
        warp(np.zeros(4), 1.0, 0)


# ---------------------------------------------------------------- inverse-CDF sampler
def _icdf_loop(w, u):
    total = 0.0
    for x in w:
        total += x
    target, acc = u * total, 0.0
    last = None
    for i, x in enumerate(w):
        acc += x
        if x > 0:
            last = i
            if acc > target:
                return i
    return last


def test_icdf_matches_searchsorted_and_loop():
    rng = np.random.default_rng(3)
    for trial in range(200):
        v = int(rng.integers(1, 60))
        w = rng.random(v) * (rng.random(v) < 0.6)
        if w.sum() == 0:
            w[rng.integers(0, v)] = 1.0
        u = float(rng.random())
        i, margin = icdf(w, u)
        c = np.cumsum(w)
        assert i == int(np.searchsorted(c, u * c[-1], side="right"))
        assert i == _icdf_loop(list(w), u)
        assert w[i] > 0 and margin >= 0


def test_icdf_edges():
    w = np.array([0.0, 1.0, 0.0, 3.0, 0.0])
    assert icdf(w, 0.0)[0] == 1
    assert icdf(w, 0.25 - 1e-12)[0] == 1
    assert icdf(w, 0.25)[0] == 3            # strict '>' at the edge
    assert icdf(w, 1.0 - 2 ** -24)[0] == 3
    assert icdf(w, 1.0)[0] == 3             # fallback: largest index with positive weight
    with pytest.raises(ValueError):
        icdf(np.zeros(3), 0.5)


def test_icdf_distribution():
    w = np.array([0.5, 0.0, 2.0, 1.5, 0.0, 1.0])
    words = philox.philox4x32_10_np(np.arange(60000), 0, 0, 0, 11, 22)[0]
    u = (words >> np.uint64(8)).astype(np.float64) / 2 ** 24
    counts = np.bincount([icdf(w, x)[0] for x in u], minlength=6)
    assert counts[1] == 0 and counts[4] == 0
    keep = w > 0
    assert stats.chisquare(counts[keep], w[keep] / w.sum() * u.size).pvalue > 1e-4


# ---------------------------------------------------------------- verification scan (Eqs. 1-3, App. A)
def _uniform_block(n_trials, w_eff, seed):
    """[n_trials][w_eff][3] Philox uniforms: position = slot, step = trial."""
    pos = np.arange(w_eff)[None, :]
    step = np.arange(n_trials)[:, None]
    w = philox.philox4x32_10_np(pos, step, 0, 0, *philox.split_seed(seed))
    return np.stack([(x >> np.uint64(8)).astype(np.float64) / 2 ** 24 for x in w[:3]], axis=-1)


V8_P = np.array([0.30, 0.05, 0.20, 0.10, 0.02, 0.18, 0.05, 0.10])
V8_QS = {
    "peaked_elsewhere": np.array([0.01, 0.60, 0.02, 0.02, 0.30, 0.02, 0.02, 0.01]),
    "uniform": np.full(8, 1 / 8),
    "equal": V8_P.copy(),
    "disjoint_support": np.array([0.0, 0.5, 0.0, 0.0, 0.5, 0.0, 0.0, 0.0]),
}


@pytest.mark.parametrize("qname", list(V8_QS))
def test_single_position_is_exact(qname):
    """Theorem 1: whatever q the draft came from, the token fixed at a position follows p.
    Also P(accept and x) = min(p, q)(x) and P(reject) = sum max(0, p - q)  (App. A)."""
    p, q = V8_P, V8_QS[qname]
    logits_p = np.log(p)[None, :]
    with np.errstate(divide="ignore"):
        qrow = np.log(q)
    n = 40000
    u = _uniform_block(n, 1, seed=list(V8_QS).index(qname))
    draft_u = philox.philox4x32_10_np(np.arange(n), 1, 2, 3, 5, 6)[0]
    out = np.zeros(8)
    acc_x = np.zeros(8)
    rejects = 0
    for t in range(n):
        d, _ = icdf(q, float(draft_u[t] >> np.uint64(8)) / 2 ** 24)
        r = verify_window(logits_p, [d], [QDesc(Q_ROW, row=qrow)], u[t], 1.0, 8)
        out[r.committed[0]] += 1
        if r.n_accepted == 1:
            acc_x[d] += 1
        else:
            rejects += 1
    assert stats.chisquare(out, p * n).pvalue > 1e-4
    se = np.sqrt(np.maximum(np.minimum(p, q), 1e-4) / n)
    assert np.all(np.abs(acc_x / n - np.minimum(p, q)) < 5 * se)
    rej = np.maximum(0, p - q).sum()
    assert abs(rejects / n - rej) < 5 * np.sqrt(max(rej, 1e-4) / n)


def test_uniform_and_onehot_descriptors_are_exact():
    """A fresh random token carries q = 1/V, a copied token a point mass; both keep the
    fixed token distributed as p."""
    p = V8_P
    logits = np.log(p)[None, :]
    n = 30000
    u = _uniform_block(n, 1, seed=77)
    words = philox.philox4x32_10_np(np.arange(n), 9, 9, 1, 1, 2)[0]
    out_u, out_o = np.zeros(8), np.zeros(8)
    for t in range(n):
        d = int((int(words[t]) * 8) >> 32)
        out_u[verify_window(logits, [d], [QDesc(Q_UNIFORM)], u[t], 1.0, 8).committed[0]] += 1
        out_o[verify_window(logits, [2], [QDesc(Q_ONEHOT)], u[t], 1.0, 8).committed[0]] += 1
    assert stats.chisquare(out_u, p * n).pvalue > 1e-4
    assert stats.chisquare(out_o, p * n).pvalue > 1e-4


def test_scan_stops_at_first_rejection_and_redrafts_the_rest():
    v = 6
    rng = np.random.default_rng(5)
    logits = rng.normal(0, 1, size=(5, v))
    p = [warp(r, 1.0, v) for r in logits]
    prev = rng.normal(0, 1, size=(5, v))
    q = [warp(r, 1.0, v) for r in prev]
    drafts = [1, 4, int(np.argmin(p[2] / q[2])), 0, 3]
    thr = [min(1.0, p[k][drafts[k]] / q[k][drafts[k]]) for k in range(5)]
    assert thr[2] < 1.0
    # force: accept, accept, reject at slot 2; later uniforms would accept but must be ignored
    u = np.zeros((5, 3))
    u[:, 0] = [thr[0] * 0.5, thr[1] * 0.5, min(thr[2] * 1.5, 0.999999), 0.0, 0.0]
    u[:, 1] = 0.4
    u[:, 2] = [0.1, 0.2, 0.3, 0.6, 0.9]
    r = verify_window(logits, drafts, [QDesc(Q_ROW, row=prev[k]) for k in range(5)], u, 1.0, v)
    assert r.n_accepted == 2 and r.accept == [True, True, False]
    resid = np.maximum(0, p[2] - q[2])
    assert r.committed == [1, 4, icdf(resid, 0.4)[0]] and r.committed[2] != drafts[2]
    assert r.redraft == [icdf(p[3], 0.6)[0], icdf(p[4], 0.9)[0]]
    assert r.redraft_rows == [3, 4]
    # all accepted: nothing resampled, nothing re-drafted
    u[:, 0] = 0.0
    r = verify_window(logits, drafts, [QDesc(Q_ROW, row=prev[k]) for k in range(5)], u, 1.0, v)
    assert r.n_accepted == 5 and r.committed == drafts and r.redraft == []


def test_ratio_corner_cases():
    logits = np.log(np.array([[0.5, 0.5, 1e-300, 1e-300]]))
    # q(d) = 0 < p(d): always accepted, even with u just below 1
    qrow = np.array([-np.inf, 0.0, 0.0, 0.0])
    r = verify_window(logits, [0], [QDesc(Q_ROW, row=qrow)], [[1 - 2 ** -24, 0.3, 0.3]], 1.0, 4)
    assert r.n_accepted == 1
    # p(d) = 0 (outside top-k of the current row): always rejected, even with u = 0
    r = verify_window(np.array([[5.0, 4.0, 0.0, 0.0]]), [2], [QDesc(Q_UNIFORM)], [[0.0, 0.3, 0.3]], 1.0, 2)
    assert r.n_accepted == 0 and r.committed[0] in (0, 1)
    # strict '<': u == ratio rejects
    lg = np.log(np.array([[0.25, 0.75]]))
    r = verify_window(lg, [0], [QDesc(Q_UNIFORM)], [[0.5, 0.0, 0.0]], 1.0, 2)
    assert r.ratio[0] == pytest.approx(0.5) and r.n_accepted == 0
    # p == q and ratio == 1: accepted for every u in [0, 1)
    r = verify_window(lg, [1], [QDesc(Q_ROW, row=lg[0])], [[1 - 2 ** -24, 0.0, 0.0]], 1.0, 2)
    assert r.n_accepted == 1
    # a point-mass q on a token that holds all of p: ratio 1, accepted, no empty-residual fallback
    r = verify_window(np.array([[9.0, 0.0]]), [0], [QDesc(Q_ONEHOT)], [[0.999999, 0.5, 0.5]], 1.0, 1)
    assert r.n_accepted == 1
    assert not (r.flags & FLAG_RESIDUAL_EMPTY)
