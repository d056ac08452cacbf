"""Logit warp, inverse-CDF sampler and the SJD verification scan
(test infrastructure; see oracle/__init__.py).  All arithmetic in fp64.

Paper passages restated here
  * top-K sampling over the softmax classifier (Sec. 3.1; K = 2000 in Sec. 5.1)
  * acceptance test r < min(1, p/q), r ~ U[0,1]                       (Eq. 1)
  * calibrated resample from max(0, p - q) / sum max(0, p - q)         (Eq. 2)
  * re-draft of every later window position from this iteration's p   (Eq. 3)

Readings taken where the paper is silent
  * temperature T > 0 divides the logits before top-K (the paper has no
    temperature; T = 1 reproduces it);
  * top-K keeps every entry >= the K-th largest value, so ties at the
    threshold are all kept (the kept set may exceed K);
  * NaN and +inf logits are treated as -inf and the row is flagged; a row
    with no finite entry puts all mass on token 0;
  * sampling is by inverse CDF in token-index order;
  * q(x) = 0 with p(x) > 0 accepts always (ratio = +inf); 0/0 rejects;
  * an all-zero residual falls back to sampling from p and is flagged.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# kinds of draft-probability descriptor (the law the draft token was drawn from)
Q_ROW = 0      # q = warp(stored logits row of the previous iteration)   (Step 1 / Eq. 3)
Q_UNIFORM = 1  # q = 1/V: freshly initialised uniformly random token      (Sec. 4.2)
Q_ONEHOT = 2   # q = delta(draft): deterministic copy of a neighbour      (Sec. 4.2 (a), (b))

FLAG_NEAR_TIE_ACCEPT = 1     # |u - min(1, p/q)| below the comparison tolerance
FLAG_NEAR_TIE_SAMPLE = 2     # inverse-CDF target within tolerance of an interval edge
FLAG_RESIDUAL_EMPTY = 4      # sum max(0, p - q) == 0 at a rejected position
FLAG_NONFINITE = 8           # a logits row held NaN / +inf
FLAG_DONE = 16               # sequence has committed all its tokens


def sanitize(logits):
    """fp64 copy with NaN / +inf replaced by -inf; returns (row, had_bad)."""
    row = np.asarray(logits, dtype=np.float64).copy()
    bad = np.isnan(row) | (row == np.inf)
    row[bad] = -np.inf
    return row, bool(bad.any())


def warp(logits, temperature: float, top_k: int):
    """p = softmax over the top-K set of logits / T  (Sec. 3.1, top-K sampling).

    Returns the length-V probability vector (zeros outside the kept set)."""
    if not temperature > 0:
        raise ValueError("temperature must be > 0")
    if top_k < 1:
        raise ValueError("top_k must be >= 1")
    row, _ = sanitize(logits)
    v = row.shape[0]
    if not np.isfinite(row).any():
        p = np.zeros(v, dtype=np.float64)
        p[0] = 1.0
        return p
    s = row / float(temperature)
    if top_k < v:
        tau = np.sort(s)[v - top_k]          # K-th largest, counting multiplicity
        keep = s >= tau
    else:
        keep = np.ones(v, dtype=bool)
    keep &= np.isfinite(s)
    m = s[keep].max()
    w = np.zeros(v, dtype=np.float64)
    w[keep] = np.exp(s[keep] - m)
    return w / w.sum()


def icdf(weights, u: float):
    """Smallest index i (token order) with weights[i] > 0 and
    sum_{j<=i} weights[j] > u * sum(weights); if rounding leaves none, the
    largest index with positive weight.

    Returns (index, margin) where margin is the distance, in units of the
    total mass, from the target to the nearer edge of the chosen interval."""
    w = np.asarray(weights, dtype=np.float64)
    c = np.cumsum(w)
    total = c[-1]
    if not total > 0:
        raise ValueError("icdf needs positive total mass")
    target = float(u) * total
    hit = np.nonzero((w > 0) & (c > target))[0]
    if hit.size:
        i = int(hit[0])
    else:
        i = int(np.nonzero(w > 0)[0][-1])
    lo = (c[i] - w[i]) / total
    hi = c[i] / total
    margin = min(abs(float(u) - lo), abs(hi - float(u)))
    return i, margin


def guided_logits(logits_cond, logits_uncond, weight: float, storage: str = "f64"):
    """Classifier-free guidance (Sec. 5.1, implementation details: guidance weight 3.0 on every run):
    one logits row from the conditional and the unconditional stream of the same image,

        l = l_u + w * (l_c - l_u).

    w = 1 gives the conditional row, w = 0 the unconditional one.  The inputs are stored logits.
    `storage` names the dtype the mixed row is stored in before verification:
      'f64'          the plain formula in fp64;
      'f32', 'bf16'  the stored code is a decision taken from floating point, so it is taken in the
                     precision of the library's arithmetic: d = fl32(l_c - l_u), l = fl32(w * d + l_u)
                     with a single rounding (a fused multiply-add), then rounded to the storage dtype.
                     The product w * d of two fp32 numbers and its sum with a bf16 / fp32 value are
                     exact in fp64 for any logits of ordinary magnitude, so rounding the fp64 result to
                     fp32 is that single rounding.
    Returns fp64 values."""
    lc = np.asarray(logits_cond, dtype=np.float64)
    lu = np.asarray(logits_uncond, dtype=np.float64)
    if storage == "f64":
        return lu + float(weight) * (lc - lu)
    w32 = np.float64(np.float32(weight))
    with np.errstate(invalid="ignore", over="ignore"):
        d = (lc - lu).astype(np.float32).astype(np.float64)
        mixed = (w32 * d + lu).astype(np.float32)
    if storage == "f32":
        return mixed.astype(np.float64)
    if storage == "bf16":
        bits = np.ascontiguousarray(mixed).view(np.uint32).astype(np.uint64)
        rounded = ((bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1)))
                   >> np.uint64(16)) << np.uint64(16)
        out = rounded.astype(np.uint32).view(np.float32).astype(np.float64)
        return np.where(np.isfinite(mixed), out, mixed.astype(np.float64))
    raise ValueError(storage)


@dataclass
class QDesc:
    """The law a draft token was drawn from (Step 1: each draft carries the
    probability produced by the previous iteration)."""
    kind: int
    row: np.ndarray | None = None    # stored logits row when kind == Q_ROW

    def dist(self, draft: int, vocab: int, temperature: float, top_k: int):
        if self.kind == Q_ROW:
            return warp(self.row, temperature, top_k)
        if self.kind == Q_UNIFORM:
            return np.full(vocab, 1.0 / vocab, dtype=np.float64)
        if self.kind == Q_ONEHOT:
            q = np.zeros(vocab, dtype=np.float64)
            q[int(draft)] = 1.0
            return q
        raise ValueError("unknown q kind")


@dataclass
class VerifyResult:
    accept: list                      # acc_k for the scanned rows (up to and incl. the rejecting one)
    n_accepted: int                   # a: number of drafts accepted (first rejected index, or W_eff)
    committed: list                   # tokens fixed by this step (accepted drafts [+ resampled token])
    redraft: list                     # tokens for old positions a+1 .. W_eff-1 (Eq. 3)
    redraft_rows: list                # old row index of each re-drafted token
    flags: int = 0
    ratio: list = field(default_factory=list)          # min(1, p/q) per scanned row
    accept_margin: list = field(default_factory=list)  # |u - min(1, ratio)| per scanned row
    resample_margin: float | None = None
    redraft_margin: list = field(default_factory=list)
    p_draft: list = field(default_factory=list)        # p_k[d_k] for every row (diagnostic)
    q_draft: list = field(default_factory=list)        # q_k[d_k] for every row (diagnostic)


def verify_window(logits, drafts, qdescs, uniforms, temperature: float, top_k: int,
                  tie_tol_accept: float = 1e-4, tie_tol_sample: float = 2e-6) -> VerifyResult:
    """One verification scan over a window (Step 3 of Sec. 4.1).

    logits   [W_eff][V] stored logits of this iteration; row k predicts the
             token at window slot k
    drafts   [W_eff] draft tokens
    qdescs   [W_eff] QDesc of each draft
    uniforms [W_eff][3] (u_acc, u_res, u_draft) per slot
    """
    logits = np.asarray(logits)
    w_eff, vocab = logits.shape
    flags = 0
    res = VerifyResult(accept=[], n_accepted=w_eff, committed=[], redraft=[], redraft_rows=[])

    # diagnostics for every row (used by the parity tests on probabilities)
    for k in range(w_eff):
        p_k = warp(logits[k], temperature, top_k)
        q_k = qdescs[k].dist(drafts[k], vocab, temperature, top_k)
        res.p_draft.append(float(p_k[int(drafts[k])]))
        res.q_draft.append(float(q_k[int(drafts[k])]))
        if sanitize(logits[k])[1]:
            flags |= FLAG_NONFINITE

    # left-to-right scan, stopping at the first rejection (Eq. 1)
    a = w_eff
    for k in range(w_eff):
        d = int(drafts[k])
        p_k = warp(logits[k], temperature, top_k)
        q_k = qdescs[k].dist(d, vocab, temperature, top_k)
        pd, qd = p_k[d], q_k[d]
        if qd > 0:
            ratio = pd / qd
        else:
            ratio = np.inf if pd > 0 else 0.0
        thr = min(1.0, ratio)
        u_acc = float(uniforms[k][0])
        acc = u_acc < thr
        res.accept.append(bool(acc))
        res.ratio.append(float(thr))
        res.accept_margin.append(abs(u_acc - thr))
        if abs(u_acc - thr) < tie_tol_accept and thr < 1.0:
            flags |= FLAG_NEAR_TIE_ACCEPT
        if acc:
            res.committed.append(d)
            continue
        a = k
        # calibrated resample at the first rejected position (Eq. 2)
        r = np.maximum(0.0, p_k - q_k)
        u_res = float(uniforms[k][1])
        if r.sum() > 0:
            t, margin = icdf(r, u_res)
        else:
            flags |= FLAG_RESIDUAL_EMPTY
            t, margin = icdf(p_k, u_res)
        res.resample_margin = margin
        if margin < tie_tol_sample:
            flags |= FLAG_NEAR_TIE_SAMPLE
        res.committed.append(int(t))
        break
    res.n_accepted = a

    # refinement: every later slot is re-drawn from this iteration's p (Eq. 3)
    for k in range(a + 1, w_eff):
        p_k = warp(logits[k], temperature, top_k)
        t, margin = icdf(p_k, float(uniforms[k][2]))
        res.redraft.append(int(t))
        res.redraft_rows.append(k)
        res.redraft_margin.append(margin)
        if margin < tie_tol_sample:
            flags |= FLAG_NEAR_TIE_SAMPLE
    res.flags = flags
    return res
