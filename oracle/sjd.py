"""Speculative Jacobi Decoding state machine (test infrastructure; see
oracle/__init__.py).  Follows Sec. 4.1 Steps 1-4 and Sec. 4.2 in the paper's
order; plain auto-regressive sampling (Sec. 3.1) and greedy Jacobi decoding
(Sec. 3.2) are included as the special cases the paper relates SJD to.

Conventions fixed here (0-indexed)
  * c[0..n) are fixed tokens (prompt of P tokens, then accepted tokens); the
    window holds W_eff = min(W, P + N - n) drafts d_k for positions n + k.
  * One step feeds [c[n-1], d_0 .. d_{W_eff-2}] at positions n-1 .. n+W_eff-2
    (the KV cache therefore holds rows for c[0..n-1)); logits row k predicts
    position n + k.  Rows are rounded to their storage dtype before use.
  * The token drawn by Eq. 2 is fixed at once together with the accepted
    prefix, so every step fixes at least one token.
  * A freshly initialised slot carries the law it was drawn from: uniform
    1/V for a random token, a point mass for a copied neighbour.
  * Uniforms: Philox4x32-10 keyed by the seed, counter = (absolute position,
    step index, sequence id, stream tag); see oracle/philox.py.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import philox
from .model import KVCache, OracleModel, round_to_storage
from .sampling import (FLAG_DONE, Q_ONEHOT, Q_ROW, Q_UNIFORM, QDesc, VerifyResult, guided_logits, icdf,
                       verify_window, warp)

INIT_RANDOM = 0       # Sec. 4.2: uniform random candidate
INIT_COPY_ABOVE = 1   # Sec. 4.2 (b): repeat the token one grid row above
INIT_COPY_LEFT = 2    # Sec. 4.2 (a): repeat the left neighbour
INIT_RESAMPLE_LEFT = 3   # Sec. 4.2 (c): draw from the distribution predicted at the left neighbour
INIT_RESAMPLE_ABOVE = 4  # Sec. 4.2 (d): draw from the distribution predicted one grid row above

SCHEDULE_SJD = 0        # Sec. 4.1: probabilistic criterion (Eqs. 1-3)
SCHEDULE_JACOBI = 1     # Sec. 3.2: every slot re-drawn each pass, a slot is fixed once its token no longer changes
SCHEDULE_NO_REFINE = 2  # appendix "effectiveness" ablation: Eqs. 1-2 only, unaccepted slots are re-initialised


@dataclass
class SampleCfg:
    temperature: float = 1.0
    top_k: int = 2000
    seed: int = 0
    window: int = 16
    init: int = INIT_RANDOM
    grid_stride: int = 0       # tokens per image row (incl. any row-end token)
    n_generate: int = 0
    logits_dtype: str = "f32"  # storage dtype of the logits: 'f32' or 'bf16'
    schedule: int = SCHEDULE_SJD


@dataclass
class SJDState:
    prompt_len: int
    committed: list                    # c[0..n)
    drafts: list = field(default_factory=list)
    qdescs: list = field(default_factory=list)
    step: int = 0
    seq: int = 0
    flags: int = 0
    rows: dict = field(default_factory=dict)   # position -> the most recent stored logits row that predicted it

    @property
    def n(self) -> int:
        return len(self.committed)


@dataclass
class StepRecord:
    n_accepted: int
    committed: list
    drafts: list
    kinds: list
    flags: int
    verify: VerifyResult | None
    logits: np.ndarray | None          # stored logits rows of this step [W_eff][V]
    q_draft: list = field(default_factory=list)   # q(d) of each new draft under its own descriptor


# ----------------------------------------------------------------------------------------------
# models: anything with  prefill(prompt)  and
#                        step_logits(committed, drafts_in) -> [len(drafts_in)+1][V]
# ----------------------------------------------------------------------------------------------
class CachedModel:
    """OracleModel driven with a KV cache: rows for c[0..n-1) stay cached, the
    rejected tail is rolled back by truncation (stale rows are overwritten)."""

    def __init__(self, model: OracleModel, capacity: int, kv_storage: str = "f64"):
        self.model = model
        self.cache: KVCache = model.new_cache(capacity, kv_storage)

    def prefill(self, prompt):
        self.cache.truncate(0)
        if len(prompt) > 1:
            self.model.forward_window(self.cache, prompt[:-1], 0, want_logits=False)

    def step_logits(self, committed, drafts_in):
        n = len(committed)
        self.cache.truncate(n - 1)
        return self.model.forward_window(self.cache, [committed[-1]] + list(drafts_in), n - 1)


class RecomputeModel:
    """Same function without a cache: full causal forward of everything."""

    def __init__(self, model: OracleModel):
        self.model = model

    def prefill(self, prompt):
        pass

    def step_logits(self, committed, drafts_in):
        full = self.model.forward_full(list(committed) + list(drafts_in))
        return full[len(committed) - 1:]


class GuidedModel:
    """Two streams of one image under classifier-free guidance (Sec. 5.1): the conditional stream
    sees the text prompt, the unconditional one a prompt of its own (same length); both see the same
    image tokens.  Every stream's logits are stored in `storage` first, then mixed row by row
    (sampling.guided_logits) and stored again; drafts, uniforms and every decision are shared, since
    there is one verification per image, on the mixed rows."""

    def __init__(self, model_cond, model_uncond, prompt_uncond, weight: float, storage: str = "f32"):
        self.mc, self.mu = model_cond, model_uncond
        self.prompt_u = [int(t) for t in prompt_uncond]
        self.weight, self.storage = float(weight), storage
        self.p_len = None

    def prefill(self, prompt):
        assert len(prompt) == len(self.prompt_u), "both streams use prompts of one length"
        self.p_len = len(prompt)
        self.mc.prefill(list(prompt))
        self.mu.prefill(list(self.prompt_u))

    def stream_logits(self, committed, drafts_in):
        """Stored logits of the two streams, (conditional, unconditional)."""
        image = list(committed[self.p_len:])
        lc = round_to_storage(self.mc.step_logits(list(committed), drafts_in), self.storage)
        lu = round_to_storage(self.mu.step_logits(self.prompt_u + image, drafts_in), self.storage)
        return lc, lu

    def step_logits(self, committed, drafts_in):
        lc, lu = self.stream_logits(committed, drafts_in)
        return guided_logits(lc, lu, self.weight, self.storage)


class TableModel:
    """Tiny context-dependent categorical model for brute-force pins:
    logits(prefix) = table[index of the last `order` tokens]."""

    def __init__(self, vocab: int, order: int, seed: int, scale: float = 1.5):
        rng = np.random.default_rng(seed)
        self.vocab, self.order = vocab, order
        self.table = rng.normal(0.0, scale, size=(vocab ** order, vocab))

    def logits_after(self, prefix):
        ctx = [0] * self.order + [int(t) for t in prefix]
        idx = 0
        for t in ctx[-self.order:]:
            idx = idx * self.vocab + t
        return self.table[idx]

    def prefill(self, prompt):
        pass

    def step_logits(self, committed, drafts_in):
        seq = list(committed) + list(drafts_in)
        n = len(committed)
        return np.stack([self.logits_after(seq[:n + k]) for k in range(len(drafts_in) + 1)])


# ----------------------------------------------------------------------------------------------
# window construction (Step 4, Sec. 4.2)
# ----------------------------------------------------------------------------------------------
def _fresh_slot(state: SJDState, drafts, scfg: SampleCfg, vocab: int, t_pos: int, step_tag: int):
    """Token and q descriptor for a newly initialised slot at absolute position t_pos.
    `drafts` are the slots of the new window already filled (positions n .. t_pos-1).

    Strategies (c) and (d) draw the token from the distribution the model predicted at a neighbour's
    position.  Reading: "predicted" is the most recent logits row computed for that position (the pass in
    which the position was last inside the window); the slot's law is then that row's top-k softmax,
    which is what Theorem 1 needs as q.  (c): the neighbour is the nearest position to the left that has
    ever been through a pass (a slot appended in this very step has not); (d): the position one grid row
    above.  Without such a row (the first window, the first image row) the slot is a uniform random token."""
    if scfg.init in (INIT_RESAMPLE_LEFT, INIT_RESAMPLE_ABOVE):
        if scfg.init == INIT_RESAMPLE_LEFT:
            src = t_pos - 1
            while src >= state.prompt_len and src not in state.rows:
                src -= 1
        else:
            src = t_pos - scfg.grid_stride
        row = state.rows.get(src) if src >= state.prompt_len else None
        if row is not None:
            u = philox.init_uniform(scfg.seed, t_pos, step_tag, state.seq)
            tok, _ = icdf(warp(row, scfg.temperature, scfg.top_k), u)
            return int(tok), QDesc(Q_ROW, row=row.copy())
        tok = philox.init_token(scfg.seed, t_pos, step_tag, state.seq, vocab)
        return int(tok), QDesc(Q_UNIFORM)
    stride = {INIT_COPY_ABOVE: scfg.grid_stride, INIT_COPY_LEFT: 1}.get(scfg.init, 0)
    src = t_pos - stride
    if scfg.init != INIT_RANDOM and stride > 0 and src >= state.prompt_len:
        n = state.n
        tok = state.committed[src] if src < n else drafts[src - n]
        return int(tok), QDesc(Q_ONEHOT)
    tok = philox.init_token(scfg.seed, t_pos, step_tag, state.seq, vocab)
    return int(tok), QDesc(Q_UNIFORM)


def _fill_window(state: SJDState, scfg: SampleCfg, vocab: int, step_tag: int):
    w_eff = max(0, min(scfg.window, state.prompt_len + scfg.n_generate - state.n))
    del state.drafts[w_eff:]
    del state.qdescs[w_eff:]
    while len(state.drafts) < w_eff:
        t_pos = state.n + len(state.drafts)
        tok, qd = _fresh_slot(state, state.drafts, scfg, vocab, t_pos, step_tag)
        state.drafts.append(tok)
        state.qdescs.append(qd)


def sjd_begin(prompt, scfg: SampleCfg, vocab: int, seq: int = 0) -> SJDState:
    """State after pre-filling the prompt: an all-fresh first window (Sec. 4.1:
    the method starts with a window of initialised candidate tokens)."""
    assert len(prompt) >= 1
    st = SJDState(prompt_len=len(prompt), committed=[int(t) for t in prompt], seq=seq)
    _fill_window(st, scfg, vocab, philox.STEP_INITIAL_WINDOW)
    return st


def q_of_draft(qd: QDesc, draft: int, vocab: int, scfg: SampleCfg) -> float:
    return float(qd.dist(draft, vocab, scfg.temperature, scfg.top_k)[int(draft)])


def sjd_step(state: SJDState, model, scfg: SampleCfg, vocab: int, logits_override=None) -> StepRecord:
    """One SJD iteration (Steps 1-4).  `logits_override` replaces the forward
    pass by externally supplied stored logits rows (lock-step comparisons)."""
    n = state.n
    w_eff = len(state.drafts)
    if w_eff == 0:
        state.flags |= FLAG_DONE
        return StepRecord(0, [], [], [], FLAG_DONE, None, None)
    j = state.step

    # Step 2: one forward pass over the window
    if logits_override is not None:
        stored = np.asarray(logits_override, dtype=np.float64)[:w_eff]
    else:
        raw = model.step_logits(state.committed, state.drafts[:w_eff - 1])
        stored = round_to_storage(raw, scfg.logits_dtype)

    for k in range(w_eff):   # the most recent prediction for every position of the window (Sec. 4.2 (c), (d))
        state.rows[n + k] = stored[k]
    # Step 3: verification scan, calibrated resample, refinement
    if scfg.schedule == SCHEDULE_JACOBI:
        vr = jacobi_window(stored, state.drafts, scfg, n, state.seq)
    else:
        uniforms = [philox.verify_uniforms(scfg.seed, n + k, j, state.seq) for k in range(w_eff)]
        vr = verify_window(stored, state.drafts, state.qdescs, uniforms, scfg.temperature, scfg.top_k)
        if scfg.schedule == SCHEDULE_NO_REFINE:
            # no refinement: the slots after the rejection are not re-drawn from this pass's rows (Eq. 3) but
            # replaced by newly initialised tokens, like the slots that enter the window
            vr.redraft, vr.redraft_rows, vr.redraft_margin = [], [], []

    # fixed tokens grow by the accepted prefix (+ the resampled token)
    state.committed.extend(vr.committed)
    # Step 4: unaccepted (re-drawn) tokens carry this iteration's rows as their q
    state.drafts = list(vr.redraft)
    state.qdescs = [QDesc(Q_ROW, row=stored[k].copy()) for k in vr.redraft_rows]
    state.step = j + 1
    _fill_window(state, scfg, vocab, j)
    flags = vr.flags
    if state.n >= state.prompt_len + scfg.n_generate:
        flags |= FLAG_DONE
    state.flags |= flags
    return StepRecord(
        n_accepted=vr.n_accepted, committed=list(vr.committed), drafts=list(state.drafts),
        kinds=[qd.kind for qd in state.qdescs], flags=flags, verify=vr, logits=stored,
        q_draft=[q_of_draft(qd, d, vocab, scfg) for qd, d in zip(state.qdescs, state.drafts)])


def jacobi_window(stored, drafts, scfg: SampleCfg, n: int, seq: int) -> VerifyResult:
    """One pass of Jacobi decoding with sampling (Sec. 3.2): every slot k is re-drawn from this pass's
    row, x'_k = icdf(warp(row_k), u_k); the longest prefix of slots whose token did not change is fixed
    (the deterministic criterion), and so is the first changed slot, whose context is fixed by then.
    Reading: the draw of a position uses the same uniform in every pass (a function of the position,
    not of the pass: the re-draft word of the Philox block with step index 0), which is what makes
    "unchanged between consecutive iterations" a fixed point: the iteration then converges to the
    image ordinary sampling would produce from the same per-position uniforms."""
    w_eff = len(drafts)
    res = VerifyResult(accept=[], n_accepted=w_eff, committed=[], redraft=[], redraft_rows=[])
    new, margins = [], []
    for k in range(w_eff):
        u = philox.verify_uniforms(scfg.seed, n + k, 0, seq)[2]
        t, margin = icdf(warp(stored[k], scfg.temperature, scfg.top_k), u)
        new.append(int(t))
        margins.append(margin)
    a = 0
    while a < w_eff and new[a] == int(drafts[a]):
        a += 1
    res.n_accepted = a
    res.accept = [True] * a + ([False] if a < w_eff else [])
    res.accept_margin = margins[:a + 1]        # a changed token is a changed inverse-CDF draw
    res.ratio = [1.0] * a + ([0.0] if a < w_eff else [])
    res.committed = [int(d) for d in drafts[:a]] + ([new[a]] if a < w_eff else [])
    if a < w_eff:
        res.resample_margin = margins[a]
    res.redraft = new[a + 1:]
    res.redraft_rows = list(range(a + 1, w_eff))
    res.redraft_margin = margins[a + 1:]
    return res


def sjd_generate(prompt, model, scfg: SampleCfg, vocab: int, seq: int = 0, max_steps=None):
    """Run SJD until N tokens are fixed.  Returns (generated tokens, number of
    forward passes, per-step committed counts)."""
    model.prefill(list(prompt))
    st = sjd_begin(prompt, scfg, vocab, seq)
    steps, accepted = 0, []
    target = len(prompt) + scfg.n_generate
    while st.n < target:
        rec = sjd_step(st, model, scfg, vocab)
        steps += 1
        accepted.append(len(rec.committed))
        if max_steps is not None and steps >= max_steps:
            break
    return st.committed[len(prompt):], steps, accepted


def ar_generate(prompt, model, scfg: SampleCfg, vocab: int, seq: int = 0, fixed_step=None):
    """Ordinary next-token sampling (Sec. 3.1): one forward pass per token.
    Token at position t uses the re-draft uniform of (t, step = t - P), or of (t, fixed_step) when
    a fixed step index is given (the per-position uniforms of the Jacobi schedule)."""
    model.prefill(list(prompt))
    c = [int(t) for t in prompt]
    p_len = len(prompt)
    for i in range(scfg.n_generate):
        row = round_to_storage(model.step_logits(c, []), scfg.logits_dtype)[0]
        u = philox.verify_uniforms(scfg.seed, len(c), i if fixed_step is None else fixed_step, seq)[2]
        tok, _ = icdf(warp(row, scfg.temperature, scfg.top_k), u)
        c.append(tok)
    return c[p_len:], scfg.n_generate


def greedy_ar_generate(prompt, model, n_generate: int, logits_dtype: str = "f32"):
    model.prefill(list(prompt))
    c = [int(t) for t in prompt]
    for _ in range(n_generate):
        row = round_to_storage(model.step_logits(c, []), logits_dtype)[0]
        c.append(int(np.argmax(row)))
    return c[len(prompt):]


def jacobi_generate(prompt, model, n_generate: int, window: int, vocab: int, seed: int = 0,
                    logits_dtype: str = "f32", seq: int = 0):
    """Greedy Jacobi decoding (Sec. 3.2): every window slot is replaced by the
    argmax of its row each iteration; the prefix of slots that did not change
    is fixed, and so is the first changed slot (its context is already fixed).
    New slots are random tokens drawn exactly as SJD's random initialisation
    draws them.  Returns (tokens, forward passes)."""
    model.prefill(list(prompt))
    c = [int(t) for t in prompt]
    p_len = len(prompt)
    total = p_len + n_generate

    def refill(drafts, step_tag):
        w_eff = min(window, total - len(c))
        drafts = drafts[:w_eff]
        while len(drafts) < w_eff:
            drafts.append(philox.init_token(seed, len(c) + len(drafts), step_tag, seq, vocab))
        return drafts

    drafts = refill([], philox.STEP_INITIAL_WINDOW)
    passes = 0
    while len(c) < total:
        rows = round_to_storage(model.step_logits(c, drafts[:-1]), logits_dtype)
        new = [int(np.argmax(r)) for r in rows]
        a = 0
        while a < len(drafts) and drafts[a] == new[a]:
            a += 1
        fixed = new[:a + 1] if a < len(drafts) else new[:a]
        c.extend(fixed)
        drafts = refill(new[len(fixed):], passes)
        passes += 1
    return c[p_len:], passes
