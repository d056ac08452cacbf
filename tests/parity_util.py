"""Comparison rules between the CUDA library's outputs and the CPU checker (test helper).

Decisions (accept flags, first rejection, fixed tokens, re-drawn tokens, laws) must be bit-exact,
except where the checker's own fp64 margin says the decision sits within rounding distance of its
boundary: |u - min(1, p/q)| < 1e-4 for an acceptance test, or an inverse-CDF target within
TOL_SAMPLE (in units of the sampled mass; for the residual of Eq. 2 the mass can be small, so the
tolerance is scaled by 1/mass) of an interval edge.  Such decisions are counted as flagged, not
failed, and everything downstream of a flagged decision in the same sequence is skipped.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from oracle import philox
from oracle.sampling import Q_ROW, QDesc, verify_window, warp

TOL_ACCEPT = 1e-4
TOL_SAMPLE = 2e-6


@dataclass
class ParityStats:
    sequences: int = 0
    decisions: int = 0
    flagged: int = 0
    skipped_sequences: int = 0

    def merge(self, other):
        self.sequences += other.sequences
        self.decisions += other.decisions
        self.flagged += other.flagged
        self.skipped_sequences += other.skipped_sequences


def residual_mass(logits_row, qdesc: QDesc, draft, temperature, top_k):
    p = warp(logits_row, temperature, top_k)
    q = qdesc.dist(draft, p.shape[0], temperature, top_k)
    return float(np.maximum(0.0, p - q).sum())


def compare_window(vr, gpu, logits, drafts, qdescs, temperature, top_k, prob_tol, where="") -> ParityStats:
    """vr: oracle VerifyResult for one sequence; gpu: dict with this sequence's n_accepted,
    committed [W], draft [W] (re-drawn tokens, left aligned), q_draft [W], kept (number of
    re-drawn tokens to compare).  Returns counts; raises AssertionError on a real mismatch."""
    st = ParityStats(sequences=1)
    w_eff = len(drafts)
    a_o, a_g = vr.n_accepted, int(gpu["n_accepted"])
    # acceptance decisions up to the first rejection of either side
    upto = min(a_o, a_g)
    st.decisions += min(w_eff, upto + 1)
    if a_o != a_g:
        k = upto  # the row where the two sides disagree
        margin = vr.accept_margin[k] if k < len(vr.accept_margin) else None
        if margin is None:
            # oracle accepted everything it scanned up to k... recompute margin for row k
            raise AssertionError(f"{where}: n_accepted {a_g} vs oracle {a_o}, no margin for row {k}")
        assert margin < TOL_ACCEPT, f"{where}: n_accepted {a_g} vs oracle {a_o}, margin {margin:.3e} at row {k}"
        st.flagged += 1
        st.skipped_sequences += 1
        return st
    com_g = [int(t) for t in gpu["committed"][:len(vr.committed)]]
    assert com_g[:a_o] == vr.committed[:a_o], f"{where}: accepted tokens differ"
    if a_o < w_eff:
        st.decisions += 1
        if com_g[a_o] != vr.committed[a_o]:
            mass = residual_mass(logits[a_o], qdescs[a_o], drafts[a_o], temperature, top_k)
            tol = max(TOL_SAMPLE, 1e-6 / max(mass, 1e-30))
            assert vr.resample_margin < tol, (f"{where}: resampled token {com_g[a_o]} vs oracle {vr.committed[a_o]}, "
                                              f"margin {vr.resample_margin:.3e}, residual mass {mass:.3e}")
            st.flagged += 1
    assert all(int(t) == -1 for t in gpu["committed"][len(vr.committed):]), f"{where}: committed tail not -1"
    kept = int(gpu.get("kept", len(vr.redraft)))
    for s in range(min(kept, len(vr.redraft))):
        st.decisions += 1
        tok_g = int(gpu["draft"][s])
        if tok_g != vr.redraft[s]:
            assert vr.redraft_margin[s] < TOL_SAMPLE, (f"{where}: re-draft slot {s}: {tok_g} vs oracle {vr.redraft[s]}, "
                                                       f"margin {vr.redraft_margin[s]:.3e}")
            st.flagged += 1
            continue
        k = vr.redraft_rows[s]
        p_tok = warp(logits[k], temperature, top_k)[tok_g]
        assert abs(float(gpu["q_draft"][s]) - p_tok) <= prob_tol + 1e-4 * p_tok, \
            f"{where}: q of re-draft slot {s}: {gpu['q_draft'][s]} vs {p_tok}"
    return st


def oracle_verify_case(case, b):
    """Run the checker on sequence b of an inputs.VerifyCase; returns (VerifyResult, qdescs)."""
    w = case.window
    qdescs = [QDesc(int(case.q_kind[b, k]), row=case.logits_prev[b, k].astype(np.float64)
                    if int(case.q_kind[b, k]) == Q_ROW else None) for k in range(w)]
    uniforms = [philox.verify_uniforms(case.seed, int(case.base_pos[b]) + k, case.step, b) for k in range(w)]
    vr = verify_window(case.logits_cur[b].astype(np.float64), case.draft[b], qdescs, uniforms, case.temperature,
                       case.top_k)
    return vr, qdescs


# ---------------------------------------------------------------------------------------------
# end-to-end lock-step: the checker re-runs every step from the library's pre-step state
# ---------------------------------------------------------------------------------------------
def storage_half_ulp(x, dtype):
    """Half a unit in the last place of |x| in the storage dtype (bf16: 8 significant bits)."""
    bits = {"bf16": 8, "f32": 24}[dtype]
    mag = np.maximum(np.abs(x), 1e-30)
    return 0.5 * 2.0 ** (np.floor(np.log2(mag)) - (bits - 1))


def oracle_model_cfg(wl):
    from oracle.model import ModelCfg
    return ModelCfg(wl.n_layers, wl.d_model, wl.n_heads, wl.n_kv_heads, wl.head_dim, wl.ffn_hidden, wl.vocab,
                    wl.rope_theta, wl.rms_eps)


class LogitErrors:
    """Running summary of |checker - library| over every compared logit: the largest difference, the
    largest difference beyond half a unit in the last place of the stored value, and how many logits lie
    beyond 1e-2 / 1.5e-2 / 2e-2 (each plus that half unit)."""
    BARS = (1e-2, 1.5e-2, 2e-2)

    def __init__(self):
        self.total = 0
        self.max_abs = 0.0
        self.max_excess = 0.0
        self.beyond = [0, 0, 0]

    def add(self, diff, half_ulp):
        excess = diff - half_ulp
        self.total += int(diff.size)
        self.max_abs = max(self.max_abs, float(diff.max()))
        self.max_excess = max(self.max_excess, float(excess.max()))
        for i, bar in enumerate(self.BARS):
            self.beyond[i] += int((excess > bar).sum())

    def line(self, label):
        return ("%s: max |diff| %.3e, beyond half a storage ulp %.3e; of %d logits %d / %d / %d beyond "
                "1e-2 / 1.5e-2 / 2e-2" % (label, self.max_abs, self.max_excess, self.total, *self.beyond))


class LockStepSequence:
    """One sequence of a batch followed by the checker.  With `also_plain_cache` a second copy of the
    checker's model keeps its K/V cache unrounded (the plain definition of the forward pass); its logits
    are only measured (`errors_plain`), the decisions and the asserted tolerance stay with the checker
    whose cache is rounded to the storage dtype."""

    def __init__(self, wl, weights_cpu, prompt_row, scfg, seq_id, logit_tol, also_plain_cache=False, guidance=0.0,
                 prompt_uncond=None):
        """With guidance != 0 the sequence is an image with two streams (prompt_row: the conditional
        prompt, prompt_uncond: the unconditional one); `step` then takes the library's stored logits of
        both streams, checks each against the checker's stream and re-takes the decisions from their
        mix (oracle.sampling.guided_logits in the storage dtype)."""
        from oracle.model import OracleModel
        from oracle.sjd import CachedModel, GuidedModel, sjd_begin
        self.wl, self.scfg, self.tol = wl, scfg, logit_tol
        om = OracleModel(oracle_model_cfg(wl), weights_cpu)
        self.model = CachedModel(om, wl.prompt_len + scfg.n_generate + 1, kv_storage=wl.dtype)
        self.guidance = float(guidance)
        if self.guidance != 0.0:
            uncond = CachedModel(om, wl.prompt_len + scfg.n_generate + 1, kv_storage=wl.dtype)
            self.model = GuidedModel(self.model, uncond, prompt_uncond, self.guidance, wl.dtype)
        self.prompt = [int(t) for t in prompt_row]
        self.model.prefill(self.prompt)
        self.errors = LogitErrors()
        self.errors_plain = None
        self.plain = None
        if also_plain_cache and wl.dtype != "f32":
            self.plain = CachedModel(om, wl.prompt_len + scfg.n_generate + 1, kv_storage="f64")
            self.plain.prefill(self.prompt)
            self.errors_plain = LogitErrors()
        self.st = sjd_begin(self.prompt, scfg, wl.vocab, seq=seq_id)
        self.stats = ParityStats(sequences=1)
        self.max_logit_err = 0.0
        self.max_logit_excess = 0.0      # largest |diff| beyond half a storage ulp
        self.steps = 0

    def logit_failures(self, diff, half_ulp):
        """Mask of logits beyond the tolerance (a test of deeper models may state a different rule)."""
        return diff > self.tol + half_ulp

    def check_window(self, draft_row, kind_row, q_row, total):
        w_eff = len(self.st.drafts)
        assert int(total) == self.st.n
        assert [int(t) for t in draft_row[:w_eff]] == self.st.drafts, "window drafts differ"
        # (the library tells a row of the other logits buffer, 0, from a retained row, 3: the same kind of law)
        assert [0 if int(t) == 3 else int(t) for t in kind_row[:w_eff]] == [q.kind for q in self.st.qdescs], \
            "window laws differ"
        assert all(int(t) == -1 for t in draft_row[w_eff:])
        from oracle.sjd import q_of_draft
        for k in range(w_eff):
            qo = q_of_draft(self.st.qdescs[k], self.st.drafts[k], self.wl.vocab, self.scfg)
            assert abs(float(q_row[k]) - qo) <= 1e-5 + 1e-4 * qo, f"q of slot {k}: {q_row[k]} vs {qo}"

    def step(self, gpu_logits_rows, out_b, check_logits=True):
        """gpu_logits_rows: [W][V] float64 array of the library's stored logits for this sequence;
        out_b: dict of this sequence's step outputs."""
        from oracle.model import round_to_storage
        from oracle.sampling import Q_ROW, QDesc
        from oracle.sjd import sjd_step
        st, scfg, vocab = self.st, self.scfg, self.wl.vocab
        w_eff = len(st.drafts)
        if w_eff == 0:
            assert int(out_b["n_committed"]) == 0 and int(out_b["flags"]) & 16
            return
        self.steps += 1
        drafts, qdescs = list(st.drafts), list(st.qdescs)
        if self.guidance != 0.0:
            from oracle.sampling import guided_logits
            gpu_c, gpu_u = gpu_logits_rows
            if check_logits:
                own_c, own_u = self.model.stream_logits(st.committed, st.drafts[:w_eff - 1])
                for own, got in ((own_c, gpu_c), (own_u, gpu_u)):
                    # (the checker's streams are already rounded to the storage dtype: compare values)
                    diff = np.abs(own - got[:w_eff])
                    self.max_logit_err = max(self.max_logit_err, float(diff.max()))
                    half_ulp = storage_half_ulp(own, scfg.logits_dtype)
                    self.max_logit_excess = max(self.max_logit_excess, float((diff - half_ulp).max()))
                    self.errors.add(diff, half_ulp)
                    assert not self.logit_failures(diff, half_ulp).any(), f"step {self.steps}: stream logits off"
            gpu_logits_rows = guided_logits(gpu_c[:w_eff], gpu_u[:w_eff], self.guidance, scfg.logits_dtype)
            check_logits = False
        if check_logits:
            own = self.model.step_logits(st.committed, st.drafts[:w_eff - 1])
            # the library's value is its fp32 result rounded to the storage dtype: allow the stated
            # tolerance on the unrounded value plus half a unit in the last place of the stored one
            diff = np.abs(own - gpu_logits_rows[:w_eff])
            err = float(diff.max())
            self.max_logit_err = max(self.max_logit_err, err)
            half_ulp = storage_half_ulp(own, scfg.logits_dtype)
            self.max_logit_excess = max(self.max_logit_excess, float((diff - half_ulp).max()))
            self.errors.add(diff, half_ulp)
            if self.plain is not None:
                plain = self.plain.step_logits(st.committed, st.drafts[:w_eff - 1])
                self.errors_plain.add(np.abs(plain - gpu_logits_rows[:w_eff]),
                                      storage_half_ulp(plain, scfg.logits_dtype))
            bad = self.logit_failures(diff, half_ulp)
            assert not bad.any(), (f"step {self.steps}: {int(bad.sum())} logits off by more than {self.tol} "
                                   f"+ half a storage ulp; max |diff| {err:.3e}")
        n_before = st.n
        rec = sjd_step(st, None, scfg, vocab, logits_override=gpu_logits_rows[:w_eff])
        vr = rec.verify
        gpu = dict(n_accepted=out_b["n_accepted"], committed=out_b["committed"], draft=out_b["draft"],
                   q_draft=out_b["q_draft"], kept=sum(1 for k in rec.kinds if k == Q_ROW))
        before = self.stats.flagged
        ps = compare_window(vr, gpu, gpu_logits_rows[:w_eff], drafts, qdescs, scfg.temperature, scfg.top_k,
                            prob_tol=1e-5, where=f"step {self.steps}")
        self.stats.merge(ParityStats(0, ps.decisions, ps.flagged, ps.skipped_sequences))
        if self.stats.flagged == before:
            # no near-tie: the whole new window (incl. freshly initialised slots) must match
            assert int(out_b["n_committed"]) == len(rec.committed)
            self.check_window(out_b["draft"], out_b["q_kind"], out_b["q_draft"], out_b["total_committed"])
            done = st.n >= self.wl.prompt_len + scfg.n_generate
            assert bool(int(out_b["flags"]) & 16) == done
            return
        # a flagged decision: follow the library so that later steps stay comparable
        m = int(out_b["n_committed"])
        a = int(out_b["n_accepted"])
        st.committed = st.committed[:n_before] + [int(t) for t in out_b["committed"][:m]]
        new_w = max(0, min(scfg.window, self.wl.prompt_len + scfg.n_generate - st.n))
        # the slots re-drawn by Eq. 3 follow the library (rows a+1 ..); the slots that enter the window are
        # a function of the state alone, so the checker initialises them itself and the windows are compared
        from oracle.sjd import SCHEDULE_NO_REFINE, _fill_window
        redrawn = 0 if scfg.schedule == SCHEDULE_NO_REFINE else max(0, min(w_eff - a - 1, new_w))
        st.drafts = [int(t) for t in out_b["draft"][:redrawn]]
        st.qdescs = [QDesc(Q_ROW, row=np.array(gpu_logits_rows[a + 1 + s], dtype=np.float64)) for s in range(redrawn)]
        _fill_window(st, scfg, vocab, st.step - 1)
        self.check_window(out_b["draft"], out_b["q_kind"], out_b["q_draft"], out_b["total_committed"])
