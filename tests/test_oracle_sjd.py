"""Pins for the CPU checker's SJD state machine: the special cases the paper
fixes (window of one = ordinary sampling, top-1 = greedy Jacobi = greedy
auto-regressive decoding, forward passes never exceed tokens), the exactness
theorem by brute-force enumeration of the joint distribution, and the window
bookkeeping of Step 4 / Sec. 4.2 on hand-built cases.  No GPU."""
import itertools

import numpy as np
import pytest
from scipy import stats

from oracle import philox
from oracle.model import ModelCfg, OracleModel
from oracle.sampling import Q_ONEHOT, Q_ROW, Q_UNIFORM, warp
from oracle.sjd import (INIT_COPY_ABOVE, INIT_COPY_LEFT, INIT_RANDOM, INIT_RESAMPLE_ABOVE, INIT_RESAMPLE_LEFT,
                        SCHEDULE_JACOBI, SCHEDULE_NO_REFINE,
                        CachedModel, RecomputeModel, SampleCfg, TableModel, ar_generate, greedy_ar_generate,
                        jacobi_generate, sjd_begin, sjd_generate, sjd_step)


def _tiny_model(seed=0, vocab=96):
    cfg = ModelCfg(n_layers=2, d_model=32, n_heads=4, n_kv_heads=2, head_dim=8, ffn_hidden=45, vocab=vocab)
    rng = np.random.default_rng(seed)
    mat = lambda o, i: rng.normal(0, 0.6, size=(o, i))
    layers = [dict(attn_norm=np.ones(32), wq=mat(32, 32), wk=mat(16, 32), wv=mat(16, 32), wo=mat(32, 32),
                   ffn_norm=np.ones(32), w_gate=mat(45, 32), w_up=mat(45, 32), w_down=mat(32, 45))
              for _ in range(2)]
    w = dict(tok_emb=mat(vocab, 32), final_norm=np.ones(32), lm_head=mat(vocab, 32), layers=layers)
    return cfg, OracleModel(cfg, w)


def _exact_joint(table: TableModel, prompt, n_gen, temperature, top_k):
    v = table.vocab
    joint = {}
    for seq in itertools.product(range(v), repeat=n_gen):
        pr, ctx = 1.0, list(prompt)
        for t in seq:
            pr *= warp(table.logits_after(ctx), temperature, top_k)[t]
            ctx.append(t)
        joint[seq] = pr
    return joint


def _chi_square_joint(counts: dict, joint: dict, n_runs: int):
    keys = sorted(joint)
    exp = np.array([joint[k] * n_runs for k in keys])
    obs = np.array([counts.get(k, 0) for k in keys], dtype=float)
    assert all(k in joint and joint[k] > 0 for k in counts), "sampled a zero-probability sequence"
    big = exp >= 5
    obs_m = np.append(obs[big], obs[~big].sum())
    exp_m = np.append(exp[big], exp[~big].sum())
    if exp_m[-1] == 0:
        obs_m, exp_m = obs_m[:-1], exp_m[:-1]
    return stats.chisquare(obs_m, exp_m).pvalue


@pytest.mark.parametrize("window,init", [(1, INIT_RANDOM), (3, INIT_RANDOM), (4, INIT_RANDOM),
                                         (3, INIT_COPY_LEFT), (4, INIT_COPY_ABOVE),
                                         (3, INIT_RESAMPLE_LEFT), (2, INIT_RESAMPLE_ABOVE)])
def test_joint_distribution_is_exact_by_enumeration(window, init):
    """Theorem 1 for whole sequences: over many seeds the generated 4-token sequences follow
    prod_i p(x_i | x_<i), whatever the window and the initialisation."""
    vocab, n_gen, n_runs = 4, 4, 12000
    table = TableModel(vocab, order=2, seed=11)
    prompt = [1, 3]
    joint = _exact_joint(table, prompt, n_gen, 1.0, 3)
    counts = {}
    max_steps = 0
    for seed in range(n_runs):
        scfg = SampleCfg(temperature=1.0, top_k=3, seed=seed, window=window, init=init,
                         grid_stride=2, n_generate=n_gen)
        toks, steps, accepted = sjd_generate(prompt, table, scfg, vocab)
        assert len(toks) == n_gen and sum(accepted) == n_gen and steps <= n_gen
        if window == 1:
            assert steps == n_gen
        max_steps = max(max_steps, steps)
        counts[tuple(toks)] = counts.get(tuple(toks), 0) + 1
    assert _chi_square_joint(counts, joint, n_runs) > 1e-4
    assert max_steps <= n_gen


def test_ordinary_sampling_is_exact_and_takes_one_pass_per_token():
    vocab, n_gen, n_runs = 4, 3, 8000
    table = TableModel(vocab, order=2, seed=12)
    prompt = [0, 2]
    joint = _exact_joint(table, prompt, n_gen, 0.8, 4)
    counts = {}
    for seed in range(n_runs):
        scfg = SampleCfg(temperature=0.8, top_k=4, seed=seed, n_generate=n_gen)
        toks, passes = ar_generate(prompt, table, scfg, vocab)
        assert passes == n_gen
        counts[tuple(toks)] = counts.get(tuple(toks), 0) + 1
    assert _chi_square_joint(counts, joint, n_runs) > 1e-4


@pytest.mark.parametrize("init", [INIT_RANDOM, INIT_COPY_ABOVE, INIT_COPY_LEFT])
@pytest.mark.parametrize("how", ["top1", "cold"])
def test_top1_sjd_equals_greedy_jacobi_equals_greedy_ar(init, how):
    """With no randomness SJD's criterion degenerates into Jacobi's deterministic one:
    same tokens as greedy decoding for every seed, never more passes than tokens."""
    cfg, model = _tiny_model(seed=1)
    prompt = [5, 9, 2, 77, 31]
    n_gen, window = 24, 6
    greedy = greedy_ar_generate(prompt, CachedModel(model, 64), n_gen)
    for seed in range(4):
        scfg = SampleCfg(temperature=1.0 if how == "top1" else 1e-4, top_k=1 if how == "top1" else cfg.vocab,
                         seed=seed, window=window, init=init, grid_stride=4, n_generate=n_gen)
        toks, steps, accepted = sjd_generate(prompt, CachedModel(model, 64), scfg, cfg.vocab)
        assert toks == greedy
        assert steps <= n_gen and sum(accepted) == n_gen
        if init == INIT_RANDOM and how == "top1":
            jtoks, jpasses = jacobi_generate(prompt, CachedModel(model, 64), n_gen, window, cfg.vocab, seed=seed)
            assert jtoks == greedy
            assert jpasses == steps


def test_cached_and_recomputed_models_give_the_same_stream():
    cfg, model = _tiny_model(seed=2)
    prompt = [1, 2, 3]
    scfg = SampleCfg(temperature=1.0, top_k=20, seed=5, window=5, n_generate=17)
    a = sjd_generate(prompt, CachedModel(model, 64), scfg, cfg.vocab)
    b = sjd_generate(prompt, RecomputeModel(model), scfg, cfg.vocab)
    assert a == b
    assert a[1] <= 17


def test_window_bookkeeping_random_init():
    vocab = 16
    table = TableModel(vocab, order=1, seed=3)
    scfg = SampleCfg(top_k=vocab, seed=9, window=4, n_generate=10)
    st = sjd_begin([7, 7, 7], scfg, vocab, seq=2)
    assert st.n == 3 and len(st.drafts) == 4
    assert [q.kind for q in st.qdescs] == [Q_UNIFORM] * 4
    assert st.drafts == [philox.init_token(9, 3 + k, philox.STEP_INITIAL_WINDOW, 2, vocab) for k in range(4)]
    n_before = st.n
    rec = sjd_step(st, table, scfg, vocab)
    m = len(rec.committed)
    assert 1 <= m <= 4 and st.n == n_before + m and st.step == 1
    assert rec.n_accepted in (m, m - 1)
    kept = 4 - m if rec.n_accepted < 4 else 0
    assert rec.kinds[:kept] == [Q_ROW] * kept
    assert rec.kinds[kept:] == [Q_UNIFORM] * (len(rec.kinds) - kept)
    # fresh slots use the step index of the step that created them
    for k in range(kept, len(rec.drafts)):
        assert rec.drafts[k] == philox.init_token(9, st.n + k, 0, 2, vocab)
    # run to the end: window shrinks, total is exact
    while st.n < 13:
        sjd_step(st, table, scfg, vocab)
        assert len(st.drafts) == min(4, 13 - st.n)
    assert st.n == 13
    assert sjd_step(st, table, scfg, vocab).committed == []


def test_copy_above_initialisation():
    vocab = 32
    table = TableModel(vocab, order=1, seed=4)
    scfg = SampleCfg(top_k=vocab, seed=1, window=6, init=INIT_COPY_ABOVE, grid_stride=4, n_generate=20)
    prompt = [3, 1, 4]
    st = sjd_begin(prompt, scfg, vocab)
    # positions 3..6 have no image token above them (3 - 4 < P): random, uniform law;
    # positions 7, 8 copy the drafts at positions 3, 4 of the same window: point-mass law
    assert [q.kind for q in st.qdescs] == [Q_UNIFORM] * 4 + [Q_ONEHOT] * 2
    assert st.drafts[4] == st.drafts[0] and st.drafts[5] == st.drafts[1]
    while st.n < 23:
        rec = sjd_step(st, table, scfg, vocab)
        kept = len([k for k in rec.kinds if k == Q_ROW])
        for k in range(kept, len(st.drafts)):
            src = st.n + k - 4
            assert src >= 3
            expect = st.committed[src] if src < st.n else st.drafts[src - st.n]
            assert st.drafts[k] == expect and st.qdescs[k].kind == Q_ONEHOT


def test_copy_left_initialisation():
    vocab = 32
    scfg = SampleCfg(top_k=vocab, seed=1, window=5, init=INIT_COPY_LEFT, n_generate=12)
    st = sjd_begin([9, 8], scfg, vocab)
    # first slot has no generated left neighbour (2 - 1 < P): random; the rest repeat it
    assert st.qdescs[0].kind == Q_UNIFORM and all(q.kind == Q_ONEHOT for q in st.qdescs[1:])
    assert len(set(st.drafts)) == 1


def test_step_bound_on_transformer_with_sampling():
    cfg, model = _tiny_model(seed=3)
    prompt = [4, 4, 8]
    for seed in range(3):
        scfg = SampleCfg(temperature=1.0, top_k=10, seed=seed, window=8, n_generate=40)
        toks, steps, accepted = sjd_generate(prompt, CachedModel(model, 64), scfg, cfg.vocab)
        assert len(toks) == 40 and sum(accepted) == 40 and steps <= 40
        assert all(1 <= a <= 8 for a in accepted)


# ---------------------------------------------------------------------------------------------
# baseline schedules on the same state machine (Sec. 3.2; the no-refinement ablation of the appendix)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("window,init", [(1, INIT_RANDOM), (5, INIT_RANDOM), (8, INIT_COPY_LEFT)])
def test_jacobi_with_sampling_converges_to_ordinary_sampling_with_the_same_uniforms(window, init):
    """With one uniform per position, the Jacobi iteration is a fixed-point iteration of a triangular
    system: whatever the window and the initial guesses, it ends at the image that one-token-at-a-time
    sampling draws from the same uniforms, in at most as many passes as tokens."""
    cfg, model = _tiny_model(seed=3)
    prompt = [7, 1, 50, 12]
    n_gen = 20
    for seed in range(5):
        scfg = SampleCfg(temperature=1.0, top_k=8, seed=seed, window=window, init=init, grid_stride=4,
                         n_generate=n_gen, schedule=SCHEDULE_JACOBI)
        toks, steps, accepted = sjd_generate(prompt, CachedModel(model, 64), scfg, cfg.vocab)
        plain, _ = ar_generate(prompt, CachedModel(model, 64), scfg, cfg.vocab, fixed_step=0)
        assert toks == plain
        assert steps <= n_gen and sum(accepted) == n_gen
        if window == 1:
            assert steps == n_gen


def test_jacobi_schedule_with_top1_is_greedy_jacobi_decoding():
    cfg, model = _tiny_model(seed=1)
    prompt = [5, 9, 2, 77, 31]
    n_gen, window = 24, 6
    greedy = greedy_ar_generate(prompt, CachedModel(model, 64), n_gen)
    for seed in range(3):
        scfg = SampleCfg(temperature=1.0, top_k=1, seed=seed, window=window, n_generate=n_gen, schedule=SCHEDULE_JACOBI)
        toks, steps, _ = sjd_generate(prompt, CachedModel(model, 64), scfg, cfg.vocab)
        jtoks, jpasses = jacobi_generate(prompt, CachedModel(model, 64), n_gen, window, cfg.vocab, seed=seed)
        assert toks == greedy == jtoks and steps == jpasses


def test_without_refinement_the_law_is_still_exact_but_nothing_is_kept():
    """Eqs. 1-2 alone (slots after a rejection re-initialised instead of re-drawn by Eq. 3): the images
    still follow the model's law, and every slot of the window after a rejection is a fresh one."""
    vocab, n_gen, n_runs = 4, 4, 12000
    table = TableModel(vocab, order=2, seed=11)
    prompt = [1, 3]
    joint = _exact_joint(table, prompt, n_gen, 1.0, 3)
    counts = {}
    for seed in range(n_runs):
        scfg = SampleCfg(temperature=1.0, top_k=3, seed=seed, window=3, n_generate=n_gen, schedule=SCHEDULE_NO_REFINE)
        toks, steps, accepted = sjd_generate(prompt, table, scfg, vocab)
        assert steps <= n_gen and sum(accepted) == n_gen
        counts[tuple(toks)] = counts.get(tuple(toks), 0) + 1
    assert _chi_square_joint(counts, joint, n_runs) > 1e-4
    scfg = SampleCfg(temperature=1.0, top_k=3, seed=5, window=3, n_generate=12, schedule=SCHEDULE_NO_REFINE)
    st = sjd_begin(prompt, scfg, vocab)
    for _ in range(6):
        if not st.drafts:
            break
        rec = sjd_step(st, table, scfg, vocab)
        assert all(k == Q_UNIFORM for k in rec.kinds)
        assert rec.verify.redraft == []


def test_resampled_initialisation_draws_from_the_neighbours_prediction():
    """Sec. 4.2 (c), (d) on a hand-built case: a model whose rows are (almost) point masses makes the
    draw from "the distribution predicted at the neighbour" visible as the neighbour row's arg-max, and the
    slot carries that row as its law; without a row (first window) the slot is a uniform random token."""
    vocab = 6

    class Peaked:
        def prefill(self, prompt):
            pass

        def step_logits(self, committed, drafts_in):
            seq = list(committed) + list(drafts_in)
            n = len(committed)
            out = np.full((len(drafts_in) + 1, vocab), -30.0)
            for k in range(len(drafts_in) + 1):
                out[k, (n + k) % vocab] = 5.0      # the row that predicts position n + k peaks at (n + k) % vocab
            return out

    for init, stride in ((INIT_RESAMPLE_LEFT, 3), (INIT_RESAMPLE_ABOVE, 3)):
        scfg = SampleCfg(temperature=1.0, top_k=vocab, seed=3, window=3, init=init, grid_stride=stride, n_generate=12)
        st = sjd_begin([0, 1], scfg, vocab)
        assert [q.kind for q in st.qdescs] == [Q_UNIFORM] * 3          # nothing predicted yet
        rec = sjd_step(st, Peaked(), scfg, vocab)
        n0, n1 = 2, st.n
        kept = len(rec.verify.redraft)
        fresh_positions = [n1 + s for s in range(kept, len(st.drafts))]
        assert fresh_positions, "the first step fixes at least one token, so at least one slot is new"
        for t in fresh_positions:
            tok, qd = st.drafts[t - n1], st.qdescs[t - n1]
            src = min(t - 1, n0 + 2) if init == INIT_RESAMPLE_LEFT else t - stride
            if src >= 2 and src in st.rows:
                assert qd.kind == Q_ROW and tok == src % vocab          # the neighbour's own prediction
                assert np.array_equal(qd.row, st.rows[src])
            else:
                assert qd.kind == Q_UNIFORM
