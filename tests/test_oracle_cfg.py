"""Pins for classifier-free guidance in the CPU checker (Sec. 5.1: guidance weight 3.0): the mixing
formula on values where it is exact, its two degenerate weights, the storage rounding against a
library cast, and the exactness theorem for guided generation by enumeration.  No GPU."""
import itertools

import numpy as np
import torch
from scipy import stats

from oracle.sampling import guided_logits, warp
from oracle.sjd import GuidedModel, SampleCfg, TableModel, sjd_generate


def test_guided_logits_hand_values():
    # dyadic values: every intermediate is exact in any precision
    lc = np.array([1.0, -2.0, 0.5, 4.0])
    lu = np.array([0.0, -1.0, 0.5, 8.0])
    for storage in ("f64", "f32", "bf16"):
        assert np.array_equal(guided_logits(lc, lu, 3.0, storage), np.array([3.0, -4.0, 0.5, -4.0]))
        assert np.array_equal(guided_logits(lc, lu, 1.0, storage), lc)      # the conditional row
        assert np.array_equal(guided_logits(lc, lu, 0.0, storage), lu)      # the unconditional row
    # moving the conditional logit up moves the mixed logit up three times as fast
    assert guided_logits([2.0], [1.0], 3.0)[0] - guided_logits([1.5], [1.0], 3.0)[0] == 1.5


def test_guided_logits_storage_rounding_matches_library_casts():
    rng = np.random.default_rng(5)
    lc = torch.from_numpy(rng.normal(0, 3, 4000).astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    lu = torch.from_numpy(rng.normal(0, 3, 4000).astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    plain = guided_logits(lc, lu, 3.0)
    f32 = guided_logits(lc, lu, 3.0, "f32")
    bf16 = guided_logits(lc, lu, 3.0, "bf16")
    # bf16 inputs, weight 3: the exact result has at most 8 + 8 + 2 significant bits: fp32 holds it
    assert np.array_equal(f32, plain)
    assert np.array_equal(bf16, torch.from_numpy(f32.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy())
    # fp32 inputs: within half an fp32 ulp of the plain formula, twice over (two roundings)
    lc32, lu32 = rng.normal(0, 3, 4000).astype(np.float32), rng.normal(0, 3, 4000).astype(np.float32)
    got = guided_logits(lc32, lu32, 2.5, "f32")
    ref = guided_logits(lc32, lu32, 2.5)
    assert np.all(np.abs(got - ref) <= 2.0 ** -22 * np.maximum(1.0, np.abs(ref)) * 4)
    assert np.array_equal(got, got.astype(np.float32).astype(np.float64))


class _Pair:
    """Two context-dependent table models that share the image tokens but not the prompt."""

    def __init__(self, vocab, weight, prompt_c, prompt_u):
        self.c, self.u = TableModel(vocab, order=2, seed=21), TableModel(vocab, order=2, seed=22, scale=1.0)
        self.vocab, self.weight, self.pc, self.pu = vocab, weight, list(prompt_c), list(prompt_u)

    def model(self, storage="f32"):
        return GuidedModel(self.c, self.u, self.pu, self.weight, storage)

    def next_token_law(self, image, temperature, top_k):
        row = guided_logits(self.c.logits_after(self.pc + image), self.u.logits_after(self.pu + image), self.weight,
                            "f32")
        return warp(row, temperature, top_k)


def test_guidance_weight_one_and_zero_reduce_to_a_single_stream():
    vocab, n_gen = 6, 12
    for weight, which in ((1.0, "c"), (0.0, "u")):
        pair = _Pair(vocab, weight, [1, 3], [0, 5])
        for seed in range(20):
            scfg = SampleCfg(temperature=1.0, top_k=4, seed=seed, window=4, n_generate=n_gen)
            guided, steps_g, _ = sjd_generate(pair.pc, pair.model(), scfg, vocab)
            single = pair.c if which == "c" else pair.u
            prompt = pair.pc if which == "c" else pair.pu
            alone, steps_a, _ = sjd_generate(prompt, single, scfg, vocab)
            assert guided == alone and steps_g == steps_a


def test_guided_joint_distribution_is_exact_by_enumeration():
    """Theorem 1 with guidance: the images follow prod_i p(x_i | x_<i) where p is the top-k softmax of
    the mixed row, although drafts were drawn from earlier mixed rows."""
    vocab, n_gen, n_runs = 4, 3, 12000
    pair = _Pair(vocab, 3.0, [1, 3], [2, 0])
    joint = {}
    for seq in itertools.product(range(vocab), repeat=n_gen):
        pr, image = 1.0, []
        for t in seq:
            pr *= pair.next_token_law(image, 1.0, 3)[t]
            image.append(t)
        joint[seq] = pr
    counts = {}
    for seed in range(n_runs):
        scfg = SampleCfg(temperature=1.0, top_k=3, seed=seed, window=3, n_generate=n_gen)
        toks, steps, accepted = sjd_generate(pair.pc, pair.model(), scfg, vocab)
        assert steps <= n_gen and sum(accepted) == n_gen
        counts[tuple(toks)] = counts.get(tuple(toks), 0) + 1
    keys = sorted(joint)
    exp = np.array([joint[k] * n_runs for k in keys])
    obs = np.array([counts.get(k, 0) for k in keys], dtype=float)
    assert all(joint[k] > 0 for k in counts), "sampled a zero-probability image"
    big = exp >= 5
    obs_m, exp_m = np.append(obs[big], obs[~big].sum()), np.append(exp[big], exp[~big].sum())
    if exp_m[-1] == 0:
        obs_m, exp_m = obs_m[:-1], exp_m[:-1]
    assert stats.chisquare(obs_m, exp_m).pvalue > 1e-4
    # guidance really changes the law: the conditional stream alone is a different distribution
    alone = warp(pair.c.logits_after(pair.pc), 1.0, 3)
    assert np.abs(alone - pair.next_token_law([], 1.0, 3)).max() > 0.05
