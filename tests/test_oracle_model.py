"""Pins for the CPU checker's decoder forward pass: library routines of torch
(fp64, CPU), textbook properties of rotary embeddings and grouped-query
attention, and cache-vs-recompute equivalence.  No GPU."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle.model import ModelCfg, OracleModel, rmsnorm, rope, round_to_storage, silu, softmax_rows


def _weights(cfg: ModelCfg, seed=0, std=0.08):
    rng = np.random.default_rng(seed)
    d, hd = cfg.d_model, cfg.head_dim

    def mat(o, i):
        return rng.normal(0, std, size=(o, i))

    layers = []
    for _ in range(cfg.n_layers):
        layers.append(dict(attn_norm=1 + 0.1 * rng.normal(size=d), wq=mat(cfg.n_heads * hd, d),
                           wk=mat(cfg.n_kv_heads * hd, d), wv=mat(cfg.n_kv_heads * hd, d),
                           wo=mat(d, cfg.n_heads * hd), ffn_norm=1 + 0.1 * rng.normal(size=d),
                           w_gate=mat(cfg.ffn_hidden, d), w_up=mat(cfg.ffn_hidden, d),
                           w_down=mat(d, cfg.ffn_hidden)))
    return dict(tok_emb=mat(cfg.vocab, d), final_norm=1 + 0.1 * rng.normal(size=d),
                lm_head=mat(cfg.vocab, d), layers=layers)


CFG = ModelCfg(n_layers=2, d_model=48, n_heads=6, n_kv_heads=2, head_dim=8, ffn_hidden=77, vocab=53)


def test_elementwise_ops_against_torch():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(5, 48))
    g = rng.normal(size=48)
    ref = F.rms_norm(torch.from_numpy(x), (48,), torch.from_numpy(g), eps=1e-5).numpy()
    np.testing.assert_allclose(rmsnorm(x, g, 1e-5), ref, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(silu(x), F.silu(torch.from_numpy(x)).numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(softmax_rows(x), torch.softmax(torch.from_numpy(x), -1).numpy(), rtol=1e-12)


def test_rope_properties():
    rng = np.random.default_rng(1)
    # two dims, theta^0 = 1: plain rotation by `pos` radians
    out = rope(np.array([[[1.0, 0.0]]]), [0.7], 10000.0)
    np.testing.assert_allclose(out[0, 0], [np.cos(0.7), np.sin(0.7)], atol=1e-15)
    # position 0 is the identity; rotations preserve norms
    x = rng.normal(size=(4, 3, 16))
    np.testing.assert_allclose(rope(x, [0, 0, 0, 0], 10000.0), x, atol=0)
    y = rope(x, [3, 17, 100, 4095], 10000.0)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    # relative-shift property: <rope(q, m), rope(k, n)> depends on m - n only
    q = rng.normal(size=(1, 1, 16))
    k = rng.normal(size=(1, 1, 16))
    dots = [float(np.sum(rope(q, [m], 1e4) * rope(k, [m - 5], 1e4))) for m in (5, 40, 1000)]
    np.testing.assert_allclose(dots, dots[0], rtol=1e-10)
    # pairing is (i, i + hd/2) with frequency theta^(-2i/hd): check one pair by hand
    hd, i, pos, theta = 16, 3, 11.0, 10000.0
    e = np.zeros((1, 1, hd))
    e[0, 0, i] = 1.0
    ang = pos * theta ** (-2 * i / hd)
    r = rope(e, [pos], theta)[0, 0]
    assert r[i] == pytest.approx(np.cos(ang)) and r[i + hd // 2] == pytest.approx(np.sin(ang))
    assert np.count_nonzero(np.abs(r) > 1e-15) == 2


def _torch_forward(cfg: ModelCfg, w, tokens, kv_cast=None):
    """Independent fp64 forward built from torch library ops (sdpa, rms_norm, silu, complex
    multiplication for the rotary step).  kv_cast: torch dtype keys/values are cast through."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    tok = torch.as_tensor(tokens)
    x = t(w["tok_emb"])[tok]
    T = x.shape[0]
    hd, half = cfg.head_dim, cfg.head_dim // 2
    freqs = torch.outer(torch.arange(T, dtype=torch.float64),
                        cfg.rope_theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd))
    cis = torch.polar(torch.ones_like(freqs), freqs)   # [T][half]

    def rot(z):  # [T][h][hd], half-split pairing
        zc = torch.complex(z[..., :half], z[..., half:]) * cis[:, None, :]
        return torch.cat([zc.real, zc.imag], dim=-1)

    for lw in w["layers"]:
        h = F.rms_norm(x, (cfg.d_model,), t(lw["attn_norm"]), eps=cfg.rms_eps)
        q = (h @ t(lw["wq"]).T).view(T, cfg.n_heads, hd)
        k = (h @ t(lw["wk"]).T).view(T, cfg.n_kv_heads, hd)
        if lw.get("q_norm") is not None:
            q = F.rms_norm(q, (hd,), t(lw["q_norm"]), eps=cfg.rms_eps)
            k = F.rms_norm(k, (hd,), t(lw["k_norm"]), eps=cfg.rms_eps)
        q, k = rot(q), rot(k)
        v = (h @ t(lw["wv"]).T).view(T, cfg.n_kv_heads, hd)
        if kv_cast is not None:
            k, v = k.to(kv_cast).to(torch.float64), v.to(kv_cast).to(torch.float64)
        rep = cfg.n_heads // cfg.n_kv_heads
        k = k.repeat_interleave(rep, dim=1)
        v = v.repeat_interleave(rep, dim=1)
        a = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                           v.transpose(0, 1)[None], is_causal=True)[0]
        x = x + a.transpose(0, 1).reshape(T, -1) @ t(lw["wo"]).T
        h = F.rms_norm(x, (cfg.d_model,), t(lw["ffn_norm"]), eps=cfg.rms_eps)
        x = x + (F.silu(h @ t(lw["w_gate"]).T) * (h @ t(lw["w_up"]).T)) @ t(lw["w_down"]).T
    x = F.rms_norm(x, (cfg.d_model,), t(w["final_norm"]), eps=cfg.rms_eps)
    return (x @ t(w["lm_head"]).T).numpy()


def test_full_forward_against_torch_library_ops():
    w = _weights(CFG)
    tokens = np.random.default_rng(2).integers(0, CFG.vocab, size=19)
    got = OracleModel(CFG, w).forward_full(tokens)
    np.testing.assert_allclose(got, _torch_forward(CFG, w, tokens), rtol=1e-10, atol=1e-12)


def test_window_forward_with_cache_equals_full_forward():
    w = _weights(CFG, seed=3)
    m = OracleModel(CFG, w)
    tokens = np.random.default_rng(4).integers(0, CFG.vocab, size=23)
    full = m.forward_full(tokens)
    cache = m.new_cache(64)
    m.forward_window(cache, tokens[:9], 0, want_logits=False)
    win = m.forward_window(cache, tokens[9:17], 9)
    np.testing.assert_allclose(win, full[9:17], rtol=1e-10, atol=1e-12)
    # roll back 5 rows, feed different tokens, then the original ones again
    cache.truncate(12)
    other = (tokens[12:20] + 1) % CFG.vocab
    m.forward_window(cache, other, 12)
    cache.truncate(12)
    again = m.forward_window(cache, tokens[12:23], 12)
    np.testing.assert_allclose(again, full[12:23], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("storage,cast", [("bf16", torch.bfloat16), ("f32", torch.float32)])
def test_cache_storage_rounding_equals_casting_keys_and_values(storage, cast):
    """A cache of storage dtype s holds keys/values rounded to s: same logits as a library forward
    whose keys and values are cast through that dtype; and it does change the result for bf16."""
    w = _weights(CFG, seed=11)
    m = OracleModel(CFG, w)
    tokens = np.random.default_rng(12).integers(0, CFG.vocab, size=21)
    cache = m.new_cache(32, storage)
    m.forward_window(cache, tokens[:8], 0, want_logits=False)
    got = np.concatenate([m.forward_window(cache, tokens[8:15], 8), m.forward_window(cache, tokens[15:21], 15)])
    ref = _torch_forward(CFG, w, tokens, kv_cast=cast)[8:21]
    np.testing.assert_allclose(got, ref, rtol=1e-9, atol=1e-11)
    plain = m.forward_full(tokens)[8:21]
    if storage == "bf16":
        assert 1e-5 < np.abs(got - plain).max() < 0.05
    else:
        assert np.abs(got - plain).max() < 1e-6


def test_causality():
    w = _weights(CFG, seed=5)
    m = OracleModel(CFG, w)
    tokens = np.random.default_rng(6).integers(0, CFG.vocab, size=12)
    a = m.forward_full(tokens)
    changed = tokens.copy()
    changed[8] = (changed[8] + 7) % CFG.vocab
    b = m.forward_full(changed)
    np.testing.assert_allclose(a[:8], b[:8], rtol=0, atol=0)
    assert np.abs(a[8:] - b[8:]).max() > 1e-6


def test_gqa_equals_mha_with_replicated_kv_heads():
    w = _weights(CFG, seed=7)
    rep = CFG.n_heads // CFG.n_kv_heads
    mha_cfg = ModelCfg(**{**CFG.__dict__, "n_kv_heads": CFG.n_heads})
    w2 = dict(w)
    w2["layers"] = []
    for lw in w["layers"]:
        lw2 = dict(lw)
        for name in ("wk", "wv"):
            m = lw[name].reshape(CFG.n_kv_heads, CFG.head_dim, CFG.d_model)
            lw2[name] = np.repeat(m, rep, axis=0).reshape(-1, CFG.d_model)
        w2["layers"].append(lw2)
    tokens = np.random.default_rng(8).integers(0, CFG.vocab, size=10)
    np.testing.assert_allclose(OracleModel(CFG, w).forward_full(tokens),
                               OracleModel(mha_cfg, w2).forward_full(tokens), rtol=1e-11, atol=1e-13)


def test_round_to_storage():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -9, -3.14159, 1e-3, 65504.0, 0.0])
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(round_to_storage(x, "bf16"), ref)
    rng = np.random.default_rng(9)
    y = rng.normal(0, 5, size=5000)
    ref = torch.tensor(y, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(round_to_storage(y, "bf16"), ref)
    np.testing.assert_array_equal(round_to_storage(y, "f32"), y.astype(np.float32).astype(np.float64))


def test_torch_tensor_weights_are_accepted():
    w = _weights(CFG, seed=10)
    bf = lambda a: torch.tensor(a).to(torch.bfloat16)
    tw = dict(tok_emb=bf(w["tok_emb"]), final_norm=bf(w["final_norm"]), lm_head=bf(w["lm_head"]),
              layers=[{k: bf(v) for k, v in lw.items()} for lw in w["layers"]])
    f64 = lambda a: a.to(torch.float64).numpy()
    nw = dict(tok_emb=f64(tw["tok_emb"]), final_norm=f64(tw["final_norm"]), lm_head=f64(tw["lm_head"]),
              layers=[{k: f64(v) for k, v in lw.items()} for lw in tw["layers"]])
    tokens = [3, 1, 4, 1, 5]
    np.testing.assert_allclose(OracleModel(CFG, tw).forward_full(tokens),
                               OracleModel(CFG, nw).forward_full(tokens), rtol=1e-12)


def _with_qk_norm(w, cfg, seed=5):
    rng = np.random.default_rng(seed)
    out = dict(w, layers=[dict(lw, q_norm=1 + 0.2 * rng.normal(size=cfg.head_dim),
                               k_norm=1 + 0.2 * rng.normal(size=cfg.head_dim)) for lw in w["layers"]])
    return out


def test_qk_norm_variant_against_torch_and_its_scale_invariance():
    """The QK-norm variant: (1) equals an independent forward built from torch's rms_norm applied per head
    before the rotary step; (2) differs from the plain model; (3) its logits do not change when W_q or W_k
    is scaled by a positive constant (each head is normalised; eps is made negligible for this check);
    (4) with a cache it still equals the full causal forward."""
    cfg = ModelCfg(n_layers=2, d_model=48, n_heads=6, n_kv_heads=2, head_dim=8, ffn_hidden=77, vocab=53, rms_eps=1e-12)
    w = _with_qk_norm(_weights(cfg, seed=3), cfg)
    tokens = [3, 17, 5, 44, 9, 9, 30]
    model = OracleModel(cfg, w)
    got = model.forward_full(tokens)
    np.testing.assert_allclose(got, _torch_forward(cfg, w, tokens), rtol=1e-9, atol=1e-11)
    plain = OracleModel(cfg, _weights(cfg, seed=3)).forward_full(tokens)
    assert np.abs(got - plain).max() > 1e-2
    scaled = dict(w, layers=[dict(lw, wq=3.0 * lw["wq"], wk=0.25 * lw["wk"]) for lw in w["layers"]])
    np.testing.assert_allclose(OracleModel(cfg, scaled).forward_full(tokens), got, rtol=1e-7, atol=1e-9)
    cache = model.new_cache(16)
    model.forward_window(cache, tokens[:4], 0, want_logits=False)
    np.testing.assert_allclose(model.forward_window(cache, tokens[4:], 4), got[4:], rtol=1e-10, atol=1e-12)
