"""Llama-style decoder forward pass in fp64 (test infrastructure; see
oracle/__init__.py).

The paper treats the model as a black box p_theta(x | x_{1:i}) evaluated for
all window positions in one forward pass under a causal mask (Sec. 3.1,
Sec. 3.2, Sec. 4.1 Step 2); its models are 7B Llama/Chameleon-style decoders
(Sec. 5.1).  The architecture constants it never states are fixed as follows:

  x      = tok_emb[token]
  per layer:
    h    = rmsnorm(x; attn_norm)            h_i = x_i * g_i / sqrt(mean(x^2) + eps)
    q,k,v= h Wq^T, h Wk^T, h Wv^T           (no bias; W stored [out][in])
    [QK-norm variant, the Chameleon family the paper's models derive from (Sec. 5.1): when the layer
         has gains q_norm / k_norm (length hd), every head of q and of k is normalised over its hd
         dimensions before the rotary step, q_h = rmsnorm(q_h; q_norm), k_h = rmsnorm(k_h; k_norm).
         Reading: the RMS form without bias, like every other normalisation of this block.]
    RoPE on q and k, half-split pairing: dims i and i + hd/2 rotate together
         by angle pos * theta^(-2i/hd), pos = absolute index from 0
    a    = causal softmax(q k^T / sqrt(hd)) v;  kv head j serves the H/KVh
         consecutive query heads j*(H/KVh) ... (j+1)*(H/KVh) - 1   (GQA)
    x   += a Wo^T
    h    = rmsnorm(x; ffn_norm)
    x   += (silu(h Wg^T) * (h Wu^T)) Wd^T   (SwiGLU)
  logits = rmsnorm(x; final_norm) W_out^T   (lm_head untied from tok_emb)

Weights are taken exactly as given (bf16-rounded values are exact inputs) and
every intermediate stays fp64; nothing is blocked, fused or reordered.

Stored tensors.  The paper never states a precision.  The workloads fix a
storage dtype (fp32 or bf16) for the two tensors that persist across
iterations: the logits handed to the verification (rounded by
round_to_storage before use) and the KV cache.  A KVCache created with
storage 'f32' / 'bf16' therefore rounds keys (after RoPE) and values to that
dtype as they are written, exactly like the stored logits; storage 'f64'
(default) is the plain definition and makes the cached forward identical to
the full causal forward.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class ModelCfg:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_hidden: int
    vocab: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5


def _f64(a):
    """Any array-like (numpy, or a torch tensor of any float dtype) -> fp64 numpy."""
    if isinstance(a, np.ndarray):
        return a.astype(np.float64, copy=False)
    if hasattr(a, "detach"):  # torch tensor, without importing torch at module level
        import torch
        return a.detach().to("cpu").to(torch.float64).numpy()
    return np.asarray(a, dtype=np.float64)


def rmsnorm(x, gain, eps):
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * _f64(gain)


def rope(x, positions, theta):
    """x: [T][heads][hd]; rotate pairs (i, i + hd/2) by positions[t] * theta^(-2i/hd)."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = np.asarray(theta, dtype=np.float64) ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]   # [T][half]
    cos = np.cos(ang)[:, None, :]
    sin = np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def softmax_rows(s):
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


class KVCache:
    """Keys (after RoPE) and values of the positions already run, per layer."""

    def __init__(self, cfg: ModelCfg, capacity: int, storage: str = "f64"):
        assert storage in ("f64", "f32", "bf16")
        self.storage = storage
        shape = (cfg.n_layers, capacity, cfg.n_kv_heads, cfg.head_dim)
        self.k = np.zeros(shape, dtype=np.float64)
        self.v = np.zeros(shape, dtype=np.float64)
        self.length = 0

    def truncate(self, length: int):
        """Roll back: rows >= length are stale and will be overwritten."""
        assert 0 <= length <= self.k.shape[1]
        self.length = length


class OracleModel:
    def __init__(self, cfg: ModelCfg, weights: dict):
        """weights: {'tok_emb','final_norm','lm_head','layers': [ {attn_norm,wq,wk,wv,wo,
        ffn_norm,w_gate,w_up,w_down} ]}; matrices stored [out_features][in_features]."""
        self.cfg = cfg
        self.w = weights
        assert cfg.n_heads % cfg.n_kv_heads == 0
        assert cfg.head_dim % 2 == 0

    def new_cache(self, capacity: int, storage: str = "f64") -> KVCache:
        return KVCache(self.cfg, capacity, storage)

    def _attention(self, q, k_all, v_all, q_pos):
        """q: [T][H][hd]; k_all, v_all: [S][KVh][hd] for positions 0..S-1;
        query t (absolute position q_pos[t]) sees keys 0 .. q_pos[t]."""
        cfg = self.cfg
        t_len = q.shape[0]
        s_len = k_all.shape[0]
        group = cfg.n_heads // cfg.n_kv_heads
        out = np.zeros((t_len, cfg.n_heads, cfg.head_dim), dtype=np.float64)
        key_pos = np.arange(s_len)
        visible = key_pos[None, :] <= np.asarray(q_pos)[:, None]          # [T][S]
        for h in range(cfg.n_heads):
            kv = h // group
            scores = q[:, h, :] @ k_all[:, kv, :].T / np.sqrt(cfg.head_dim)  # [T][S]
            scores = np.where(visible, scores, -np.inf)
            out[:, h, :] = softmax_rows(scores) @ v_all[:, kv, :]
        return out

    def _layer(self, li, x, positions, cache: KVCache | None):
        cfg = self.cfg
        lw = self.w["layers"][li]
        t_len = x.shape[0]
        h = rmsnorm(x, lw["attn_norm"], cfg.rms_eps)
        q = (h @ _f64(lw["wq"]).T).reshape(t_len, cfg.n_heads, cfg.head_dim)
        k = (h @ _f64(lw["wk"]).T).reshape(t_len, cfg.n_kv_heads, cfg.head_dim)
        v = (h @ _f64(lw["wv"]).T).reshape(t_len, cfg.n_kv_heads, cfg.head_dim)
        if lw.get("q_norm") is not None:      # QK-norm variant: per head, over the head dimension
            q = rmsnorm(q, lw["q_norm"], cfg.rms_eps)
            k = rmsnorm(k, lw["k_norm"], cfg.rms_eps)
        q = rope(q, positions, cfg.rope_theta)
        k = rope(k, positions, cfg.rope_theta)
        if cache is not None:
            p0 = int(positions[0])
            assert p0 == cache.length, "window must start right after the cached prefix"
            if cache.storage != "f64":
                k = round_to_storage(k, cache.storage)
                v = round_to_storage(v, cache.storage)
            cache.k[li, p0:p0 + t_len] = k
            cache.v[li, p0:p0 + t_len] = v
            k_all = cache.k[li, :p0 + t_len]
            v_all = cache.v[li, :p0 + t_len]
        else:
            k_all, v_all = k, v
        a = self._attention(q, k_all, v_all, positions).reshape(t_len, cfg.n_heads * cfg.head_dim)
        x = x + a @ _f64(lw["wo"]).T
        h = rmsnorm(x, lw["ffn_norm"], cfg.rms_eps)
        g = h @ _f64(lw["w_gate"]).T
        u = h @ _f64(lw["w_up"]).T
        x = x + (silu(g) * u) @ _f64(lw["w_down"]).T
        return x

    def hidden(self, tokens, cache: KVCache | None = None, pos0: int = 0):
        """Final-layer residual stream for `tokens` placed at absolute positions
        pos0, pos0+1, ...  With a cache, rows [0, pos0) must already be cached
        and the new keys/values are appended (cache.length advances)."""
        tokens = np.asarray(tokens, dtype=np.int64)
        t_len = tokens.shape[0]
        positions = np.arange(pos0, pos0 + t_len)
        emb = self.w["tok_emb"]
        x = _f64(emb[tokens.tolist()]) if hasattr(emb, "detach") else _f64(emb[tokens])
        for li in range(self.cfg.n_layers):
            x = self._layer(li, x, positions, cache)
        if cache is not None:
            cache.length = pos0 + t_len
        return x

    def logits_from_hidden(self, x):
        h = rmsnorm(x, self.w["final_norm"], self.cfg.rms_eps)
        return h @ _f64(self.w["lm_head"]).T

    def forward_full(self, tokens):
        """Full-sequence causal forward: logits[t] predicts token t+1."""
        assert len(tokens) > 0
        return self.logits_from_hidden(self.hidden(tokens, cache=None, pos0=0))

    def forward_window(self, cache: KVCache, tokens, pos0: int, want_logits: bool = True):
        """Forward of `tokens` at positions pos0.. against the cached prefix [0, pos0)."""
        x = self.hidden(tokens, cache=cache, pos0=pos0)
        return self.logits_from_hidden(x) if want_logits else None


def round_to_storage(logits, dtype: str):
    """Round fp64 logits to the dtype they are stored in ('f32' or 'bf16',
    round-to-nearest-even) and return them as fp64 values."""
    x = np.asarray(logits, dtype=np.float64)
    if dtype == "f32":
        return x.astype(np.float32).astype(np.float64)
    if dtype == "bf16":
        f = np.ascontiguousarray(x.astype(np.float32))
        bits = f.view(np.uint32).astype(np.uint64)
        rounded = ((bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1)))
                   >> np.uint64(16)) << np.uint64(16)
        out = rounded.astype(np.uint32).view(np.float32).astype(np.float64)
        return np.where(np.isfinite(f), out, f.astype(np.float64))
    raise ValueError(dtype)
