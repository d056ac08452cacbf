"""Seeded synthetic inputs shaped like the paper's workloads.

Inputs only: shapes, value distributions and seeds.  Nothing here computes any
part of the decoding method; both the CUDA library and the CPU checker consume
what this module returns.

Workloads (Sec. 5.1 and the resolution study of the paper: 7B decoders, top-K
2000, roughly 1000 / 2300 / 4100 image tokens per image, windows of 16-64):

  tiny      2 layers, d=256, 4 heads x 64, SwiGLU 683, vocab 1024, fp32;
            prompt 16, 16x16 grid, W=16, top-k 64
  verify    isolated verification: B x 32 rows over a 16384 vocabulary, bf16
            logits ~ N(0, 3^2) with 5 % of entries raised by 6; previous-iteration
            logits = those plus N(0, 1) drift; drafts drawn from the previous rows
  7b        32 layers, d=4096, 32 heads x 128, SwiGLU 11008, vocab 65536, bf16;
            prompt 64, 48 rows of 48 tokens + 1 row-end token, W=32, top-k 2000
  8b-gqa    as 7b with 8 kv heads, SwiGLU 14336, vocab 184320; prompt 128,
            64x64 grid, W=64, top-k 2048
"""
from __future__ import annotations

from dataclasses import asdict, dataclass, replace

import numpy as np
import torch


@dataclass
class Workload:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_hidden: int
    vocab: int
    dtype: str            # 'f32' or 'bf16' (weights, activations, KV cache, stored logits)
    prompt_len: int
    n_generate: int
    grid_stride: int
    window: int
    top_k: int
    temperature: float = 1.0
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5
    weight_seed: int = 0
    prompt_seed: int = 1
    philox_seed: int = 2024

    def as_dict(self):
        return asdict(self)

    def with_(self, **kw):
        return replace(self, **kw)

    def n_params(self) -> int:
        d, hd = self.d_model, self.head_dim
        per_layer = (self.n_heads * hd * d + 2 * self.n_kv_heads * hd * d + d * self.n_heads * hd
                     + 3 * self.ffn_hidden * d + 2 * d)
        return self.n_layers * per_layer + 2 * self.vocab * d + d

    def step_weight_bytes(self) -> int:
        """Bytes of weight matrices one forward pass must stream (embedding table excluded:
        only a few of its rows are gathered)."""
        esz = 4 if self.dtype == "f32" else 2
        return (self.n_params() - self.vocab * self.d_model) * esz


WORKLOADS = {
    "tiny": Workload("tiny", 2, 256, 4, 4, 64, 683, 1024, "f32", 16, 256, 16, 16, 64),
    "7b": Workload("7b", 32, 4096, 32, 32, 128, 11008, 65536, "bf16", 64, 2352, 49, 32, 2000),
    "8b-gqa": Workload("8b-gqa", 32, 4096, 32, 8, 128, 14336, 184320, "bf16", 128, 4096, 64, 64, 2048),
    # reduced-depth variants of the large shapes for parity tests the CPU checker can afford
    "7b-2l": Workload("7b-2l", 2, 4096, 32, 32, 128, 11008, 65536, "bf16", 64, 2352, 49, 32, 2000),
    "8b-gqa-2l": Workload("8b-gqa-2l", 2, 4096, 32, 8, 128, 14336, 184320, "bf16", 128, 4096, 64, 64, 2048),
    # small bf16 model with GQA and ragged sizes, for fast end-to-end parity
    "small-bf16": Workload("small-bf16", 2, 512, 8, 2, 64, 1408, 4096, "bf16", 24, 192, 16, 16, 200),
}


def torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _randn(shape, std, gen, dtype):
    return (torch.randn(shape, generator=gen, dtype=torch.float32, device=gen.device) * std).to(dtype)


def make_weights(wl: Workload, gain_jitter: float = 0.0, std: float = 0.02, device="cpu", qk_norm: bool = False):
    """Random-init weights N(0, std^2) rounded to the workload dtype.  Matrices are
    [out_features][in_features].  Norm gains are 1 (+ optional jitter so tests exercise the
    gain path).  Generated on `device` with that device's generator: CPU tensors are what
    parity tests feed to both sides; the benchmark generates its 7B weights on the GPU.
    qk_norm: add per-layer gains q_norm / k_norm [head_dim] (1 + 0.2 N(0, 1)) for the QK-norm variant of
    the Chameleon family; they are drawn after everything else, so the other weights do not change."""
    dt = torch_dtype(wl.dtype)
    gen = torch.Generator(device=device).manual_seed(wl.weight_seed)
    d, hd = wl.d_model, wl.head_dim

    def gain():
        g = torch.ones(d, dtype=torch.float32, device=gen.device)
        if gain_jitter:
            g = g + gain_jitter * torch.randn(d, generator=gen, device=gen.device)
        return g.to(dt)

    w = {"tok_emb": _randn((wl.vocab, d), std, gen, dt), "layers": []}
    for _ in range(wl.n_layers):
        w["layers"].append({
            "attn_norm": gain(),
            "wq": _randn((wl.n_heads * hd, d), std, gen, dt),
            "wk": _randn((wl.n_kv_heads * hd, d), std, gen, dt),
            "wv": _randn((wl.n_kv_heads * hd, d), std, gen, dt),
            "wo": _randn((d, wl.n_heads * hd), std, gen, dt),
            "ffn_norm": gain(),
            "w_gate": _randn((wl.ffn_hidden, d), std, gen, dt),
            "w_up": _randn((wl.ffn_hidden, d), std, gen, dt),
            "w_down": _randn((d, wl.ffn_hidden), std, gen, dt),
        })
    w["final_norm"] = gain()
    w["lm_head"] = _randn((wl.vocab, d), std, gen, dt)
    if qk_norm:
        for lw in w["layers"]:
            for name in ("q_norm", "k_norm"):
                lw[name] = (torch.ones(hd, dtype=torch.float32, device=gen.device)
                            + 0.2 * torch.randn(hd, generator=gen, device=gen.device)).to(dt)
    return w


def make_prompt(wl: Workload, batch: int = 1):
    """[batch][prompt_len] int32 token ids, uniform over the vocabulary."""
    rng = np.random.default_rng(wl.prompt_seed)
    return rng.integers(0, wl.vocab, size=(batch, wl.prompt_len), dtype=np.int64).astype(np.int32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 array -> values representable in bf16 (round to nearest even), as fp32."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


@dataclass
class VerifyCase:
    batch: int
    window: int
    vocab: int
    dtype: str
    logits_cur: np.ndarray    # [B][W][V] fp32 values representable in dtype
    logits_prev: np.ndarray   # [B][W][V]
    draft: np.ndarray         # [B][W] int32
    q_kind: np.ndarray        # [B][W] int32 (0 row / 1 uniform / 2 one-hot)
    base_pos: np.ndarray      # [B] absolute position of window slot 0
    step: int
    temperature: float
    top_k: int
    seed: int


def make_verify_case(batch: int, window: int = 32, vocab: int = 16384, dtype: str = "bf16",
                     top_k: int = 2000, temperature: float = 1.0, seed: int | None = None,
                     mixed_kinds: bool = False, drift: float = 1.0) -> VerifyCase:
    """The isolated-verification workload.  Current logits ~ N(0, 9) with a random 5 %
    of each row raised by 6; previous-iteration logits = current + N(0, drift^2); both
    rounded to `dtype`.  Drafts are drawn from the previous rows restricted to their
    top_k largest entries by the Gumbel-max trick (a plain numpy draw, independent of
    the samplers under test).  With mixed_kinds, some slots are marked as uniformly
    initialised or copied tokens instead."""
    seed = 100 + batch if seed is None else seed
    rng = np.random.default_rng(seed)
    cur = rng.normal(0.0, 3.0, size=(batch, window, vocab)).astype(np.float32)
    cur += (6.0 * (rng.random(size=cur.shape) < 0.05)).astype(np.float32)
    prev = cur + rng.normal(0.0, drift, size=cur.shape).astype(np.float32)
    if dtype == "bf16":
        cur, prev = round_bf16(cur), round_bf16(prev)
    gumbel = -np.log(-np.log(rng.random(size=prev.shape)))
    scaled = prev.astype(np.float64) / temperature
    if top_k < vocab:
        kth = np.partition(scaled, vocab - top_k, axis=-1)[..., vocab - top_k][..., None]
        scaled = np.where(scaled >= kth, scaled, -np.inf)
    draft = np.argmax(scaled + gumbel, axis=-1).astype(np.int32)
    kind = np.zeros((batch, window), dtype=np.int32)
    if mixed_kinds:
        kind = rng.choice(np.array([0, 0, 1, 2], dtype=np.int32), size=(batch, window))
        uni = kind == 1
        draft = np.where(uni, rng.integers(0, vocab, size=draft.shape), draft).astype(np.int32)
        # a copied token is usually plausible under the current row: take its arg-max half the time
        top = np.argmax(cur, axis=-1).astype(np.int32)
        draft = np.where((kind == 2) & (rng.random(size=draft.shape) < 0.5), top, draft).astype(np.int32)
    base = rng.integers(16, 4096, size=(batch,), dtype=np.int64).astype(np.int32)
    return VerifyCase(batch, window, vocab, dtype, cur, prev, draft, kind, base,
                      step=int(rng.integers(1, 1000)), temperature=temperature, top_k=top_k, seed=seed)
