"""ctypes binding of libsjd.so: same names as include/sjd.h, argument marshalling only.

PyTorch supplies device memory and streams; every step of the decoding path runs inside the
library's CUDA kernels.  Loading fails loudly if the library has not been built
(`python -m paper_2410_01699_b200.build`); there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsjd.so")

SJD_OK = 0
SJD_ERR_BAD_ARG, SJD_ERR_CAPACITY, SJD_ERR_UNSUPPORTED = -1, -2, -3
SJD_ERR_CUDA, SJD_ERR_DEVICE_TIMEOUT, SJD_ERR_STATE = -4, -5, -6
SJD_F32, SJD_BF16 = 0, 1
SJD_INIT_RANDOM, SJD_INIT_COPY_ABOVE, SJD_INIT_COPY_LEFT, SJD_INIT_RESAMPLE_LEFT, SJD_INIT_RESAMPLE_ABOVE = 0, 1, 2, 3, 4
SJD_Q_ROW, SJD_Q_UNIFORM, SJD_Q_ONEHOT, SJD_Q_RING = 0, 1, 2, 3
SJD_SCHEDULE_SJD, SJD_SCHEDULE_JACOBI, SJD_SCHEDULE_NO_REFINE = 0, 1, 2
SJD_FLAG_NEAR_TIE_ACCEPT, SJD_FLAG_RESIDUAL_EMPTY, SJD_FLAG_NONFINITE, SJD_FLAG_DONE = 1, 4, 8, 16

DTYPES = {"f32": SJD_F32, "bf16": SJD_BF16}
TORCH_DTYPES = {SJD_F32: torch.float32, SJD_BF16: torch.bfloat16}

EXPORTS = ["sjd_workspace_bytes", "sjd_init", "sjd_prefill", "sjd_step", "sjd_get_window", "sjd_peek_logits",
           "sjd_verify_workspace_bytes", "sjd_verify", "sjd_last_device_status", "sjd_last_cuda_error",
           "sjd_destroy", "sjd_strerror", "sjd_launch_count", "sjd_trace", "sjd_trace_read", "sjd_verify_static",
           "sjd_gemm_workspace_bytes", "sjd_gemm", "sjd_attention_workspace_bytes", "sjd_attention", "sjd_get_info",
           "sjd_prefill_ragged", "sjd_get_tokens"]


class SJDError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().sjd_strerror(status).decode()
        if status == SJD_ERR_CUDA:
            msg += " [cudaError %d]" % lib().sjd_last_cuda_error()
        super().__init__("%s: %s (%d)" % (where, msg, status))


class sjd_model_cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "ffn_hidden",
                                         "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32), ("max_window", C.c_int32), ("max_ring", C.c_int32),
                ("kv_pages", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class sjd_weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, _PP) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down",
                                   "q_norm", "k_norm")]


class sjd_sample_cfg(C.Structure):
    _fields_ = [("temperature", C.c_float), ("top_k", C.c_int32), ("seed", C.c_uint64), ("window", C.c_int32),
                ("init", C.c_int32), ("grid_stride", C.c_int32), ("n_generate", C.c_int32), ("seq_base", C.c_int32),
                ("guidance", C.c_float), ("schedule", C.c_int32)]


class sjd_step_out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("n_accepted", "n_committed", "committed", "draft", "q_kind", "q_draft",
                                          "total_committed", "flags")]


class sjd_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("tensor_core_projections", "tensor_core_attention", "step_graph",
                                         "rows_per_step")]


_lib = None


def lib():
    """The loaded library; raises if it is missing or lacks a declared symbol."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libsjd.so is not built: run `python -m paper_2410_01699_b200.build` "
                           "(needs nvcc with sm_100a support); there is no fallback path")
    L = C.CDLL(LIB_PATH)
    for name in EXPORTS:
        if not hasattr(L, name):
            raise RuntimeError("libsjd.so does not export %s" % name)
    L.sjd_workspace_bytes.restype = C.c_size_t
    L.sjd_workspace_bytes.argtypes = [C.POINTER(sjd_model_cfg)]
    L.sjd_init.restype = C.c_int
    L.sjd_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(sjd_model_cfg), C.POINTER(sjd_weights), C.c_void_p,
                           C.c_size_t]
    L.sjd_prefill.restype = C.c_int
    L.sjd_prefill.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.POINTER(sjd_sample_cfg), C.c_void_p]
    L.sjd_prefill_ragged.restype = C.c_int
    L.sjd_prefill_ragged.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(C.c_int32), C.c_int,
                                     C.POINTER(sjd_sample_cfg), C.c_void_p]
    L.sjd_step.restype = C.c_int
    L.sjd_step.argtypes = [C.c_void_p, C.POINTER(sjd_step_out), C.c_void_p]
    L.sjd_get_tokens.restype = C.c_int
    L.sjd_get_tokens.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
    L.sjd_get_window.restype = C.c_int
    L.sjd_get_window.argtypes = [C.c_void_p, C.POINTER(sjd_step_out), C.c_void_p]
    L.sjd_peek_logits.restype = C.c_int
    L.sjd_peek_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.sjd_verify_workspace_bytes.restype = C.c_size_t
    L.sjd_verify_workspace_bytes.argtypes = [C.c_int, C.c_int]
    L.sjd_verify.restype = C.c_int
    L.sjd_verify.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.POINTER(sjd_sample_cfg), C.c_uint32, C.POINTER(sjd_step_out), C.c_void_p,
                             C.c_size_t, C.c_void_p]
    L.sjd_verify_static.restype = C.c_int
    L.sjd_verify_static.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.POINTER(sjd_sample_cfg), C.c_uint32, C.POINTER(sjd_step_out),
                                    C.c_void_p]
    L.sjd_gemm_workspace_bytes.restype = C.c_size_t
    L.sjd_gemm_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
    L.sjd_gemm.restype = C.c_int
    L.sjd_gemm.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                           C.c_size_t, C.c_void_p]
    L.sjd_attention_workspace_bytes.restype = C.c_size_t
    L.sjd_attention_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
    L.sjd_attention.restype = C.c_int
    L.sjd_attention.argtypes = [C.c_int] * 6 + [C.c_void_p] * 5 + [C.c_size_t, C.c_void_p]
    L.sjd_get_info.restype = C.c_int
    L.sjd_get_info.argtypes = [C.c_void_p, C.POINTER(sjd_info)]
    L.sjd_last_device_status.restype = C.c_int
    L.sjd_last_device_status.argtypes = [C.c_void_p]
    L.sjd_last_cuda_error.restype = C.c_int
    L.sjd_launch_count.restype = C.c_int64
    L.sjd_trace.restype = C.c_int
    L.sjd_trace.argtypes = [C.c_void_p, C.c_int]
    L.sjd_trace_read.restype = C.c_int
    L.sjd_trace_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.POINTER(C.c_double)]
    L.sjd_destroy.restype = None
    L.sjd_destroy.argtypes = [C.c_void_p]
    L.sjd_strerror.restype = C.c_char_p
    L.sjd_strerror.argtypes = [C.c_int]
    _lib = L
    return L


def _check(status: int, where: str):
    if status != SJD_OK:
        raise SJDError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_model_cfg(wl, max_batch: int, max_seq: int, max_window: int, max_ring: int = 0,
                   kv_pages: int = 0) -> sjd_model_cfg:
    """wl: anything with the model fields of inputs.Workload."""
    return sjd_model_cfg(wl.n_layers, wl.d_model, wl.n_heads, wl.n_kv_heads, wl.head_dim, wl.ffn_hidden, wl.vocab,
                         wl.rope_theta, wl.rms_eps, DTYPES[wl.dtype], max_batch, max_seq, max_window, max_ring, kv_pages)


def make_sample_cfg(temperature=1.0, top_k=2000, seed=0, window=16, init=SJD_INIT_RANDOM, grid_stride=0,
                    n_generate=0, seq_base=0, guidance=0.0, schedule=0) -> sjd_sample_cfg:
    return sjd_sample_cfg(float(temperature), int(top_k), int(seed), int(window), int(init), int(grid_stride),
                          int(n_generate), int(seq_base), float(guidance), int(schedule))


class StepOut:
    """Caller-owned result buffers of one step (device tensors, or pinned host tensors)."""

    def __init__(self, batch: int, window: int, device="cuda", pinned: bool = False):
        kw = dict(device="cpu", pin_memory=True) if pinned else dict(device=device)
        i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, **kw)
        self.n_accepted, self.n_committed = i32(batch), i32(batch)
        self.committed, self.draft, self.q_kind = i32(batch, window), i32(batch, window), i32(batch, window)
        self.q_draft = torch.zeros(batch, window, dtype=torch.float32, **kw)
        self.total_committed, self.flags = i32(batch), i32(batch)
        self.c = sjd_step_out(*[C.c_void_p(t.data_ptr()) for t in (
            self.n_accepted, self.n_committed, self.committed, self.draft, self.q_kind, self.q_draft,
            self.total_committed, self.flags)])

    def host(self):
        """dict of numpy copies (synchronises the current stream)."""
        torch.cuda.current_stream().synchronize()
        names = ("n_accepted", "n_committed", "committed", "draft", "q_kind", "q_draft", "total_committed", "flags")
        return {n: getattr(self, n).cpu().numpy().copy() for n in names}


def sjd_workspace_bytes(cfg: sjd_model_cfg) -> int:
    return int(lib().sjd_workspace_bytes(C.byref(cfg)))


def sjd_verify_workspace_bytes(batch: int, window: int) -> int:
    return int(lib().sjd_verify_workspace_bytes(batch, window))


def sjd_verify(logits_cur, logits_prev, draft, q_kind, base_pos, sample: sjd_sample_cfg, step: int, out: StepOut,
               ws=None):
    """Isolated verification (Eqs. 1-3).  logits_*: [B][W][V] cuda tensors (float32 or bfloat16)."""
    b, w, v = logits_cur.shape
    dt = {torch.float32: SJD_F32, torch.bfloat16: SJD_BF16}[logits_cur.dtype]
    if ws is None:
        ws = torch.empty(sjd_verify_workspace_bytes(b, w), dtype=torch.uint8, device=logits_cur.device)
    st = lib().sjd_verify(b, w, v, dt, _ptr(logits_cur), _ptr(logits_prev), _ptr(draft), _ptr(q_kind), _ptr(base_pos),
                          C.byref(sample), C.c_uint32(step), C.byref(out.c), _ptr(ws), ws.numel(), _stream())
    _check(st, "sjd_verify")
    return ws


SJD_VERIFY_STATIC_MAX_ROWS, SJD_VERIFY_STATIC_MAX_BATCH = 2048, 256


def sjd_verify_static(logits_cur, logits_prev, draft, q_kind, base_pos, sample: sjd_sample_cfg, step: int,
                      out: StepOut):
    """sjd_verify for callers that cannot allocate: no scratch argument, the library's built-in
    scratch array is used (batch * window <= SJD_VERIFY_STATIC_MAX_ROWS).  Calls on one device must
    not overlap; make the first call on a device outside any stream capture."""
    b, w, v = logits_cur.shape
    dt = {torch.float32: SJD_F32, torch.bfloat16: SJD_BF16}[logits_cur.dtype]
    st = lib().sjd_verify_static(b, w, v, dt, _ptr(logits_cur), _ptr(logits_prev), _ptr(draft), _ptr(q_kind),
                                 _ptr(base_pos), C.byref(sample), C.c_uint32(step), C.byref(out.c), _stream())
    _check(st, "sjd_verify_static")


def sjd_gemm(x, w, out=None, accumulate=False):
    """out[M][N] (+)= x[M][K] @ w[N][K]^T on the tensor-core weight-streaming kernel.
    x: float32 cuda, w: bfloat16 cuda.  Returns (out, status word tensor)."""
    m, k = x.shape
    n = w.shape[0]
    if out is None:
        out = torch.zeros(m, n, dtype=torch.float32, device=x.device)
    nbytes = int(lib().sjd_gemm_workspace_bytes(m, n, k))
    if nbytes == 0:
        raise SJDError(SJD_ERR_UNSUPPORTED, "sjd_gemm_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=x.device)
    _check(lib().sjd_gemm(m, n, k, _ptr(x), _ptr(w), _ptr(out), 1 if accumulate else 0, _ptr(ws), nbytes, _stream()),
           "sjd_gemm")
    return out, ws[:4].view(torch.int32)


def sjd_attention(q, kv_cache, in_pos, window, n_kv_heads, out=None, ws=None):
    """Window-causal attention on the tensor-core kernel.  q: float32 cuda [B*W][H][hd]; kv_cache:
    bfloat16 cuda [B][2][KVh][max_seq][hd]; in_pos: int32 cuda [B*W].  Returns (out, status word)."""
    m, h, hd = q.shape
    b, max_seq = kv_cache.shape[0], kv_cache.shape[3]
    if out is None:
        out = torch.empty_like(q)
    nbytes = int(lib().sjd_attention_workspace_bytes(b, window, h, hd))
    if nbytes == 0:
        raise SJDError(SJD_ERR_UNSUPPORTED, "sjd_attention_workspace_bytes")
    if ws is None:
        ws = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    _check(lib().sjd_attention(b, window, h, n_kv_heads, hd, max_seq, _ptr(q), _ptr(kv_cache), _ptr(in_pos), _ptr(out),
                               _ptr(ws), nbytes, _stream()), "sjd_attention")
    return out, ws[:4].view(torch.int32)


class Context:
    """sjd_init / sjd_prefill / sjd_step on borrowed torch tensors."""

    def __init__(self, cfg: sjd_model_cfg, weights: dict, device="cuda"):
        self.cfg = cfg
        self.device = torch.device(device)
        self.weights = weights  # keep the tensors alive: the library borrows them
        nbytes = sjd_workspace_bytes(cfg)
        if nbytes == 0:
            raise SJDError(SJD_ERR_BAD_ARG, "sjd_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        n_layers = cfg.n_layers
        self._arrays = {}
        w = sjd_weights()
        w.tok_emb, w.final_norm, w.lm_head = (weights[k].data_ptr() for k in ("tok_emb", "final_norm", "lm_head"))
        names = ["attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"]
        if n_layers and "q_norm" in weights["layers"][0]:   # QK-norm variant
            names += ["q_norm", "k_norm"]
        for name in names:
            arr = (C.c_void_p * n_layers)(*[weights["layers"][l][name].data_ptr() for l in range(n_layers)])
            self._arrays[name] = arr
            setattr(w, name, C.cast(arr, _PP))
        self._w = w
        self._ctx = C.c_void_p()
        _check(lib().sjd_init(C.byref(self._ctx), C.byref(cfg), C.byref(w), _ptr(self.workspace), nbytes), "sjd_init")
        self.batch = self.window = 0
        self._guided = False

    def prefill(self, prompt, sample: sjd_sample_cfg):
        """prompt: int32 cuda tensor [B][P]."""
        assert prompt.dtype == torch.int32 and prompt.is_cuda and prompt.is_contiguous()
        self._prompt = prompt
        self.batch, self.window = int(prompt.shape[0]), int(sample.window)
        self._guided = float(sample.guidance) != 0.0
        _check(lib().sjd_prefill(self._ctx, self.batch, _ptr(prompt), int(prompt.shape[1]), C.byref(sample),
                                 _stream()), "sjd_prefill")

    def prefill_ragged(self, prompt, prompt_lens, sample: sjd_sample_cfg):
        """prompt: int32 cuda tensor [B][row_stride]; prompt_lens: B host integers (sequence b uses the first
        prompt_lens[b] tokens of its row)."""
        assert prompt.dtype == torch.int32 and prompt.is_cuda and prompt.is_contiguous()
        self._prompt = prompt
        self.batch, self.window = int(prompt.shape[0]), int(sample.window)
        self._guided = float(sample.guidance) != 0.0
        lens = (C.c_int32 * self.batch)(*[int(x) for x in prompt_lens])
        _check(lib().sjd_prefill_ragged(self._ctx, self.batch, _ptr(prompt), lens, int(prompt.shape[1]), C.byref(sample),
                                        _stream()), "sjd_prefill_ragged")

    def step(self, out: StepOut | None = None):
        _check(lib().sjd_step(self._ctx, C.byref(out.c) if out is not None else None, _stream()), "sjd_step")

    def get_window(self, out: StepOut):
        _check(lib().sjd_get_window(self._ctx, C.byref(out.c), _stream()), "sjd_get_window")

    def get_tokens(self, row_stride: int | None = None):
        """(tokens int32 [images][row_stride], counts int32 [images]) on the device: every image's prompt and the
        tokens fixed so far; see sjd_get_tokens."""
        images = self.batch // 2 if self._guided else self.batch
        row_stride = int(row_stride or self.cfg.max_seq)
        tokens = torch.zeros(images, row_stride, dtype=torch.int32, device=self.device)
        counts = torch.zeros(images, dtype=torch.int32, device=self.device)
        _check(lib().sjd_get_tokens(self._ctx, _ptr(tokens), row_stride, _ptr(counts), _stream()), "sjd_get_tokens")
        return tokens, counts

    def peek_logits(self):
        t = torch.empty(self.batch, self.window, self.cfg.vocab, dtype=TORCH_DTYPES[self.cfg.dtype], device=self.device)
        _check(lib().sjd_peek_logits(self._ctx, _ptr(t), t.numel() * t.element_size(), _stream()), "sjd_peek_logits")
        return t

    def trace(self, enable: bool):
        _check(lib().sjd_trace(self._ctx, 1 if enable else 0), "sjd_trace")

    def trace_read(self):
        """{'ms': {class: ms}, 'launches': {class: n}, 'gemm_weight_bytes': float}"""
        ms, n, wb = (C.c_double * 4)(), (C.c_int64 * 4)(), C.c_double()
        _check(lib().sjd_trace_read(self._ctx, ms, n, C.byref(wb)), "sjd_trace_read")
        names = ("gemm", "attention", "verify", "other")
        return {"ms": dict(zip(names, list(ms))), "launches": dict(zip(names, list(n))),
                "gemm_weight_bytes": float(wb.value)}

    def info(self) -> dict:
        """Which kernels the steps of this (pre-filled) context run; see sjd_get_info."""
        i = sjd_info()
        _check(lib().sjd_get_info(self._ctx, C.byref(i)), "sjd_get_info")
        return {n: int(getattr(i, n)) for n, _ in sjd_info._fields_}

    def device_status(self) -> int:
        return int(lib().sjd_last_device_status(self._ctx))

    def close(self):
        if self._ctx:
            lib().sjd_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sjd_launch_count() -> int:
    return int(lib().sjd_launch_count())


def weights_to_device(weights: dict, device="cuda") -> dict:
    out = {k: v.to(device).contiguous() for k, v in weights.items() if k != "layers"}
    out["layers"] = [{k: v.to(device).contiguous() for k, v in lw.items()} for lw in weights["layers"]]
    return out
