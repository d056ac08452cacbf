// Context, workspace layout and the per-step launch sequence (Sec. 4.1: pre-fill, then one forward
// pass + verification + window slide per iteration).  All decoding state (committed tokens, window,
// counters, step index) lives in device memory, so consecutive steps are enqueued back to back with
// no host round trip.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <new>
#include <vector>

#include "common.cuh"

namespace sjd {
// Key-range splits of the attention grid: heads * batch * splits CTAs, two of which fit one SM (their
// K/V rings take ~99 KB each), so the grid is sized to fill one wave of 2 * 148 slots and no more.
#ifndef SJD_ATTN_SLOTS
#define SJD_ATTN_SLOTS (2 * 148)
#endif
int attention_splits(int n_heads, int batch) {
  int s = SJD_ATTN_SLOTS / (n_heads * batch);
  return s < 1 ? 1 : (s > 16 ? 16 : s);
}

namespace {

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }
inline size_t esize(int dtype) { return dtype == SJD_F32 ? 4 : 2; }

constexpr int kMaxGemmCtas = 160;    // upper bound on the SM count used to size split-K scratch

struct WMap {
  TensorMap map;
  bool valid = false;
};
struct LayerMaps {
  WMap wq, wk, wv, wo, w_gate, w_up, w_down;
  WMap gate_gu, up_gu;   // gate and up matrices in boxes of gu_rows rows: the gate|up launch that applies SwiGLU itself
};
struct XMaps {
  TensorMap h, attn, act;
};

struct Layout {
  size_t kv, logits[2], stats[2], row_out, counters, step, status;
  size_t x, h, qkv, q, attn, gu, act, partial, rope;
  size_t xs_h, xs_attn, xs_act, gemm_planes, ss_part;
  size_t committed, n, w_eff, draft, q_kind, q_row, q_draft, in_tok, in_pos;
  size_t ring, ring_stats, n_prev, w_prev;   // Sec. 4.2 (d): retained logits rows (max_ring > 0)
  size_t prompt_lens;                        // [max_batch] prompt length of every sequence
  size_t page_table;                         // [max_batch][pages_per_seq] (paged cache, kv_pages > 0)
  size_t total;
};

bool cfg_valid(const sjd_model_cfg *c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->d_model < 1 || c->n_heads < 1 || c->n_kv_heads < 1 || c->head_dim < 2 ||
      c->ffn_hidden < 1 || c->vocab < 1 || c->max_batch < 1 || c->max_seq < 2 || c->max_window < 1)
    return false;
  if (c->head_dim % 2 != 0 || c->n_heads % c->n_kv_heads != 0) return false;
  if (!(c->rms_eps > 0.0f) || !(c->rope_theta > 0.0f)) return false;
  if (c->max_ring < 0 || c->kv_pages < 0) return false;
  return true;
}

Layout make_layout(const sjd_model_cfg &c) {
  Layout L;
  const size_t es = esize(c.dtype);
  const size_t Mx = (size_t)c.max_batch * c.max_window;
  const size_t nq = (size_t)c.n_heads * c.head_dim, nk = (size_t)c.n_kv_heads * c.head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align256(bytes);
    return o;
  };
  // contiguous: max_seq rows for every sequence; paged: kv_pages pages shared by the batch plus one spare page
  // that unassigned table entries point to
  L.kv = c.kv_pages > 0 ? take((size_t)(c.kv_pages + 1) * c.n_layers * 2 * nk * KV_PAGE * es)
                        : take((size_t)c.n_layers * c.max_batch * 2 * nk * c.max_seq * es);
  L.logits[0] = take(Mx * c.vocab * es);
  L.logits[1] = take(Mx * c.vocab * es);
  L.stats[0] = take(Mx * sizeof(RowStats));
  L.stats[1] = take(Mx * sizeof(RowStats));
  L.row_out = take(Mx * sizeof(RowOut));
  L.counters = take(((size_t)c.max_batch + 1) * 4);
  L.step = take(4);
  L.status = take(4);
  L.x = take(Mx * c.d_model * 4);
  L.h = take(Mx * c.d_model * 4);
  L.qkv = take(Mx * (nq + 2 * nk) * 4);
  L.q = take(Mx * nq * 4);
  L.attn = take(Mx * nq * 4);
  L.gu = take(Mx * 2 * c.ffn_hidden * 4);
  L.act = take(Mx * c.ffn_hidden * 4);
  size_t part = 0;
  for (int b = 1; b <= c.max_batch; ++b) {
    const size_t need = (size_t)b * c.max_window * c.n_heads * attention_splits(c.n_heads, b) * (c.head_dim + 2);
    part = need > part ? need : part;
  }
  L.partial = take(part * 4);
  // bf16 hi/lo planes of the GEMM inputs, stream-K partials and tickets (tensor-core path)
  const size_t Ma = (Mx + 15) / 16 * 16;
  L.xs_h = take(2 * Ma * c.d_model * 2);
  L.xs_attn = take(2 * Ma * nq * 2);
  L.xs_act = take(2 * Ma * c.ffn_hidden * 2);
  {
    // fp32 partial planes of one GEMM launch: the largest splits * rows * columns over the launches
    const int tiles[4] = {(int)((nq + 2 * nk) / 128), c.d_model / 128, 2 * c.ffn_hidden / 128, c.d_model / 128};
    const int kbs[4] = {c.d_model / 64, (int)(nq / 64), c.d_model / 64, c.ffn_hidden / 64};
    const size_t cols[4] = {nq + 2 * nk, (size_t)c.d_model, (size_t)2 * c.ffn_hidden, (size_t)c.d_model};
    size_t need = 0;
    for (int i = 0; i < 4; ++i) {
      for (size_t rows = 16; rows < Mx + 16 && rows <= 1024; rows += 16) {   // splits shrink as the token slabs grow
        const size_t m = rows < Mx ? rows : Mx;
        const size_t n = (size_t)gemm_tc_splits(gemm_tc_plan((int)m), tiles[i] > 0 ? tiles[i] : 1, kbs[i],
                                                 kMaxGemmCtas) * m * cols[i];
        need = n > need ? n : need;
      }
    }
    L.gemm_planes = take(need * 4);
  }
  L.ss_part = take(Mx * (size_t)resid_gain_parts(c.d_model) * 4);
  L.rope = take((size_t)c.max_seq * (c.head_dim / 2) * sizeof(float2));
  L.committed = take((size_t)c.max_batch * c.max_seq * 4);
  L.n = take((size_t)c.max_batch * 4);
  L.w_eff = take((size_t)c.max_batch * 4);
  L.draft = take(Mx * 4);
  L.q_kind = take(Mx * 4);
  L.q_row = take(Mx * 4);
  L.q_draft = take(Mx * 4);
  L.in_tok = take(Mx * 4);
  L.in_pos = take(Mx * 4);
  const size_t ring_rows = (size_t)c.max_batch * (c.max_ring > 0 ? c.max_ring : 0);
  L.ring = take(ring_rows * c.vocab * es);
  L.ring_stats = take(ring_rows * sizeof(RowStats));
  L.n_prev = take((size_t)c.max_batch * 4);
  L.w_prev = take((size_t)c.max_batch * 4);
  L.prompt_lens = take((size_t)c.max_batch * 4);
  L.page_table = take(c.kv_pages > 0 ? (size_t)c.max_batch * ((c.max_seq + KV_PAGE - 1) / KV_PAGE) * 4 : 0);
  L.total = off;
  return L;
}

// Optional per-class timing of the launches of a step with CUDA events on the launching stream
// (diagnostics: which kernels the step time goes to).  Off by default; when on, every launch is
// bracketed by two events and each step ends with a stream synchronisation.
enum TraceClass { TC_GEMM = 0, TC_ATTENTION = 1, TC_VERIFY = 2, TC_OTHER = 3, TC_COUNT = 4 };
struct Tracer {
  bool on = false;
  std::vector<cudaEvent_t> ev;
  std::vector<int> cls;
  size_t used = 0;
  double ms[TC_COUNT] = {0, 0, 0, 0};
  long long launches[TC_COUNT] = {0, 0, 0, 0};
  double gemm_weight_bytes = 0;
  void begin(int c, cudaStream_t s) {
    if (!on) return;
    if (used + 2 > ev.size()) {
      cudaEvent_t a = nullptr, b = nullptr;
      cudaEventCreate(&a);
      cudaEventCreate(&b);
      ev.push_back(a);
      ev.push_back(b);
    }
    cls.push_back(c);
    cudaEventRecord(ev[used], s);
  }
  void end(cudaStream_t s) {
    if (!on) return;
    cudaEventRecord(ev[used + 1], s);
    used += 2;
  }
  int flush(cudaStream_t s) {
    if (!on || used == 0) return SJD_OK;
    SJD_CUDA(cudaStreamSynchronize(s));
    for (size_t i = 0; i < used; i += 2) {
      float t = 0.0f;
      SJD_CUDA(cudaEventElapsedTime(&t, ev[i], ev[i + 1]));
      ms[cls[i / 2]] += t;
      launches[cls[i / 2]] += 1;
    }
    used = 0;
    cls.clear();
    return SJD_OK;
  }
  ~Tracer() {
    for (cudaEvent_t e : ev) cudaEventDestroy(e);
  }
};

// prompt: [B][ld] token ids, sequence b uses the first st.prompt_lens[b] of its row
__global__ void prefill_setup_kernel(const int32_t *prompt, int ld, SeqState st, uint32_t *step, int32_t *counters,
                                     int B) {
  const int b = blockIdx.x;
  const int P = st.prompt_lens[b];
  for (int i = threadIdx.x; i < P; i += blockDim.x) st.committed[(size_t)b * st.max_seq + i] = prompt[(size_t)b * ld + i];
  if (threadIdx.x == 0) {
    st.n[b] = P;
    st.w_eff[b] = 0;
    counters[b] = 0;
    if (b == 0) {
      counters[B] = 0;
      *step = kStepInitialWindow;
    }
  }
}

__global__ void prefill_inputs_kernel(const int32_t *prompt, int ld, const int32_t *prompt_lens, int c0, int rows,
                                      int32_t *in_tok, int32_t *in_pos) {
  const int b = blockIdx.x;
  const int P = prompt_lens[b];
  for (int k = threadIdx.x; k < rows; k += blockDim.x) {
    const int pos = c0 + k;
    const bool act = pos < P - 1;
    in_tok[b * rows + k] = act ? prompt[(size_t)b * ld + pos] : 0;
    in_pos[b * rows + k] = act ? pos : -1;
  }
}

// one block per image; `streams` sequences per image hold the same window (2 under guidance), the first is read
__global__ void get_window_kernel(SeqState st, sjd_step_out o, int W, int streams) {
  const int b = blockIdx.x, sb = b * streams;
  for (int k = threadIdx.x; k < W; k += blockDim.x) {
    const int i = b * W + k, si = sb * W + k;
    if (o.draft) o.draft[i] = st.draft[si];
    if (o.q_kind) o.q_kind[i] = st.q_kind[si];
    if (o.q_draft) o.q_draft[i] = st.q_draft[si];
  }
  if (threadIdx.x == 0 && o.total_committed) o.total_committed[b] = st.n[sb];
}

// one block per image: the fixed tokens of its (first) stream
__global__ void get_tokens_kernel(SeqState st, int32_t *tokens, int row_stride, int32_t *counts, int streams) {
  const int b = blockIdx.x, sb = b * streams;
  const int n = st.n[sb];
  for (int i = threadIdx.x; i < n && i < row_stride; i += blockDim.x)
    tokens[(size_t)b * row_stride + i] = st.committed[(size_t)sb * st.max_seq + i];
  if (threadIdx.x == 0 && counts) counts[b] = n;
}

}  // namespace
}  // namespace sjd

using namespace sjd;

struct sjd_ctx {
  sjd_model_cfg cfg;
  Layout lay;
  char *ws;
  const void *tok_emb, *final_norm, *lm_head;
  std::vector<const void *> attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down;
  std::vector<const void *> q_norm, k_norm;   // QK-norm gains per layer (null entries: the plain model)
  QkNorm qk_norm(int l) const { return QkNorm{q_norm[l], k_norm[l], cfg.rms_eps}; }
  sjd_sample_cfg sample;
  int batch, prompt_len, window;   // prompt_len: the longest prompt of the batch
  std::vector<int32_t> prompt_lens;  // per sequence (host copy; the device copy is in the workspace)
  std::vector<int32_t> page_table;   // paged cache: host copy of [max_batch][pages_per_seq]
  bool prefilled;
  uint32_t host_step;  // number of sjd_step calls since prefill == device step index
  cudaStream_t last_stream;
  // One captured CUDA graph per logits-buffer parity: a step is ~330 launches, and replaying a graph
  // takes the host out of the critical path.  Keyed by the caller's output pointers.
  struct StepGraph {
    cudaGraphExec_t exec = nullptr;
    sjd_step_out out;
    bool has_out = false;
    long long launches = 0;
  } graphs[2];
  cudaStream_t capture_stream = nullptr;
  bool graphs_enabled = true;
  void drop_graphs() {
    for (int i = 0; i < 2; ++i) {
      if (graphs[i].exec) cudaGraphExecDestroy(graphs[i].exec);
      graphs[i].exec = nullptr;
    }
  }
  ~sjd_ctx() {
    drop_graphs();
    if (capture_stream) cudaStreamDestroy(capture_stream);
  }
  Tracer tracer;
  bool use_tc = false;   // bf16 model on a device with tensor memory: tensor-core GEMM path
  bool all_tc = false;   // every projection of the model is covered by it
  bool gu_fused = false; // gate|up projection with SwiGLU in its epilogue (every layer has the maps for it)
  int gu_rows = 0;       // feature rows of the gate (and of the up) matrix per CTA of that launch
  int head_rows = 0;     // weight rows per CTA of the logits projection (0: 128)
  WMap wmap_head_r;      // lm_head in boxes of head_rows rows
  int n_ctas = 0;
  std::vector<LayerMaps> wmaps;
  WMap wmap_head;
  std::map<int, XMaps> xmaps;   // keyed by padded row count
  TensorMap kv_map;             // whole KV cache as [planes][max_seq][head_dim]
  bool kv_map_valid = false;
  int rows_alloc() const { return ((cfg.max_batch * cfg.max_window) + 15) / 16 * 16; }

  template <typename T> T *at(size_t off) const { return reinterpret_cast<T *>(ws + off); }
  SeqState state() const {
    SeqState st;
    st.committed = at<int32_t>(lay.committed);
    st.n = at<int32_t>(lay.n);
    st.w_eff = at<int32_t>(lay.w_eff);
    st.draft = at<int32_t>(lay.draft);
    st.q_kind = at<int32_t>(lay.q_kind);
    st.q_row = at<int32_t>(lay.q_row);
    st.q_draft = at<float>(lay.q_draft);
    st.in_tok = at<int32_t>(lay.in_tok);
    st.in_pos = at<int32_t>(lay.in_pos);
    st.max_seq = cfg.max_seq;
    st.prompt_lens = at<int32_t>(lay.prompt_lens);
    st.n_generate = sample.n_generate;
    st.init = sample.init;
    st.grid_stride = sample.grid_stride;
    return st;
  }
  int pages_per_seq() const { return (cfg.max_seq + KV_PAGE - 1) / KV_PAGE; }
  KvLayout kv_layer(int l) const {
    KvLayout kv;
    const size_t per_layer = (size_t)cfg.max_batch * 2 * cfg.n_kv_heads * cfg.max_seq * cfg.head_dim * esize(cfg.dtype);
    kv.n_kv_heads = cfg.n_kv_heads;
    kv.max_seq = cfg.max_seq;
    kv.head_dim = cfg.head_dim;
    kv.layer = l;
    kv.n_layers = cfg.n_layers;
    if (cfg.kv_pages > 0) {   // one pool for all layers; the page table says where a sequence's rows are
      kv.base = ws + lay.kv;
      kv.page_table = reinterpret_cast<const int32_t *>(ws + lay.page_table);
      kv.pages_per_seq = pages_per_seq();
    } else {
      kv.base = ws + lay.kv + (size_t)l * per_layer;
      kv.page_table = nullptr;
      kv.pages_per_seq = 0;
    }
    return kv;
  }
};

namespace sjd {
namespace {

// One forward pass of M = batch * rows_per_seq rows whose tokens / positions are in st.in_tok / in_pos.
// Two pipelines: the tensor-core one (bf16 model, every projection covered by the weight-streaming
// GEMM: partial planes + fused consumer kernels) and the generic one (any dtype and shape).
#define SJD_TRY(call) do { rc = (call); if (rc != SJD_OK) return rc; } while (0)
#define SJD_TR(klass, call) do { tr.begin(klass, stream); rc = (call); tr.end(stream); if (rc != SJD_OK) return rc; } while (0)

int forward_generic(sjd_ctx *c, int rows_per_seq, void *logits_out, cudaStream_t stream) {
  const sjd_model_cfg &g = c->cfg;
  const int dt = g.dtype;
  const int M = c->batch * rows_per_seq;
  const int d = g.d_model, F = g.ffn_hidden;
  const int nq = g.n_heads * g.head_dim, nk = g.n_kv_heads * g.head_dim, nqkv = nq + 2 * nk;
  const SeqState st = c->state();
  float *x = c->at<float>(c->lay.x);
  float *h = c->at<float>(c->lay.h);
  float *qkv = c->at<float>(c->lay.qkv);
  float *q = c->at<float>(c->lay.q);
  float *attn = c->at<float>(c->lay.attn);
  float *gu = c->at<float>(c->lay.gu);
  float *act = c->at<float>(c->lay.act);
  float *partial = c->at<float>(c->lay.partial);
  const float2 *rope = c->at<float2>(c->lay.rope);
  const int splits = attention_splits(g.n_heads, c->batch);
  int rc;
  Tracer &tr = c->tracer;
  const double es = (double)esize(dt);
  auto gemm = [&](const void *w, const float *a, int lda, void *out, int ldc, int n_out, int k_in, int epi) -> int {
    if (tr.on) tr.gemm_weight_bytes += (double)n_out * (double)k_in * es;
    tr.begin(TC_GEMM, stream);
    const int r = launch_gemm_simt(dt, a, lda, w, out, ldc, M, n_out, k_in, epi, stream);
    tr.end(stream);
    return r;
  };
  SJD_TR(TC_OTHER, launch_embed(dt, c->tok_emb, st.in_tok, x, M, d, g.vocab, stream));
  for (int l = 0; l < g.n_layers; ++l) {
    SJD_TR(TC_OTHER, launch_rmsnorm(dt, x, c->attn_norm[l], h, M, d, g.rms_eps, stream));
    SJD_TRY(gemm(c->wq[l], h, d, qkv, nqkv, nq, d, EPI_STORE_F32));
    SJD_TRY(gemm(c->wk[l], h, d, qkv + nq, nqkv, nk, d, EPI_STORE_F32));
    SJD_TRY(gemm(c->wv[l], h, d, qkv + nq + nk, nqkv, nk, d, EPI_STORE_F32));
    const KvLayout kv = c->kv_layer(l);
    SJD_TR(TC_OTHER, launch_rope_append(dt, qkv, st.in_pos, rope, q, kv, M, rows_per_seq, g.n_heads, c->qk_norm(l), stream));
    SJD_TR(TC_ATTENTION, launch_attention(dt, q, kv, st.in_pos, attn, partial, M, rows_per_seq, g.n_heads, splits, stream));
    SJD_TRY(gemm(c->wo[l], attn, nq, x, d, d, nq, EPI_ADD_F32));
    SJD_TR(TC_OTHER, launch_rmsnorm(dt, x, c->ffn_norm[l], h, M, d, g.rms_eps, stream));
    SJD_TRY(gemm(c->w_gate[l], h, d, gu, 2 * F, F, d, EPI_STORE_F32));
    SJD_TRY(gemm(c->w_up[l], h, d, gu + F, 2 * F, F, d, EPI_STORE_F32));
    SJD_TR(TC_OTHER, launch_swiglu(gu, act, M, F, stream));
    SJD_TRY(gemm(c->w_down[l], act, F, x, d, d, F, EPI_ADD_F32));
  }
  if (logits_out) {
    SJD_TR(TC_OTHER, launch_rmsnorm(dt, x, c->final_norm, h, M, d, g.rms_eps, stream));
    SJD_TRY(gemm(c->lm_head, h, d, logits_out, g.vocab, g.vocab, d, EPI_STORE_T));
  }
  return SJD_OK;
}

int forward_tc(sjd_ctx *c, const XMaps &xm, int rows_per_seq, void *logits_out, cudaStream_t stream) {
  const sjd_model_cfg &g = c->cfg;
  const int dt = g.dtype;
  const int M = c->batch * rows_per_seq;
  const int d = g.d_model, F = g.ffn_hidden;
  const int nq = g.n_heads * g.head_dim, nk = g.n_kv_heads * g.head_dim, nqkv = nq + 2 * nk;
  const SeqState st = c->state();
  float *x = c->at<float>(c->lay.x);
  float *q = c->at<float>(c->lay.q);
  float *attn = c->at<float>(c->lay.attn);
  float *partial = c->at<float>(c->lay.partial);
  float *planes = c->at<float>(c->lay.gemm_planes);
  int *status = c->at<int>(c->lay.status);
  const float2 *rope = c->at<float2>(c->lay.rope);
  const int att_splits = attention_splits(g.n_heads, c->batch);
  const int Ma = c->rows_alloc();
  const HiLoOut hl_h{c->at<__nv_bfloat16>(c->lay.xs_h), (size_t)Ma * d};
  const HiLoOut hl_attn{c->at<__nv_bfloat16>(c->lay.xs_attn), (size_t)Ma * nq};
  const HiLoOut hl_act{c->at<__nv_bfloat16>(c->lay.xs_act), (size_t)Ma * F};
  float *ss_part = c->at<float>(c->lay.ss_part);
  const RowScale rs{ss_part, resid_gain_parts(d), 1.0f / (float)d, g.rms_eps};
  int rc;
  Tracer &tr = c->tracer;

  // one GEMM launch over n_mats matrices sharing the activation operand; returns the planes it wrote
  auto gemm = [&](const WMap *const *wm, int n_mats, const int *n_out, const TensorMap &x_map, int k_in, int ldc, void *out,
                  bool bf16_out, PlaneSet *ps, int tile_rows = 0, const HiLoOut *act = nullptr) -> int {
    GemmTcCall call;
    memset(&call, 0, sizeof(call));
    call.tile_rows = tile_rows;
    if (act) {
      call.act_hi = act->base;
      call.act_lo_off = act->lo_offset;
    }
    int tiles = 0, col = 0;
    for (int j = 0; j < n_mats; ++j) {
      call.w_map[j] = &wm[j]->map;
      call.n_out[j] = n_out[j];
      call.col_off[j] = col;
      col += n_out[j];
      tiles += n_out[j] / 128;
      if (tr.on) tr.gemm_weight_bytes += (double)n_out[j] * (double)k_in * 2.0;
    }
    for (int j = n_mats; j < 3; ++j) call.w_map[j] = call.w_map[0];
    call.n_mats = n_mats;
    call.x_map = &x_map;
    call.x_lo_row = Ma;
    call.M = M;
    call.K = k_in;
    call.splits = (bf16_out || act) ? 1 : gemm_tc_splits(gemm_tc_plan(M), tiles, k_in / 64, c->n_ctas);
    call.out = out;
    call.plane_stride = (size_t)M * ldc;
    call.ldc = ldc;
    call.store_bf16 = bf16_out ? 1 : 0;
    call.status = status;
    call.n_sms = c->n_ctas;
    if (bf16_out || act) {   // the logits projection and the gate|up launch apply the pending row scale themselves
      call.ss_part = rs.ss_part;
      call.n_part = rs.n_part;
      call.inv_d = rs.inv_d;
      call.eps = rs.eps;
    }
    if (ps) *ps = PlaneSet{reinterpret_cast<const float *>(out), call.plane_stride, ldc, call.splits};
    tr.begin(TC_GEMM, stream);
    const int r = launch_gemm_tc(call, stream);
    tr.end(stream);
    return r;
  };

  SJD_TR(TC_OTHER, launch_embed(dt, c->tok_emb, st.in_tok, x, M, d, g.vocab, stream));
  PlaneSet pending{nullptr, 0, 0, 0};   // planes still to be added into the residual stream
  for (int l = 0; l < g.n_layers; ++l) {
    const LayerMaps &lm = c->wmaps[l];
    PlaneSet ps;
    SJD_TR(TC_OTHER, launch_resid_gain(dt, x, pending, c->attn_norm[l], hl_h, ss_part, M, d, stream));
    {
      const WMap *wm[3] = {&lm.wq, &lm.wk, &lm.wv};
      const int n_out[3] = {nq, nk, nk};
      SJD_TRY(gemm(wm, 3, n_out, xm.h, d, nqkv, planes, false, &ps));
    }
    const KvLayout kv = c->kv_layer(l);
    SJD_TR(TC_OTHER, launch_qkv_finish(dt, ps, rs, st.in_pos, rope, q, kv, M, rows_per_seq, g.n_heads, c->qk_norm(l), stream));
    if (c->kv_map_valid && attention_mma_supported(g.head_dim, rows_per_seq)) {
      SJD_TR(TC_ATTENTION, launch_attention_mma(c->kv_map, l * g.max_batch * 2 * g.n_kv_heads, kv, q, st.in_pos, partial, attn,
                                                hl_attn, status, M, rows_per_seq, g.n_heads, g.n_kv_heads, g.head_dim,
                                                att_splits, stream));
      if (att_splits > 1)
        SJD_TR(TC_ATTENTION,
               launch_attention_combine(partial, st.in_pos, attn, M, g.n_heads, g.head_dim, att_splits, stream, hl_attn));
    } else {
      SJD_TR(TC_ATTENTION,
             launch_attention(dt, q, kv, st.in_pos, attn, partial, M, rows_per_seq, g.n_heads, att_splits, stream, hl_attn));
    }
    {
      const WMap *wm[1] = {&lm.wo};
      const int n_out[1] = {d};
      SJD_TRY(gemm(wm, 1, n_out, xm.attn, nq, d, planes, false, &ps));
    }
    SJD_TR(TC_OTHER, launch_resid_gain(dt, x, ps, c->ffn_norm[l], hl_h, ss_part, M, d, stream));
    if (c->gu_fused) {
      const WMap *wm[2] = {&lm.gate_gu, &lm.up_gu};
      const int n_out[2] = {F, F};
      SJD_TRY(gemm(wm, 2, n_out, xm.h, d, F, nullptr, false, nullptr, c->gu_rows, &hl_act));
    } else {
      const WMap *wm[2] = {&lm.w_gate, &lm.w_up};
      const int n_out[2] = {F, F};
      SJD_TRY(gemm(wm, 2, n_out, xm.h, d, 2 * F, planes, false, &ps));
      SJD_TR(TC_OTHER, launch_swiglu_finish(ps, rs, hl_act, M, F, stream));
    }
    {
      const WMap *wm[1] = {&lm.w_down};
      const int n_out[1] = {d};
      SJD_TRY(gemm(wm, 1, n_out, xm.act, F, d, planes, false, &pending));
    }
  }
  if (logits_out) {
    SJD_TR(TC_OTHER, launch_resid_gain(dt, x, pending, c->final_norm, hl_h, ss_part, M, d, stream));
    const int head_rows = M <= 128 ? c->head_rows : 0;   // several token slabs share 128-row tiles through L2
    const WMap *wm[1] = {head_rows ? &c->wmap_head_r : &c->wmap_head};
    const int n_out[1] = {g.vocab};
    SJD_TRY(gemm(wm, 1, n_out, xm.h, d, g.vocab, logits_out, true, nullptr, head_rows));
  }
  return SJD_OK;
}
#undef SJD_TR
#undef SJD_TRY

int forward(sjd_ctx *c, int rows_per_seq, void *logits_out, cudaStream_t stream) {
  const int M = c->batch * rows_per_seq;
  if (c->use_tc && c->all_tc && M <= 1024) {
    auto it = c->xmaps.find((M + 15) / 16 * 16);
    if (it != c->xmaps.end()) {
      // every kernel of this pipeline waits for its predecessor itself: launch them overlapped
      g_pdl = !c->tracer.on;
      const int rc = forward_tc(c, it->second, rows_per_seq, logits_out, stream);
      g_pdl = false;
      return rc;
    }
  }
  return forward_generic(c, rows_per_seq, logits_out, stream);
}

int run_verify(sjd_ctx *c, const sjd_step_out *out, cudaStream_t stream) {
  VerifyParams p;
  memset(&p, 0, sizeof(p));
  const SeqState st = c->state();
  p.logits[0] = c->ws + c->lay.logits[0];
  p.logits[1] = c->ws + c->lay.logits[1];
  p.stats[0] = c->at<RowStats>(c->lay.stats[0]);
  p.stats[1] = c->at<RowStats>(c->lay.stats[1]);
  p.draft = st.draft;
  p.q_kind = st.q_kind;
  p.q_row = st.q_row;
  p.prev_stats_valid = 1;
  p.row_out = c->at<RowOut>(c->lay.row_out);
  p.seq_counter = c->at<int32_t>(c->lay.counters);
  p.done_counter = p.seq_counter + c->batch;
  p.w_eff = st.w_eff;
  p.base_pos = nullptr;
  p.step_ptr = c->at<uint32_t>(c->lay.step);
  p.B = c->batch;
  p.W = c->window;
  p.V = c->cfg.vocab;
  p.temperature = c->sample.temperature;
  p.top_k = c->sample.top_k;
  p.seed_lo = (uint32_t)(c->sample.seed & 0xFFFFFFFFull);
  p.seed_hi = (uint32_t)(c->sample.seed >> 32);
  p.seq_base = (uint32_t)c->sample.seq_base;
  p.e2e = 1;
  p.schedule = c->sample.schedule;
  p.st = st;
  if (c->sample.guidance != 0.0f) {   // sequences 2i, 2i + 1 = conditional and unconditional stream of image i
    p.paired = 1;
    p.guidance = c->sample.guidance;
    p.B = c->batch / 2;
    p.done_counter = p.seq_counter + p.B;
  }
  if (out) p.out = *out;
  if (c->sample.init == SJD_INIT_RESAMPLE_ABOVE) {   // retained rows: read by this launch, refreshed after it
    p.ring = c->ws + c->lay.ring;
    p.ring_stats = c->at<RowStats>(c->lay.ring_stats);
    p.ring_len = c->cfg.max_ring;
    p.n_prev = c->at<int32_t>(c->lay.n_prev);
    p.w_prev = c->at<int32_t>(c->lay.w_prev);
    const int rc = launch_verify(p, c->cfg.dtype, stream);
    return rc != SJD_OK ? rc : launch_retain_rows(p, c->cfg.dtype, stream);
  }
  return launch_verify(p, c->cfg.dtype, stream);
}

}  // namespace
}  // namespace sjd

extern "C" size_t sjd_workspace_bytes(const sjd_model_cfg *cfg) {
  if (!cfg_valid(cfg) || (cfg->dtype != SJD_F32 && cfg->dtype != SJD_BF16)) return 0;
  return make_layout(*cfg).total;
}

extern "C" int sjd_init(sjd_ctx **out, const sjd_model_cfg *cfg, const sjd_weights *w, void *workspace,
                        size_t workspace_bytes) {
  if (!out || !cfg || !w || !workspace) return SJD_ERR_BAD_ARG;
  *out = nullptr;
  if (!cfg_valid(cfg)) return SJD_ERR_BAD_ARG;
  if (cfg->dtype != SJD_F32 && cfg->dtype != SJD_BF16) return SJD_ERR_UNSUPPORTED;
  if (cfg->head_dim > 128 || cfg->max_window > 64) return SJD_ERR_UNSUPPORTED;
  if (((uintptr_t)workspace & 255u) != 0) return SJD_ERR_BAD_ARG;
  if (!w->tok_emb || !w->final_norm || !w->lm_head || !w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo ||
      !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down)
    return SJD_ERR_BAD_ARG;
  for (int l = 0; l < cfg->n_layers; ++l)
    if (!w->attn_norm[l] || !w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate[l] ||
        !w->w_up[l] || !w->w_down[l])
      return SJD_ERR_BAD_ARG;
  const Layout lay = make_layout(*cfg);
  if (workspace_bytes < lay.total) return SJD_ERR_CAPACITY;

  sjd_ctx *c = new (std::nothrow) sjd_ctx();
  if (!c) return SJD_ERR_BAD_ARG;
  c->cfg = *cfg;
  c->lay = lay;
  c->ws = (char *)workspace;
  c->tok_emb = w->tok_emb;
  c->final_norm = w->final_norm;
  c->lm_head = w->lm_head;
  const int L = cfg->n_layers;
  c->attn_norm.assign(w->attn_norm, w->attn_norm + L);
  c->wq.assign(w->wq, w->wq + L);
  c->wk.assign(w->wk, w->wk + L);
  c->wv.assign(w->wv, w->wv + L);
  c->wo.assign(w->wo, w->wo + L);
  c->ffn_norm.assign(w->ffn_norm, w->ffn_norm + L);
  c->w_gate.assign(w->w_gate, w->w_gate + L);
  c->w_up.assign(w->w_up, w->w_up + L);
  c->w_down.assign(w->w_down, w->w_down + L);
  c->q_norm.assign(L, nullptr);
  c->k_norm.assign(L, nullptr);
  if (w->q_norm && w->k_norm) {
    c->q_norm.assign(w->q_norm, w->q_norm + L);
    c->k_norm.assign(w->k_norm, w->k_norm + L);
  }
  c->prefilled = false;
  c->batch = c->prompt_len = c->window = 0;
  c->host_step = 0;
  c->last_stream = nullptr;
  memset(&c->sample, 0, sizeof(c->sample));

  // rotary table in double precision: (cos, sin)(pos * theta^(-2i/hd))
  const int half = cfg->head_dim / 2;
  std::vector<float2> table((size_t)cfg->max_seq * half);
  for (int i = 0; i < half; ++i) {
    const double inv_freq = pow((double)cfg->rope_theta, -2.0 * i / cfg->head_dim);
    for (int pos = 0; pos < cfg->max_seq; ++pos) {
      const double a = (double)pos * inv_freq;
      table[(size_t)pos * half + i] = make_float2((float)cos(a), (float)sin(a));
    }
  }
  cudaError_t e = cudaMemcpy(c->ws + lay.rope, table.data(), table.size() * sizeof(float2), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(c->ws + lay.counters, 0, ((size_t)cfg->max_batch + 1) * 4);
  if (e == cudaSuccess) e = cudaMemset(c->ws + lay.status, 0, 4);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    delete c;
    return SJD_ERR_CUDA;
  }
  // tensor-core path: bf16 weights on a device of compute capability 10.x; one TMA descriptor per
  // weight matrix whose shape the kernel covers (the others use the generic kernel)
  c->wmaps.resize(L);
  int dev = 0, cc_major = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && cfg->dtype == SJD_BF16 &&
      cc_major == 10 && sms > 0) {
    c->use_tc = true;
    c->n_ctas = sms < kMaxGemmCtas ? sms : kMaxGemmCtas;
    const int d = cfg->d_model, F = cfg->ffn_hidden;
    const int nq = cfg->n_heads * cfg->head_dim, nk = cfg->n_kv_heads * cfg->head_dim;
    auto mk = [&](WMap &m, const void *w, int n_out, int k_in) {
      m.valid = n_out % 128 == 0 && k_in % 64 == 0 && make_tensor_map_bf16(&m.map, w, n_out, k_in, 128) == SJD_OK;
    };
    for (int l = 0; l < L; ++l) {
      LayerMaps &lm = c->wmaps[l];
      mk(lm.wq, c->wq[l], nq, d);
      mk(lm.wk, c->wk[l], nk, d);
      mk(lm.wv, c->wv[l], nk, d);
      mk(lm.wo, c->wo[l], d, nq);
      mk(lm.w_gate, c->w_gate[l], F, d);
      mk(lm.w_up, c->w_up[l], F, d);
      mk(lm.w_down, c->w_down[l], d, F);
    }
    mk(c->wmap_head, c->lm_head, cfg->vocab, d);
    c->all_tc = c->wmap_head.valid;
    // gate|up with SwiGLU in the epilogue: 64 gate rows and the same 64 up rows per CTA, one K split.
    // (Measured on the 7B shapes: 40 rows per CTA, which fills one wave of two CTAs per SM exactly, is no
    // faster than 64: every CTA reads the whole activation operand, so smaller tiles raise that traffic.)
    {
      int r = 64;
      if (const char *e = getenv("SJD_GU_ROWS")) r = atoi(e);   // tuning: 0 switches the fused launch off, else 8..64
      c->gu_rows = r;
      c->gu_fused = r >= 8 && r <= 64 && d % 64 == 0;
      for (int l = 0; l < L && c->gu_fused; ++l) {
        LayerMaps &lm = c->wmaps[l];
        lm.gate_gu.valid = make_tensor_map_bf16(&lm.gate_gu.map, c->w_gate[l], F, d, r) == SJD_OK;
        lm.up_gu.valid = make_tensor_map_bf16(&lm.up_gu.map, c->w_up[l], F, d, r) == SJD_OK;
        c->gu_fused = lm.gate_gu.valid && lm.up_gu.valid;
      }
    }
    // logits projection: optional tile height below 128 rows (SJD_HEAD_ROWS; measured on the 7B shapes: 112
    // rows = two full waves of CTAs is 4 % slower than 128 rows in 1.7 waves, so the default stays 128)
    if (const char *e = getenv("SJD_HEAD_ROWS")) {
      const int r = atoi(e);
      if (r >= 8 && r < 128 && c->wmap_head.valid &&
          make_tensor_map_bf16(&c->wmap_head_r.map, c->lm_head, cfg->vocab, d, r) == SJD_OK) {
        c->wmap_head_r.valid = true;
        c->head_rows = r;
      }
    }
    // the cache as one 3-D tensor map for the tensor-core attention; unwritten rows must read as finite
    // numbers (a masked probability of 0 times NaN would poison the output), so the cache starts at zero
    // (paged cache: the planes are the pool's [page][layer][k|v][kv_head], each KV_PAGE rows long)
    const bool paged = cfg->kv_pages > 0;
    const long planes = paged ? (long)(cfg->kv_pages + 1) * L * 2 * cfg->n_kv_heads
                              : (long)L * cfg->max_batch * 2 * cfg->n_kv_heads;
    const long plane_rows = paged ? KV_PAGE : cfg->max_seq;
    if (attention_mma_supported(cfg->head_dim, cfg->max_window) &&
        make_kv_tensor_map(&c->kv_map, c->ws + lay.kv, planes, plane_rows, cfg->head_dim) == SJD_OK &&
        cudaMemset(c->ws + lay.kv, 0, (size_t)planes * plane_rows * cfg->head_dim * 2) == cudaSuccess)
      c->kv_map_valid = true;
    for (int l = 0; l < L; ++l) {
      const LayerMaps &lm = c->wmaps[l];
      c->all_tc = c->all_tc && lm.wq.valid && lm.wk.valid && lm.wv.valid && lm.wo.valid && lm.w_gate.valid &&
                  lm.w_up.valid && lm.w_down.valid;
    }
  }
  *out = c;
  return SJD_OK;
}

extern "C" int sjd_prefill(sjd_ctx *c, int batch, const int32_t *prompt, int prompt_len, const sjd_sample_cfg *sample,
                           void *cuda_stream) {
  if (batch < 1 || batch > (1 << 20)) return SJD_ERR_BAD_ARG;
  const std::vector<int32_t> lens((size_t)batch, prompt_len);
  return sjd_prefill_ragged(c, batch, prompt, lens.data(), prompt_len, sample, cuda_stream);
}

extern "C" int sjd_prefill_ragged(sjd_ctx *c, int batch, const int32_t *prompt, const int32_t *prompt_lens, int row_stride,
                                  const sjd_sample_cfg *sample, void *cuda_stream) {
  if (!c || !prompt || !prompt_lens || !sample || batch < 1 || row_stride < 1) return SJD_ERR_BAD_ARG;
  int prompt_len = 0;   // the longest
  for (int b = 0; b < batch; ++b) {
    if (prompt_lens[b] < 1 || prompt_lens[b] > row_stride) return SJD_ERR_BAD_ARG;
    prompt_len = prompt_lens[b] > prompt_len ? prompt_lens[b] : prompt_len;
  }
  int rc = check_sample_cfg(sample, c->cfg.vocab);
  if (rc != SJD_OK) return rc;
  if (sample->n_generate < 0) return SJD_ERR_BAD_ARG;
  if (batch > c->cfg.max_batch || sample->window > c->cfg.max_window) return SJD_ERR_CAPACITY;
  if ((long)prompt_len + sample->n_generate > c->cfg.max_seq) return SJD_ERR_CAPACITY;
  if (sample->guidance != 0.0f) {   // streams come in pairs that share every position
    if (batch % 2 != 0) return SJD_ERR_BAD_ARG;
    for (int b = 0; b < batch; b += 2)
      if (prompt_lens[b] != prompt_lens[b + 1]) return SJD_ERR_BAD_ARG;
  }
  if (sample->init == SJD_INIT_RESAMPLE_ABOVE && c->cfg.max_ring < sample->grid_stride + sample->window)
    return SJD_ERR_CAPACITY;   // a retained row must outlive the window that draws from it
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  c->sample = *sample;
  c->batch = batch;
  c->prompt_len = prompt_len;
  if (c->cfg.kv_pages > 0) {
    // every sequence gets the pages its own prompt and generated tokens need, in order, from page 0; entries
    // past a sequence's last page point to the spare page
    const int pps = c->pages_per_seq();
    c->page_table.assign((size_t)c->cfg.max_batch * pps, c->cfg.kv_pages);
    long next = 0;
    for (int b = 0; b < batch; ++b) {
      const int need = (prompt_lens[b] + sample->n_generate + KV_PAGE - 1) / KV_PAGE;
      if (next + need > c->cfg.kv_pages) return SJD_ERR_CAPACITY;
      for (int i = 0; i < need; ++i) c->page_table[(size_t)b * pps + i] = (int32_t)(next + i);
      next += need;
    }
    SJD_CUDA(cudaMemcpyAsync(c->ws + c->lay.page_table, c->page_table.data(), c->page_table.size() * sizeof(int32_t),
                             cudaMemcpyHostToDevice, stream));
  }
  c->prompt_lens.assign(prompt_lens, prompt_lens + batch);
  SJD_CUDA(cudaMemcpyAsync(c->ws + c->lay.prompt_lens, c->prompt_lens.data(), (size_t)batch * sizeof(int32_t),
                           cudaMemcpyHostToDevice, stream));
  c->window = sample->window;
  c->host_step = 0;
  c->last_stream = stream;
  c->prefilled = false;
  c->drop_graphs();
  if (c->use_tc) {
    // activation descriptors for the two row counts used: the step's window and the pre-fill chunk
    const int Ma = c->rows_alloc();
    const int nq = c->cfg.n_heads * c->cfg.head_dim;
    const int row_counts[2] = {batch * sample->window, batch * c->cfg.max_window};
    for (int i = 0; i < 2; ++i) {
      const int Mp = (row_counts[i] + 15) / 16 * 16;
      if (row_counts[i] > 1024 || c->xmaps.count(Mp)) continue;
      XMaps xm;
      const int box = gemm_tc_plan(row_counts[i]).slab_rows;
      const bool ok = make_tensor_map_bf16(&xm.h, c->ws + c->lay.xs_h, 2L * Ma, c->cfg.d_model, box) == SJD_OK &&
                      make_tensor_map_bf16(&xm.attn, c->ws + c->lay.xs_attn, 2L * Ma, nq, box) == SJD_OK &&
                      make_tensor_map_bf16(&xm.act, c->ws + c->lay.xs_act, 2L * Ma, c->cfg.ffn_hidden, box) == SJD_OK;
      if (ok) c->xmaps[Mp] = xm;
    }
  }
  const SeqState st = c->state();
  prefill_setup_kernel<<<batch, 128, 0, stream>>>(prompt, row_stride, st, c->at<uint32_t>(c->lay.step),
                                                  c->at<int32_t>(c->lay.counters), batch);
  SJD_CHECK_LAUNCH();
  // cache keys/values of c[0..P-1) in chunks of max_window rows per sequence
  const int rows = c->cfg.max_window;
  for (int c0 = 0; c0 < prompt_len - 1; c0 += rows) {
    prefill_inputs_kernel<<<batch, 64, 0, stream>>>(prompt, row_stride, st.prompt_lens, c0, rows, st.in_tok, st.in_pos);
    SJD_CHECK_LAUNCH();
    rc = forward(c, rows, nullptr, stream);
    if (rc != SJD_OK) return rc;
  }
  // first window: no rows to verify (w_eff = 0), the slide initialises every slot (Sec. 4.2) with the
  // initial-window step tag and bumps the step index to 0
  rc = run_verify(c, nullptr, stream);
  if (rc != SJD_OK) return rc;
  c->prefilled = true;
  return SJD_OK;
}

namespace {
// forward pass + verification of one step, enqueued on `stream`
int enqueue_step(sjd_ctx *c, const sjd_step_out *out, int cur, cudaStream_t stream) {
  int rc = forward(c, c->window, c->ws + c->lay.logits[cur], stream);
  if (rc != SJD_OK) return rc;
  c->tracer.begin(TC_VERIFY, stream);
  g_pdl = !c->tracer.on;
  rc = run_verify(c, out, stream);
  g_pdl = false;
  c->tracer.end(stream);
  return rc;
}

bool same_out(const sjd_step_out &a, const sjd_step_out *b) {
  sjd_step_out z;
  memset(&z, 0, sizeof(z));
  return memcmp(&a, b ? b : &z, sizeof(sjd_step_out)) == 0;
}
}  // namespace

extern "C" int sjd_step(sjd_ctx *c, const sjd_step_out *out, void *cuda_stream) {
  if (!c) return SJD_ERR_BAD_ARG;
  if (!c->prefilled) return SJD_ERR_STATE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  c->last_stream = stream;
  const int cur = (int)(c->host_step & 1u);
  if (c->graphs_enabled && c->use_tc && !c->tracer.on) {
    sjd_ctx::StepGraph &g = c->graphs[cur];
    if (g.exec && !(g.has_out && same_out(g.out, out))) {
      cudaGraphExecDestroy(g.exec);
      g.exec = nullptr;
    }
    if (!g.exec) {
      // capture on a private stream (the caller's may be the legacy default stream), replay on the caller's
      if (!c->capture_stream && cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking) != cudaSuccess)
        c->graphs_enabled = false;
      if (c->graphs_enabled) {
        const long long before = g_launch_count.load();
        cudaGraph_t graph = nullptr;
        bool ok = cudaStreamBeginCapture(c->capture_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
        if (ok) {
          const int rc = enqueue_step(c, out, cur, c->capture_stream);
          const cudaError_t e = cudaStreamEndCapture(c->capture_stream, &graph);
          ok = rc == SJD_OK && e == cudaSuccess && graph != nullptr;
        }
        const long long captured = g_launch_count.load() - before;   // kernels recorded, not run
        g_launch_count.store(before);
        if (ok) ok = cudaGraphInstantiate(&g.exec, graph, 0) == cudaSuccess;
        if (graph) cudaGraphDestroy(graph);
        if (ok) {
          memset(&g.out, 0, sizeof(g.out));
          if (out) g.out = *out;
          g.has_out = true;
          g.launches = captured;
        } else {
          g.exec = nullptr;
          c->graphs_enabled = false;   // fall back to direct launches for good
          cudaGetLastError();
        }
      }
    }
    if (g.exec) {
      SJD_CUDA(cudaGraphLaunch(g.exec, stream));
      g_launch_count.fetch_add(g.launches, std::memory_order_relaxed);
      c->host_step += 1;
      return SJD_OK;
    }
  }
  const int rc = enqueue_step(c, out, cur, stream);
  if (rc != SJD_OK) return rc;
  c->host_step += 1;
  return c->tracer.flush(stream);
}

extern "C" int sjd_get_window(sjd_ctx *c, const sjd_step_out *out, void *cuda_stream) {
  if (!c || !out) return SJD_ERR_BAD_ARG;
  if (!c->prefilled) return SJD_ERR_STATE;
  const int streams = c->sample.guidance != 0.0f ? 2 : 1;
  get_window_kernel<<<c->batch / streams, 64, 0, (cudaStream_t)cuda_stream>>>(c->state(), *out, c->window, streams);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

extern "C" int sjd_get_tokens(sjd_ctx *c, int32_t *tokens, int row_stride, int32_t *counts, void *cuda_stream) {
  if (!c || !tokens || row_stride < 1) return SJD_ERR_BAD_ARG;
  if (!c->prefilled) return SJD_ERR_STATE;
  if ((long)row_stride < (long)c->prompt_len + c->sample.n_generate) return SJD_ERR_CAPACITY;
  const int streams = c->sample.guidance != 0.0f ? 2 : 1;
  get_tokens_kernel<<<c->batch / streams, 256, 0, (cudaStream_t)cuda_stream>>>(c->state(), tokens, row_stride, counts, streams);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

extern "C" int sjd_peek_logits(sjd_ctx *c, void *dst, size_t bytes, void *cuda_stream) {
  if (!c || !dst) return SJD_ERR_BAD_ARG;
  if (!c->prefilled || c->host_step == 0) return SJD_ERR_STATE;
  const size_t need = (size_t)c->batch * c->window * c->cfg.vocab * esize(c->cfg.dtype);
  if (bytes < need) return SJD_ERR_CAPACITY;
  const int last = (int)((c->host_step - 1) & 1u);
  SJD_CUDA(cudaMemcpyAsync(dst, c->ws + c->lay.logits[last], need, cudaMemcpyDefault, (cudaStream_t)cuda_stream));
  return SJD_OK;
}

extern "C" int sjd_get_info(sjd_ctx *c, sjd_info *info) {
  if (!c || !info) return SJD_ERR_BAD_ARG;
  if (!c->prefilled) return SJD_ERR_STATE;
  const int M = c->batch * c->window;
  const bool tc = c->use_tc && c->all_tc && M <= 1024 && c->xmaps.count((M + 15) / 16 * 16) != 0;
  info->tensor_core_projections = tc ? 1 : 0;
  info->tensor_core_attention =
      (tc && c->kv_map_valid && attention_mma_supported(c->cfg.head_dim, c->window)) ? 1 : 0;
  info->step_graph = (c->graphs_enabled && c->use_tc) ? 1 : 0;
  info->rows_per_step = M;
  return SJD_OK;
}

extern "C" int sjd_last_device_status(sjd_ctx *c) {
  if (!c) return SJD_ERR_BAD_ARG;
  SJD_CUDA(cudaStreamSynchronize(c->last_stream));
  int32_t status = 0;
  SJD_CUDA(cudaMemcpy(&status, c->ws + c->lay.status, 4, cudaMemcpyDeviceToHost));
  return status == 0 ? SJD_OK : SJD_ERR_DEVICE_TIMEOUT;
}

extern "C" int sjd_trace(sjd_ctx *c, int enable) {
  if (!c) return SJD_ERR_BAD_ARG;
  c->tracer.on = enable != 0;
  c->tracer.used = 0;
  c->tracer.cls.clear();
  if (enable) {
    for (int i = 0; i < TC_COUNT; ++i) {
      c->tracer.ms[i] = 0;
      c->tracer.launches[i] = 0;
    }
    c->tracer.gemm_weight_bytes = 0;
  }
  return SJD_OK;
}

extern "C" int sjd_trace_read(sjd_ctx *c, double *ms, int64_t *launches, double *gemm_weight_bytes) {
  if (!c || !ms || !launches || !gemm_weight_bytes) return SJD_ERR_BAD_ARG;
  for (int i = 0; i < TC_COUNT; ++i) {
    ms[i] = c->tracer.ms[i];
    launches[i] = c->tracer.launches[i];
  }
  *gemm_weight_bytes = c->tracer.gemm_weight_bytes;
  return SJD_OK;
}

extern "C" void sjd_destroy(sjd_ctx *c) { delete c; }
