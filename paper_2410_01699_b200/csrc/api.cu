// C-ABI entry points that need no context: isolated verification, error strings.
#include <string.h>

#include "common.cuh"

namespace sjd {
thread_local int g_last_cuda_error = 0;
std::atomic<long long> g_launch_count{0};
thread_local bool g_pdl = false;

int check_sample_cfg(const sjd_sample_cfg *s, int vocab) {
  if (!s) return SJD_ERR_BAD_ARG;
  if (!(s->temperature > 0.0f) || s->top_k < 1 || s->window < 1) return SJD_ERR_BAD_ARG;
  if (s->window > 64) return SJD_ERR_CAPACITY;
  if (s->init < SJD_INIT_RANDOM || s->init > SJD_INIT_RESAMPLE_ABOVE) return SJD_ERR_BAD_ARG;
  if ((s->init == SJD_INIT_COPY_ABOVE || s->init == SJD_INIT_RESAMPLE_ABOVE) && s->grid_stride < 1) return SJD_ERR_BAD_ARG;
  if (s->seq_base < 0) return SJD_ERR_BAD_ARG;
  if (!(s->guidance == s->guidance) || s->guidance > 1e6f || s->guidance < -1e6f) return SJD_ERR_BAD_ARG;
  if (s->schedule < SJD_SCHEDULE_SJD || s->schedule > SJD_SCHEDULE_NO_REFINE) return SJD_ERR_BAD_ARG;
  (void)vocab;
  return SJD_OK;
}
}  // namespace sjd

using namespace sjd;

extern "C" size_t sjd_verify_workspace_bytes(int batch, int window) { return verify_scratch_bytes(batch, window); }

namespace sjd {
// Argument checks and parameter set-up shared by the two isolated-verification entry points;
// `scratch` holds verify_scratch_bytes(batch, window) bytes, 16-byte aligned.
int verify_isolated(int batch, int window, int vocab, int logits_dtype, const void *logits_cur, const void *logits_prev,
                    const int32_t *draft, const int32_t *q_kind, const int32_t *base_pos, const sjd_sample_cfg *sample,
                    uint32_t step, const sjd_step_out *out, void *scratch, cudaStream_t stream) {
  if (batch < 1 || window < 1 || vocab < 1 || !logits_cur || !draft || !sample || !out || !scratch)
    return SJD_ERR_BAD_ARG;
  if (!logits_prev && !q_kind) return SJD_ERR_BAD_ARG;  // rows of law SJD_Q_ROW need their logits
  if (logits_dtype != SJD_F32 && logits_dtype != SJD_BF16) return SJD_ERR_UNSUPPORTED;
  if (window > 64) return SJD_ERR_CAPACITY;
  if (!(sample->temperature > 0.0f) || sample->top_k < 1 || sample->seq_base < 0) return SJD_ERR_BAD_ARG;
  if (sample->guidance != 0.0f) return SJD_ERR_UNSUPPORTED;   // guidance pairs the streams of a context (sjd_step)
  if (sample->schedule < SJD_SCHEDULE_SJD || sample->schedule > SJD_SCHEDULE_NO_REFINE) return SJD_ERR_BAD_ARG;
  if (((uintptr_t)scratch & 15u) != 0) return SJD_ERR_BAD_ARG;

  const size_t rows = (size_t)batch * window;
  char *w = (char *)scratch;
  VerifyParams p;
  memset(&p, 0, sizeof(p));
  p.logits[0] = logits_cur;
  p.logits[1] = logits_prev ? logits_prev : logits_cur;
  p.stats[0] = (RowStats *)w;
  p.stats[1] = (RowStats *)(w + rows * sizeof(RowStats));
  p.row_out = (RowOut *)(w + 2 * rows * sizeof(RowStats));
  p.seq_counter = (int32_t *)(w + 2 * rows * sizeof(RowStats) + rows * sizeof(RowOut));
  p.done_counter = p.seq_counter + batch;
  // the ticket counters must start at zero whatever an earlier call left in the scratch
  SJD_CUDA(cudaMemsetAsync(p.seq_counter, 0, ((size_t)batch + 1) * sizeof(int32_t), stream));
  p.draft = draft;
  p.q_kind = q_kind;
  p.base_pos = base_pos;
  p.step = step;
  p.B = batch;
  p.W = window;
  p.V = vocab;
  p.temperature = sample->temperature;
  p.top_k = sample->top_k;
  p.seed_lo = (uint32_t)(sample->seed & 0xFFFFFFFFull);
  p.seed_hi = (uint32_t)(sample->seed >> 32);
  p.seq_base = (uint32_t)sample->seq_base;
  p.e2e = 0;
  p.schedule = sample->schedule;
  p.out = *out;
  return launch_verify(p, logits_dtype, stream);
}
}  // namespace sjd

extern "C" int sjd_verify(int batch, int window, int vocab, int logits_dtype, const void *logits_cur,
                          const void *logits_prev, const int32_t *draft, const int32_t *q_kind,
                          const int32_t *base_pos, const sjd_sample_cfg *sample, uint32_t step,
                          const sjd_step_out *out, void *ws, size_t ws_bytes, void *cuda_stream) {
  if (!ws) return SJD_ERR_BAD_ARG;
  if (batch >= 1 && window >= 1 && ws_bytes < verify_scratch_bytes(batch, window)) return SJD_ERR_CAPACITY;
  return verify_isolated(batch, window, vocab, logits_dtype, logits_cur, logits_prev, draft, q_kind, base_pos, sample,
                         step, out, ws, (cudaStream_t)cuda_stream);
}

extern "C" int sjd_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" int64_t sjd_launch_count(void) { return (int64_t)g_launch_count.load(); }

extern "C" const char *sjd_strerror(int status) {
  switch (status) {
    case SJD_OK: return "ok";
    case SJD_ERR_BAD_ARG: return "bad argument";
    case SJD_ERR_CAPACITY: return "capacity exceeded (batch, window, sequence, vocabulary or workspace)";
    case SJD_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case SJD_ERR_CUDA: return "CUDA runtime error (see sjd_last_cuda_error)";
    case SJD_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case SJD_ERR_STATE: return "call out of order";
    default: return "unknown status";
  }
}

// ---- the projection of Step 2 in isolation (tensor-core weight-streaming GEMM)
namespace {
inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
constexpr int kGemmSmsMax = 160;
}  // namespace

extern "C" size_t sjd_gemm_workspace_bytes(int M, int N, int K) {
  if (!gemm_tc_supported(M, N, K)) return 0;
  const int mp = (M + 15) / 16 * 16;
  const int splits = gemm_tc_splits(gemm_tc_plan(M), N / 128, K / 64, kGemmSmsMax);
  return 256 + up256((size_t)splits * M * N * 4) + up256((size_t)2 * mp * K * 2);
}

extern "C" int sjd_gemm(int M, int N, int K, const float *x, const void *w, float *out, int accumulate, void *ws,
                        size_t ws_bytes, void *cuda_stream) {
  if (M < 1 || N < 1 || K < 1 || !x || !w || !out || !ws) return SJD_ERR_BAD_ARG;
  if (!gemm_tc_supported(M, N, K)) return SJD_ERR_UNSUPPORTED;
  if (((uintptr_t)ws & 255u) != 0) return SJD_ERR_BAD_ARG;
  if (ws_bytes < sjd_gemm_workspace_bytes(M, N, K)) return SJD_ERR_CAPACITY;
  int dev = 0, cc_major = 0, sms = 0;
  SJD_CUDA(cudaGetDevice(&dev));
  SJD_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev));
  SJD_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (cc_major != 10) return SJD_ERR_UNSUPPORTED;
  sms = sms < kGemmSmsMax ? sms : kGemmSmsMax;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const int mp = (M + 15) / 16 * 16;
  const GemmTcPlan plan = gemm_tc_plan(M);
  const int splits = gemm_tc_splits(plan, N / 128, K / 64, sms);
  const int splits_max = gemm_tc_splits(plan, N / 128, K / 64, kGemmSmsMax);
  char *p = (char *)ws;
  int *status = (int *)p;
  float *planes = (float *)(p + 256);
  __nv_bfloat16 *xs = (__nv_bfloat16 *)(p + 256 + up256((size_t)splits_max * M * N * 4));
  SJD_CUDA(cudaMemsetAsync(p, 0, 256, stream));
  SJD_CUDA(cudaMemsetAsync(xs, 0, (size_t)2 * mp * K * 2, stream));
  int rc = launch_split_hilo(x, HiLoOut{xs, (size_t)mp * K}, (size_t)M * K, stream);
  if (rc != SJD_OK) return rc;
  TensorMap wm, xm;
  rc = make_tensor_map_bf16(&wm, w, N, K, 128);
  if (rc != SJD_OK) return rc;
  rc = make_tensor_map_bf16(&xm, xs, 2L * mp, K, plan.slab_rows);
  if (rc != SJD_OK) return rc;
  GemmTcCall g;
  memset(&g, 0, sizeof(g));
  g.w_map[0] = g.w_map[1] = g.w_map[2] = &wm;
  g.n_mats = 1;
  g.n_out[0] = N;
  g.x_map = &xm;
  g.x_lo_row = mp;
  g.M = M;
  g.K = K;
  g.splits = splits;
  g.out = planes;
  g.plane_stride = (size_t)M * N;
  g.ldc = N;
  g.store_bf16 = 0;
  g.status = status;
  g.n_sms = sms;
  rc = launch_gemm_tc(g, stream);
  if (rc != SJD_OK) return rc;
  return launch_sum_planes(planes, (size_t)M * N, splits, out, (size_t)M * N, accumulate, stream);
}

#ifdef SJD_TIMELINE
// timeline builds only: allocate / read the device timeline (see common.cuh)
namespace sjd {
void timeline_set_fused(TimelineBuf *);
void timeline_set_gemm(TimelineBuf *);
void timeline_set_attn(TimelineBuf *);
void timeline_set_combine(TimelineBuf *);
void timeline_set_verify(TimelineBuf *);
}  // namespace sjd
extern "C" int sjd_timeline_attach(void *device_buf) {
  TimelineBuf *b = (TimelineBuf *)device_buf;
  timeline_set_fused(b);
  timeline_set_gemm(b);
  timeline_set_attn(b);
  timeline_set_combine(b);
  timeline_set_verify(b);
  return SJD_OK;
}
extern "C" size_t sjd_timeline_bytes(void) { return sizeof(TimelineBuf); }
#endif

// ---- the window attention of Step 2 in isolation (tensor-core split-KV kernel, bf16 cache)
namespace sjd {
int attention_splits(int n_heads, int batch);   // engine.cu
}
namespace {
int attn_splits(int n_heads, int batch) { return sjd::attention_splits(n_heads, batch); }
}  // namespace

extern "C" size_t sjd_attention_workspace_bytes(int batch, int window, int n_heads, int head_dim) {
  if (batch < 1 || window < 1 || n_heads < 1 || !attention_mma_supported(head_dim, window)) return 0;
  return 256 + (size_t)batch * window * n_heads * attn_splits(n_heads, batch) * (head_dim + 2) * 4;
}

extern "C" int sjd_attention(int batch, int window, int n_heads, int n_kv_heads, int head_dim, int max_seq, const float *q,
                             const void *kv_cache, const int32_t *in_pos, float *out, void *ws, size_t ws_bytes,
                             void *cuda_stream) {
  if (batch < 1 || window < 1 || n_heads < 1 || n_kv_heads < 1 || max_seq < 1 || !q || !kv_cache || !in_pos || !out || !ws)
    return SJD_ERR_BAD_ARG;
  if (n_heads % n_kv_heads != 0) return SJD_ERR_BAD_ARG;
  if (!attention_mma_supported(head_dim, window)) return SJD_ERR_UNSUPPORTED;
  if (((uintptr_t)ws & 255u) != 0) return SJD_ERR_BAD_ARG;
  if (ws_bytes < sjd_attention_workspace_bytes(batch, window, n_heads, head_dim)) return SJD_ERR_CAPACITY;
  int dev = 0, cc_major = 0;
  SJD_CUDA(cudaGetDevice(&dev));
  SJD_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev));
  if (cc_major < 9) return SJD_ERR_UNSUPPORTED;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  int *status = (int *)ws;
  float *partial = (float *)((char *)ws + 256);
  SJD_CUDA(cudaMemsetAsync(status, 0, 256, stream));
  TensorMap kv_map;
  int rc = make_kv_tensor_map(&kv_map, kv_cache, (long)batch * 2 * n_kv_heads, max_seq, head_dim);
  if (rc != SJD_OK) return rc;
  const int splits = attn_splits(n_heads, batch);
  const int M = batch * window;
  const KvLayout contiguous = {const_cast<void *>(kv_cache), n_kv_heads, max_seq, head_dim, nullptr, 0, 0, 1};
  rc = launch_attention_mma(kv_map, 0, contiguous, q, in_pos, partial, out, HiLoOut{nullptr, 0}, status, M, window,
                            n_heads, n_kv_heads, head_dim, splits, stream);
  if (rc != SJD_OK || splits == 1) return rc;
  return launch_attention_combine(partial, in_pos, out, M, n_heads, head_dim, splits, stream, HiLoOut{nullptr, 0});
}
