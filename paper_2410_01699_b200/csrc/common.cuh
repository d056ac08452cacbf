// Shared declarations of the SJD CUDA library: status helpers, Philox4x32-10,
// small warp/block primitives, and the launch prototypes of every kernel file.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <atomic>

#include "sjd.h"

namespace sjd {

extern thread_local int g_last_cuda_error;
extern std::atomic<long long> g_launch_count;  // kernels launched by this library in this process

#define SJD_CUDA(expr)                          \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) {                   \
      ::sjd::g_last_cuda_error = (int)e__;      \
      return SJD_ERR_CUDA;                      \
    }                                           \
  } while (0)

#define SJD_CHECK_LAUNCH()                                              \
  do {                                                                  \
    ::sjd::g_launch_count.fetch_add(1, std::memory_order_relaxed);      \
    SJD_CUDA(cudaGetLastError());                                       \
  } while (0)

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  While g_pdl is set, kernels are launched with the
// programmatic-stream-serialization attribute: a kernel may start (set up, prefetch data that does
// not depend on its predecessor) before the previous kernel in the stream has finished.  Every such
// kernel calls pdl_trigger() early and pdl_wait() before it touches anything an earlier kernel writes
// or still reads; outside such launches both are no-ops.
// ---------------------------------------------------------------------------------------------
extern thread_local bool g_pdl;

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 Args &&...args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = g_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// ---------------------------------------------------------------------------------------------
// Optional device timeline (build with -DSJD_TIMELINE): block 0 of every kernel of the tensor-core
// pipeline stamps %globaltimer at entry, after its grid-dependency wait and at its end into one
// buffer, which shows how the overlapped launches really interleave.  Off in normal builds.
// ---------------------------------------------------------------------------------------------
#ifdef SJD_TIMELINE
struct TimelineBuf {
  unsigned int n;
  unsigned int pad;
  struct Rec { unsigned long long t; int tag; int phase; } rec[1 << 16];
};
#define SJD_TIMELINE_TU(name)                                                                       \
  static __device__ TimelineBuf *g_tl_buf;                                                         \
  void timeline_set_##name(TimelineBuf *p) { cudaMemcpyToSymbol(g_tl_buf, &p, sizeof(p)); }        \
  __device__ __forceinline__ void tl_mark(int tag, int phase) {                                    \
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && g_tl_buf) {                      \
      unsigned long long t;                                                                        \
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));                                         \
      const unsigned int i = atomicAdd(&g_tl_buf->n, 1u);                                          \
      if (i < (1u << 16)) {                                                                        \
        g_tl_buf->rec[i].t = t;                                                                    \
        g_tl_buf->rec[i].tag = tag;                                                                \
        g_tl_buf->rec[i].phase = phase;                                                            \
      }                                                                                            \
    }                                                                                              \
  }
#define SJD_TL(tag, phase, cond) do { if (cond) tl_mark(tag, phase); } while (0)
#else
#define SJD_TIMELINE_TU(name)
#define SJD_TL(tag, phase, cond) do { } while (0)
#endif
enum TimelineTag { TL_EMBED = 0, TL_RESID = 1, TL_GEMM = 2, TL_QKV = 3, TL_ATTN = 4, TL_COMBINE = 5, TL_SWIGLU = 6, TL_VERIFY = 7 };

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): 128-bit counter, 64-bit key, ten rounds of
// two 32x32->64 multiplies with a Weyl key schedule.
// ---------------------------------------------------------------------------------------------
struct Philox4 {
  uint32_t w[4];
};

__host__ __device__ inline Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)M0 * c0;
    const uint64_t p1 = (uint64_t)M1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
    k0 += W0;
    k1 += W1;
  }
  Philox4 out;
  out.w[0] = c0; out.w[1] = c1; out.w[2] = c2; out.w[3] = c3;
  return out;
}

constexpr uint32_t kStreamVerify = 0u;         // words 0,1,2: accept / residual / re-draft uniforms
constexpr uint32_t kStreamInit = 1u;           // word 0: random token of a fresh slot
constexpr uint32_t kStepInitialWindow = 0xFFFFFFFFu;

__host__ __device__ inline float u24(uint32_t word) { return (float)(word >> 8) * (1.0f / 16777216.0f); }

// ---------------------------------------------------------------------------------------------
// warp helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---------------------------------------------------------------------------------------------
// Per-row verification records (device scratch)
// ---------------------------------------------------------------------------------------------
struct RowStats {      // what is needed to evaluate p(x) of a stored logits row at any x
  uint32_t tau_key;    // order-preserving key of the top-k threshold (entries with key >= it are kept)
  float xmax;          // largest logit of the row (-inf for a row with no finite entry)
  float z;             // sum over kept entries of exp((x - xmax) / T)
  uint32_t flags;      // SJD_FLAG_NONFINITE
};

struct RowOut {
  float p_draft;       // p_k[d_k]
  float q_draft;       // q_k[d_k]
  float thr;           // min(1, p/q)
  int32_t accept;      // u_acc < thr
  int32_t redraft_tok; // d'_k ~ p_k (Eq. 3)
  float redraft_p;     // p_k[d'_k]: the q the re-drawn token carries
  int32_t resample_tok;// t_k ~ norm(max(0, p_k - q_k)) if this row rejected (Eq. 2), else -1
  uint32_t flags;
};

// Decoding state of a context, all device-resident (see engine.cu)
struct SeqState {
  int32_t *committed;   // [B][max_seq]
  int32_t *n;           // [B] committed count
  int32_t *w_eff;       // [B] drafts in the current window
  int32_t *draft;       // [B][W]
  int32_t *q_kind;      // [B][W]
  int32_t *q_row;       // [B][W] row of the previous logits buffer that produced the draft
  float *q_draft;       // [B][W]
  int32_t *in_tok;      // [B][W] model inputs of the next step
  int32_t *in_pos;      // [B][W] their absolute positions, -1 = inactive row
  int32_t max_seq;
  const int32_t *prompt_lens;   // [B] prompt length of every sequence (ragged batches)
  int32_t n_generate;
  int32_t init;
  int32_t grid_stride;
};

struct VerifyParams {
  const void *logits[2];   // [B][W][V]; index (step & 1) is this iteration's buffer when use_step_ptr
  RowStats *stats[2];      // [B][W] alongside
  const int32_t *draft;    // [B][W]
  const int32_t *q_kind;   // [B][W] or null (all ROW)
  const int32_t *q_row;    // [B][W] or null (slot k was produced by row k)
  int prev_stats_valid;    // stats of the previous buffer are already there (end-to-end mode)
  RowOut *row_out;         // [B][W]
  int32_t *seq_counter;    // [B] zero on entry, zero on exit
  int32_t *done_counter;   // [1] zero on entry, zero on exit
  const int32_t *w_eff;    // [B] or null (= W)
  const int32_t *base_pos; // [B] absolute position of slot 0, or null (0)
  uint32_t *step_ptr;      // device step index (end-to-end), bumped by the last block
  uint32_t step;           // used when step_ptr == null
  int B, W, V;
  int staged;              // row fits the dynamic shared buffer
  int defer_residual;      // register route: rejected rows leave the Eq. 2 draw to the sequence's last block
  int fast;                // bf16 rows, 16-byte aligned, V % 8 == 0, V / 8 <= 8 * blockDim.x: a block may keep a row in registers
  float temperature;
  int top_k;
  uint32_t seed_lo, seed_hi;
  uint32_t seq_base;       // global id of sequence 0 (batch sharded across GPUs)
  int e2e;                 // 1: update SeqState (window slide); 0: isolated verification
  // Classifier-free guidance (paired != 0): sequences 2i and 2i + 1 of the forward pass are the conditional
  // and the unconditional stream of image i; B counts images; every logits row is read as
  // l_u + guidance * (l_c - l_u) rounded to the storage dtype, and the slide writes both streams' state.
  int paired;
  float guidance;
  int schedule;            // sjd_schedule_kind
  // Sec. 4.2 (d): ring of retained rows [image][ring_len][V] (storage dtype, as verification saw them) with
  // their statistics; slot = position % ring_len.  n_prev / w_prev [image]: fixed tokens and window size
  // before the slide of the last verification (what the retaining copy goes by).  ring == null: not in use.
  void *ring;
  RowStats *ring_stats;
  int ring_len;
  int32_t *n_prev, *w_prev;
  SeqState st;
  sjd_step_out out;
};

// kernel launchers (each returns an sjd_status)
int launch_verify(const VerifyParams &p, int dtype, cudaStream_t stream);
// after a verification: copy the rows of the window it verified (and their statistics) into the ring
int launch_retain_rows(const VerifyParams &p, int dtype, cudaStream_t stream);
size_t verify_scratch_bytes(int batch, int window);
int check_sample_cfg(const sjd_sample_cfg *s, int vocab);

// ---- model forward (model_kernels.cu, attention.cu); `dtype` selects float / bf16 storage
enum GemmEpilogue { EPI_STORE_F32 = 0, EPI_STORE_T = 1, EPI_ADD_F32 = 2 };

// C[M][N] (epilogue) = A[M][K] * Wt[N][K]^T, fp32 accumulation.  A is fp32, Wt is of `dtype`;
// C is fp32 (EPI_STORE_F32, EPI_ADD_F32: C += product) or `dtype` (EPI_STORE_T).  lda/ldc in elements.
int launch_gemm_simt(int dtype, const void *A, int lda, const void *Wt, void *C, int ldc, int M, int N, int K,
                     int epilogue, cudaStream_t stream);
// ---- tensor-core weight-streaming GEMM (gemm_tc.cu), bf16 weights
struct alignas(64) TensorMap {   // an encoded TMA descriptor (same size and alignment as the driver's)
  unsigned char bytes[128];
};
// bf16 row-major [rows][cols] matrix cut into boxes of box_rows x 64 columns, 128-byte swizzle
int make_tensor_map_bf16(TensorMap *out, const void *base, long rows, long cols, int box_rows);
bool gemm_tc_supported(int M, int N, int K);
// Shape of a launch of M rows: token slabs and rows per slab (a multiple of 16: the box height of the
// activation tensor map).
struct GemmTcPlan {
  int n_slabs, slab_rows;
};
GemmTcPlan gemm_tc_plan(int M);
int gemm_tc_splits(const GemmTcPlan &pl, int tiles, int k_blocks, int n_sms);   // tiles: 128-row weight tiles of the launch
// One launch over up to three weight matrices that share the activation operand X (two bf16 planes:
// hi at row 0, lo at row x_lo_row of x_map, each [rows][K]).  Matrix j has n_out[j] rows and writes
// output columns [col_off[j], col_off[j] + n_out[j]).  splits > 1 (or store_bf16 == 0): fp32 planes
// out[s][m][ldc], plane_stride elements apart, one per K split; store_bf16 (splits == 1): bf16 out[m][ldc].
struct GemmTcCall {
  const TensorMap *w_map[3];
  int n_mats;
  int n_out[3], col_off[3];
  const TensorMap *x_map;
  int x_lo_row;
  int M, K;
  int splits;
  void *out;
  size_t plane_stride;
  int ldc;
  int store_bf16;
  int *status;
  const float *ss_part;   // optional per-row RMS scale applied in the epilogue (see RowScale); null: none
  int n_part;
  float inv_d, eps;
  int n_sms;
  // weight rows per tile (0: 128).  Fewer rows make more, smaller tiles (their tensor maps must have been
  // made with that box height); the unused rows of the 128-row MMA cost nothing on a bandwidth-bound launch.
  int tile_rows;
  // gate|up mode (act_hi != null): n_mats == 2, matrices gate and up of n_out[0] rows each, tile_rows <= 64,
  // splits == 1; instead of planes the launch stores silu(gate) * up (both under the row scale) as bf16
  // hi/lo planes [M][n_out[0]], the lo plane act_lo_off elements after the hi plane.
  __nv_bfloat16 *act_hi;
  size_t act_lo_off;
};
int launch_gemm_tc(const GemmTcCall &g, cudaStream_t stream);
int launch_sum_planes(const float *planes, size_t plane_stride, int splits, float *out, size_t total, int accumulate,
                      cudaStream_t stream);
// The fp32 partial planes a GEMM launch left: value(m, col) = sum_s base[s * plane_stride + m * ld + col]
struct PlaneSet {
  const float *base;
  size_t plane_stride;
  int ld;
  int splits;     // 0: no planes (nothing to add)
};
// Optional second output of the activation-producing kernels: the value split as bf16 hi + bf16 lo
// (hi = bf16(v), lo = bf16(v - hi)), planes `lo_offset` elements apart, row stride = row length.
struct HiLoOut {
  __nv_bfloat16 *base;   // null: not wanted
  size_t lo_offset;
};

int launch_split_hilo(const float *x, HiLoOut o, size_t total, cudaStream_t stream);
// consumer kernels of the tensor-core path (fused_kernels.cu)
struct KvLayout;
// partial sums of squares of the residual rows: scale(m) = 1/sqrt(sum_j ss_part[m][j] * inv_d + eps)
struct RowScale {
  const float *ss_part;   // [M][n_part]; null: scale 1
  int n_part;
  float inv_d, eps;
};
int resid_gain_parts(int d);
int launch_resid_gain(int dtype, float *x, PlaneSet ps, const void *gain, HiLoOut h, float *ss_part, int M, int d,
                      cudaStream_t stream);
int launch_swiglu_finish(PlaneSet ps, RowScale rs, HiLoOut act, int M, int F, cudaStream_t stream);

// x[m][:] = tok_emb[tok[m]][:]  (fp32 residual stream)
int launch_embed(int dtype, const void *tok_emb, const int32_t *tok, float *x, int M, int d, int vocab,
                 cudaStream_t stream);
// h[m][:] = x[m][:] * gain[:] / sqrt(mean(x[m]^2) + eps)  (gain of `dtype`)
int launch_rmsnorm(int dtype, const float *x, const void *gain, float *h, int M, int d, float eps, cudaStream_t stream,
                   HiLoOut hilo = HiLoOut{nullptr, 0});
// Rotate q and k by their absolute position (pairs i, i + hd/2), store q as fp32 [M][H*hd],
// append k and v to the cache row in_pos[m] of sequence m / rows_per_seq.  Rows with in_pos < 0 are skipped.
// Cache of one layer.  Contiguous: base is this layer's [B][2][KVh][max_seq][hd].  Paged (page_table != null): base is
// the pool [page][layer][2][KVh][KV_PAGE][hd] shared by all layers, and logical page i of sequence b (positions
// i * KV_PAGE .. i * KV_PAGE + KV_PAGE - 1) lives in physical page page_table[b * pages_per_seq + i].
constexpr int KV_PAGE = 64;
struct KvLayout {
  void *base;
  int n_kv_heads, max_seq, head_dim;
  const int32_t *page_table;
  int pages_per_seq, layer, n_layers;
};
// element offset of the cache row (sequence b, which = 0 keys / 1 values, kv head kh, position pos)
__device__ __forceinline__ size_t kv_row_offset(const KvLayout &kv, int b, int which, int kh, int pos) {
  if (kv.page_table == nullptr)
    return (((size_t)(b * 2 + which) * kv.n_kv_heads + kh) * kv.max_seq + pos) * kv.head_dim;
  const int page = kv.page_table[b * kv.pages_per_seq + pos / KV_PAGE];
  return (((((size_t)page * kv.n_layers + kv.layer) * 2 + which) * kv.n_kv_heads + kh) * KV_PAGE + pos % KV_PAGE) *
         kv.head_dim;
}
// QK-norm variant: every head of q and of k is RMS-normalised over its head_dim entries (gains of `dtype`,
// length head_dim) before the rotary step; null gains: the plain model.
struct QkNorm {
  const void *q_gain, *k_gain;
  float eps;
};
int launch_rope_append(int dtype, const float *qkv, const int32_t *in_pos, const float2 *rope_table, float *q,
                       KvLayout kv, int M, int rows_per_seq, int n_heads, QkNorm qkn, cudaStream_t stream);
int launch_qkv_finish(int dtype, PlaneSet ps, RowScale rs, const int32_t *in_pos, const float2 *rope_table, float *q,
                      KvLayout kv, int M, int rows_per_seq, int n_heads, QkNorm qkn, cudaStream_t stream);
// act[m][f] = silu(gu[m][f]) * gu[m][F + f]
int launch_swiglu(const float *gu, float *act, int M, int F, cudaStream_t stream, HiLoOut hilo = HiLoOut{nullptr, 0});
// Window-causal attention: query row m (sequence m / rows_per_seq, position in_pos[m]) attends cache rows
// 0 .. in_pos[m].  q, out: fp32 [M][H*hd]; cache of `dtype`.  partial: fp32 scratch [M][H][splits][hd + 2].
int launch_attention(int dtype, const float *q, KvLayout kv, const int32_t *in_pos, float *out, float *partial,
                     int M, int rows_per_seq, int n_heads, int splits, cudaStream_t stream,
                     HiLoOut hilo = HiLoOut{nullptr, 0});
// merge of the split-KV partials only (used after launch_attention_mma)
int launch_attention_combine(const float *partial, const int32_t *in_pos, float *out, int M, int n_heads, int head_dim,
                             int splits, cudaStream_t stream, HiLoOut hilo);
// tensor-core split-KV attention for bf16 caches (attention_mma.cu)
int make_kv_tensor_map(TensorMap *out, const void *base, long planes, long max_seq, int head_dim);
bool attention_mma_supported(int head_dim, int rows_per_seq);
// plane0: first plane of this layer in the contiguous map [planes][max_seq][hd]; with kv.page_table set the map is
// the pool's [planes][KV_PAGE][hd] and the plane of a tile comes from the page table.
int launch_attention_mma(const TensorMap &kv_map, int plane0, KvLayout kv, const float *q, const int32_t *in_pos, float *partial,
                         float *out, HiLoOut hilo, int *status, int M, int rows_per_seq, int n_heads, int n_kv_heads,
                         int head_dim, int splits, cudaStream_t stream);

}  // namespace sjd
