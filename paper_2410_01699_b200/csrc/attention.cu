// Window-causal attention of the W window queries over the cached prefix plus the in-window causal
// block (Sec. 3.2 / Sec. 4.1 Step 2: one forward pass over the window under a causal mask), as split-KV
// flash decoding: every block owns one (sequence, head, key range), keeps an online softmax per query
// and writes an unnormalised partial; a second kernel merges the partials.  Generic FMA version that
// serves fp32 and bf16 storage with fp32 arithmetic.
#include <float.h>

#include "common.cuh"

namespace sjd {
SJD_TIMELINE_TU(combine)
namespace {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

constexpr int TK = 32;        // keys per tile (one per lane)
constexpr int NWARPS = 8;
constexpr int MAXQ = 8;       // queries per warp: window <= 64
constexpr int MAXD = 4;       // head dims per lane: head_dim <= 128

template <typename T>
__global__ void __launch_bounds__(NWARPS * 32) attention_partial_kernel(
    const float *__restrict__ q, KvLayout kv, const int32_t *__restrict__ in_pos, float *__restrict__ partial,
    int rows_per_seq, int n_heads, int splits) {
  extern __shared__ float smem[];
  const int hd = kv.head_dim;
  const int W = rows_per_seq;
  float *Qs = smem;                       // [W][hd]
  float *Ks = Qs + W * hd;                // [TK][hd + 1]
  float *Vs = Ks + TK * (hd + 1);         // [TK][hd]
  float *Ss = Vs + TK * hd;               // [W][TK]
  __shared__ int s_pos[64];
  __shared__ int s_len;

  const int h = blockIdx.x, b = blockIdx.y, s = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kvh = h / (n_heads / kv.n_kv_heads);
  const int m0 = b * W;

  if (tid < 64) s_pos[tid] = tid < W ? in_pos[m0 + tid] : -1;
  __syncthreads();
  if (tid == 0) {
    int len = 0;
    for (int i = 0; i < W; ++i) len = max(len, s_pos[i] + 1);
    s_len = len;
  }
  for (int i = tid; i < W * hd; i += blockDim.x) {
    const int qi = i / hd, d = i % hd;
    Qs[i] = q[((size_t)(m0 + qi) * n_heads + h) * hd + d];
  }
  __syncthreads();
  const int len = s_len;
  int chunk = (len + splits - 1) / splits;
  chunk = (chunk + TK - 1) / TK * TK;
  const int k_begin = s * chunk;
  const int k_end = min(len, k_begin + chunk);

  static_assert(KV_PAGE % TK == 0, "a key tile must lie inside one cache page");
  const T *cache = reinterpret_cast<const T *>(kv.base);
  const float scale = rsqrtf((float)hd);

  float m_run[MAXQ], l_run[MAXQ], o[MAXQ][MAXD];
#pragma unroll
  for (int i = 0; i < MAXQ; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.0f;
#pragma unroll
    for (int j = 0; j < MAXD; ++j) o[i][j] = 0.0f;
  }

  for (int t0 = k_begin; t0 < k_end; t0 += TK) {
    const int nk = min(TK, k_end - t0);
    const T *kbase = cache + kv_row_offset(kv, b, 0, kvh, t0);   // the tile's rows are contiguous
    const T *vbase = cache + kv_row_offset(kv, b, 1, kvh, t0);
    for (int i = tid; i < TK * hd; i += blockDim.x) {
      const int r = i / hd, d = i % hd;
      float kx = 0.0f, vx = 0.0f;
      if (r < nk) {
        kx = to_f<T>(kbase[(size_t)r * hd + d]);
        vx = to_f<T>(vbase[(size_t)r * hd + d]);
      }
      Ks[r * (hd + 1) + d] = kx;
      Vs[r * hd + d] = vx;
    }
    __syncthreads();
    // scores: lane = key, this warp's queries
    float sc[MAXQ];
#pragma unroll
    for (int i = 0; i < MAXQ; ++i) sc[i] = 0.0f;
    for (int d = 0; d < hd; ++d) {
      const float kx = Ks[lane * (hd + 1) + d];
#pragma unroll
      for (int i = 0; i < MAXQ; ++i) {
        const int qi = warp + i * NWARPS;
        if (qi < W) sc[i] = fmaf(Qs[qi * hd + d], kx, sc[i]);
      }
    }
    const int key = t0 + lane;
#pragma unroll
    for (int i = 0; i < MAXQ; ++i) {
      const int qi = warp + i * NWARPS;
      if (qi >= W) continue;
      const bool visible = lane < nk && key <= s_pos[qi];
      const float sv = visible ? sc[i] * scale : -INFINITY;
      const float tmax = warp_max(sv);
      const float m_new = fmaxf(m_run[i], tmax);
      float pexp = 0.0f, alpha = 1.0f;
      if (m_new > -INFINITY) {
        pexp = visible ? expf(sv - m_new) : 0.0f;
        alpha = m_run[i] > -INFINITY ? expf(m_run[i] - m_new) : 0.0f;
      }
      const float psum = warp_sum(pexp);
      l_run[i] = l_run[i] * alpha + psum;
      m_run[i] = m_new;
      Ss[qi * TK + lane] = pexp;
#pragma unroll
      for (int j = 0; j < MAXD; ++j) o[i][j] *= alpha;
    }
    __syncwarp();
    // P V: lane = head dims lane, lane+32, ...
#pragma unroll
    for (int i = 0; i < MAXQ; ++i) {
      const int qi = warp + i * NWARPS;
      if (qi >= W) continue;
      for (int kk = 0; kk < nk; ++kk) {
        const float pv = Ss[qi * TK + kk];
#pragma unroll
        for (int j = 0; j < MAXD; ++j) {
          const int d = lane + 32 * j;
          if (d < hd) o[i][j] = fmaf(pv, Vs[kk * hd + d], o[i][j]);
        }
      }
    }
    __syncthreads();
  }

  // partial record per (row, head, split): [m, l, o[hd]]
#pragma unroll
  for (int i = 0; i < MAXQ; ++i) {
    const int qi = warp + i * NWARPS;
    if (qi >= W) continue;
    float *dst = partial + (((size_t)(m0 + qi) * n_heads + h) * splits + s) * (hd + 2);
    if (lane == 0) {
      dst[0] = m_run[i];
      dst[1] = l_run[i];
    }
#pragma unroll
    for (int j = 0; j < MAXD; ++j) {
      const int d = lane + 32 * j;
      if (d < hd) dst[2 + d] = o[i][j];
    }
  }
}

__global__ void attention_combine_kernel(const float *__restrict__ partial, const int32_t *__restrict__ in_pos,
                                         float *__restrict__ out, int n_heads, int hd, int splits, HiLoOut hilo) {
  pdl_trigger();
  SJD_TL(TL_COMBINE, 0, threadIdx.x == 0);
  pdl_wait();
  SJD_TL(TL_COMBINE, 1, threadIdx.x == 0);
  const int m = blockIdx.x, h = blockIdx.y;
  const float *src = partial + ((size_t)m * n_heads + h) * splits * (hd + 2);
  const size_t base = ((size_t)m * n_heads + h) * hd;
  float *dst = out + base;
  constexpr int NS = 8;
  if (splits <= NS && hd <= (int)blockDim.x) {
    // Few key ranges (the usual case): every thread fetches the row's position, all record heads and its own
    // entry of every record at once, so the kernel costs one memory round trip instead of three in a row.
    // Same arithmetic, in the same order, as the general path below.
    const int d = threadIdx.x;
    const int pos = in_pos[m];
    float mm[NS], ll[NS], vv[NS];
#pragma unroll
    for (int s = 0; s < NS; ++s) {
      const bool on = s < splits;
      mm[s] = on ? src[(size_t)s * (hd + 2)] : -INFINITY;
      ll[s] = on ? src[(size_t)s * (hd + 2) + 1] : 0.0f;
      vv[s] = on && d < hd ? src[(size_t)s * (hd + 2) + 2 + d] : 0.0f;
    }
    if (d >= hd) return;
    float v = 0.0f;
    if (pos >= 0) {
      float gmax = -INFINITY;
#pragma unroll
      for (int s = 0; s < NS; ++s) gmax = fmaxf(gmax, mm[s]);
      float denom = 0.0f, acc = 0.0f;
#pragma unroll
      for (int s = 0; s < NS; ++s)
        if (s < splits && mm[s] > -INFINITY) denom += ll[s] * expf(mm[s] - gmax);
#pragma unroll
      for (int s = 0; s < NS; ++s)
        if (s < splits) acc += vv[s] * (mm[s] > -INFINITY ? expf(mm[s] - gmax) : 0.0f);
      v = denom > 0.0f ? acc / denom : 0.0f;
    }
    dst[d] = v;
    if (hilo.base) {
      const __nv_bfloat16 hi = __float2bfloat16_rn(v);
      hilo.base[base + d] = hi;
      hilo.base[hilo.lo_offset + base + d] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
    return;
  }
  if (in_pos[m] < 0) {
    for (int d = threadIdx.x; d < hd; d += blockDim.x) {
      dst[d] = 0.0f;
      if (hilo.base) {
        hilo.base[base + d] = __float2bfloat16_rn(0.0f);
        hilo.base[hilo.lo_offset + base + d] = __float2bfloat16_rn(0.0f);
      }
    }
    return;
  }
  // heads of the records once (one thread per key range), then the weights from shared memory: the
  // loads over the records below do not wait on one another
  __shared__ float s_m[64], s_l[64], s_w[64];
  const int ns = splits < 64 ? splits : 64;
  if ((int)threadIdx.x < ns) {
    s_m[threadIdx.x] = src[(size_t)threadIdx.x * (hd + 2)];
    s_l[threadIdx.x] = src[(size_t)threadIdx.x * (hd + 2) + 1];
  }
  __syncthreads();
  float gmax = -INFINITY;
  for (int s = 0; s < ns; ++s) gmax = fmaxf(gmax, s_m[s]);
  float denom = 0.0f;
  for (int s = 0; s < ns; ++s)
    if (s_m[s] > -INFINITY) denom += s_l[s] * expf(s_m[s] - gmax);
  if ((int)threadIdx.x < ns) s_w[threadIdx.x] = s_m[threadIdx.x] > -INFINITY ? expf(s_m[threadIdx.x] - gmax) : 0.0f;
  __syncthreads();
  for (int d = threadIdx.x; d < hd; d += blockDim.x) {
    float acc = 0.0f;
#pragma unroll 4
    for (int s = 0; s < ns; ++s) acc += src[(size_t)s * (hd + 2) + 2 + d] * s_w[s];
    const float v = denom > 0.0f ? acc / denom : 0.0f;
    dst[d] = v;
    if (hilo.base) {
      const __nv_bfloat16 hi = __float2bfloat16_rn(v);
      hilo.base[base + d] = hi;
      hilo.base[hilo.lo_offset + base + d] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
  }
}

template <typename T>
int attention_t(const float *q, KvLayout kv, const int32_t *in_pos, float *out, float *partial, int M, int rows_per_seq,
                int n_heads, int splits, cudaStream_t stream, HiLoOut hilo) {
  const int hd = kv.head_dim, W = rows_per_seq;
  if (W > NWARPS * MAXQ || hd > 32 * MAXD || M % W != 0) return SJD_ERR_UNSUPPORTED;
  const size_t smem = sizeof(float) * ((size_t)W * hd + TK * (hd + 1) + TK * hd + (size_t)W * TK);
  if (smem > 48 * 1024)
    SJD_CUDA(cudaFuncSetAttribute(attention_partial_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid(n_heads, M / W, splits);
  attention_partial_kernel<T><<<grid, NWARPS * 32, smem, stream>>>(q, kv, in_pos, partial,
                                                                  W, n_heads, splits);
  SJD_CHECK_LAUNCH();
  attention_combine_kernel<<<dim3(M, n_heads), 128, 0, stream>>>(partial, in_pos, out, n_heads, hd, splits, hilo);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

}  // namespace

int launch_attention_combine(const float *partial, const int32_t *in_pos, float *out, int M, int n_heads, int head_dim,
                             int splits, cudaStream_t stream, HiLoOut hilo) {
  SJD_CUDA(launch_kernel(attention_combine_kernel, dim3(M, n_heads), dim3(128), 0, stream, partial, in_pos, out, n_heads,
                         head_dim, splits, hilo));
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_attention(int dtype, const float *q, KvLayout kv, const int32_t *in_pos, float *out, float *partial, int M,
                     int rows_per_seq, int n_heads, int splits, cudaStream_t stream, HiLoOut hilo) {
  if (dtype == SJD_F32)
    return attention_t<float>(q, kv, in_pos, out, partial, M, rows_per_seq, n_heads, splits, stream, hilo);
  if (dtype == SJD_BF16)
    return attention_t<__nv_bfloat16>(q, kv, in_pos, out, partial, M, rows_per_seq, n_heads, splits, stream, hilo);
  return SJD_ERR_UNSUPPORTED;
}

}  // namespace sjd
