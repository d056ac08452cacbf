// Generic kernels of the decoder forward pass (Sec. 3.1: the auto-regressive transformer; Sec. 4.1
// Step 2: one pass over the window).  These cover every shape and both dtypes with plain FMA
// arithmetic and fp32 accumulation.  Activations between kernels are fp32 (they are a few hundred KB);
// only weights, the KV cache and the stored logits are in the model dtype.
#include "common.cuh"

namespace sjd {
namespace {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ void store_hilo(const HiLoOut &o, size_t idx, float v) {
  if (!o.base) return;
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  o.base[idx] = hi;
  o.base[o.lo_offset + idx] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// ------------------------------------------------------------------------------------ GEMM (FMA)
// 32 x 64 output tile per block of 256 threads, K in slices of 32; every access is bounds-checked so
// any M, N, K (683, 1408, ...) works.  Sums run over k in increasing order: deterministic.
constexpr int GM = 32, GN = 64, GK = 32;

template <typename T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const float *__restrict__ A, int lda, const T *__restrict__ Wt,
                                                        void *__restrict__ Cv, int ldc, int M, int N, int K) {
  __shared__ float As[GM][GK + 1];
  __shared__ float Ws[GN][GK + 1];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * GM, n0 = blockIdx.x * GN;
  const int ty = tid >> 4, tx = tid & 15;  // rows ty*2..+1, cols tx*4..+3
  float acc[2][4] = {};
  for (int k0 = 0; k0 < K; k0 += GK) {
    for (int i = tid; i < GM * GK; i += 256) {
      const int r = i / GK, c = i % GK;
      const int m = m0 + r, k = k0 + c;
      As[r][c] = (m < M && k < K) ? A[(size_t)m * lda + k] : 0.0f;
    }
    for (int i = tid; i < GN * GK; i += 256) {
      const int r = i / GK, c = i % GK;
      const int n = n0 + r, k = k0 + c;
      Ws[r][c] = (n < N && k < K) ? to_f<T>(Wt[(size_t)n * K + k]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < GK; ++kk) {
      const float a0 = As[ty * 2][kk], a1 = As[ty * 2 + 1][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float w = Ws[tx * 4 + j][kk];
        acc[0][j] = fmaf(a0, w, acc[0][j]);
        acc[1][j] = fmaf(a1, w, acc[1][j]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int m = m0 + ty * 2 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      const size_t idx = (size_t)m * ldc + n;
      if (EPI == EPI_STORE_F32) reinterpret_cast<float *>(Cv)[idx] = acc[i][j];
      else if (EPI == EPI_ADD_F32) reinterpret_cast<float *>(Cv)[idx] += acc[i][j];
      else reinterpret_cast<T *>(Cv)[idx] = from_f<T>(acc[i][j]);
    }
  }
}

template <typename T>
int gemm_simt_t(const void *A, int lda, const void *Wt, void *C, int ldc, int M, int N, int K, int epi,
                cudaStream_t stream) {
  dim3 grid((N + GN - 1) / GN, (M + GM - 1) / GM);
  const float *a = reinterpret_cast<const float *>(A);
  const T *w = reinterpret_cast<const T *>(Wt);
  if (epi == EPI_STORE_F32) gemm_simt_kernel<T, EPI_STORE_F32><<<grid, 256, 0, stream>>>(a, lda, w, C, ldc, M, N, K);
  else if (epi == EPI_STORE_T) gemm_simt_kernel<T, EPI_STORE_T><<<grid, 256, 0, stream>>>(a, lda, w, C, ldc, M, N, K);
  else if (epi == EPI_ADD_F32) gemm_simt_kernel<T, EPI_ADD_F32><<<grid, 256, 0, stream>>>(a, lda, w, C, ldc, M, N, K);
  else return SJD_ERR_BAD_ARG;
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

// ------------------------------------------------------------------------------------ embedding
template <typename T>
__global__ void embed_kernel(const T *__restrict__ emb, const int32_t *__restrict__ tok, float *__restrict__ x, int d,
                             int vocab) {
  pdl_trigger();
  pdl_wait();
  const int m = blockIdx.x;
  int t = tok[m];
  t = min(max(t, 0), vocab - 1);
  const T *row = emb + (size_t)t * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)m * d + i] = to_f<T>(row[i]);
}

// ------------------------------------------------------------------------------------ RMSNorm
template <typename T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float *__restrict__ x, const T *__restrict__ gain,
                                                      float *__restrict__ h, int d, float eps, HiLoOut hilo) {
  __shared__ float red[8];
  const int m = blockIdx.x, tid = threadIdx.x;
  const float *row = x + (size_t)m * d;
  float ss = 0.0f;
  for (int i = tid; i < d; i += 256) ss = fmaf(row[i], row[i], ss);
  ss = warp_sum(ss);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  float tot = 0.0f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float scale = rsqrtf(tot / (float)d + eps);
  for (int i = tid; i < d; i += 256) {
    const float v = row[i] * scale * to_f<T>(gain[i]);
    h[(size_t)m * d + i] = v;
    store_hilo(hilo, (size_t)m * d + i, v);
  }
}

// ------------------------------------------------------------------------------------ RoPE + KV append
template <typename T>
__global__ void rope_append_kernel(const float *__restrict__ qkv, const int32_t *__restrict__ in_pos,
                                   const float2 *__restrict__ rope, float *__restrict__ q, KvLayout kv, int rows_per_seq,
                                   int n_heads, QkNorm qkn) {
  const int m = blockIdx.x;
  const int pos = in_pos[m];
  if (pos < 0) return;
  const int b = m / rows_per_seq;
  const int hd = kv.head_dim, half = hd >> 1, nkv = kv.n_kv_heads;
  const int nq = n_heads * hd, nk = nkv * hd;
  const float *row = qkv + (size_t)m * (nq + 2 * nk);
  const float2 *cs = rope + (size_t)pos * half;
  T *cache = reinterpret_cast<T *>(kv.base);
  // rotated pairs of q and k
  for (int i = threadIdx.x; i < (n_heads + nkv) * half; i += blockDim.x) {
    const int head = i / half, j = i % half;
    const float2 c = cs[j];
    float g1 = 1.0f, g2 = 1.0f;
    if (qkn.q_gain) {   // QK-norm: this head's RMS over its hd entries (every thread of the head sums them itself)
      const float *hv = row + (head < n_heads ? head * hd : nq + (head - n_heads) * hd);
      float ss = 0.0f;
      for (int t = 0; t < hd; ++t) ss += hv[t] * hv[t];
      const float rinv = rsqrtf(ss / (float)hd + qkn.eps);
      const T *gain = reinterpret_cast<const T *>(head < n_heads ? qkn.q_gain : qkn.k_gain);
      g1 = rinv * to_f<T>(gain[j]);
      g2 = rinv * to_f<T>(gain[j + half]);
    }
    if (head < n_heads) {
      const float x1 = g1 * row[head * hd + j], x2 = g2 * row[head * hd + j + half];
      q[(size_t)m * nq + head * hd + j] = x1 * c.x - x2 * c.y;
      q[(size_t)m * nq + head * hd + j + half] = x2 * c.x + x1 * c.y;
    } else {
      const int kh = head - n_heads;
      const float x1 = g1 * row[nq + kh * hd + j], x2 = g2 * row[nq + kh * hd + j + half];
      T *dst = cache + kv_row_offset(kv, b, 0, kh, pos);
      dst[j] = from_f<T>(x1 * c.x - x2 * c.y);
      dst[j + half] = from_f<T>(x2 * c.x + x1 * c.y);
    }
  }
  for (int i = threadIdx.x; i < nk; i += blockDim.x) {
    const int kh = i / hd, j = i % hd;
    cache[kv_row_offset(kv, b, 1, kh, pos) + j] = from_f<T>(row[nq + nk + i]);
  }
}

// ------------------------------------------------------------------------------------ SwiGLU
__global__ void swiglu_kernel(const float *__restrict__ gu, float *__restrict__ act, int M, int F, HiLoOut hilo) {
  const size_t total = (size_t)M * F;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t m = i / F, f = i % F;
    const float g = gu[m * 2 * F + f], u = gu[m * 2 * F + F + f];
    const float v = g / (1.0f + expf(-g)) * u;
    act[i] = v;
    store_hilo(hilo, i, v);
  }
}

}  // namespace

#define SJD_DISPATCH(dtype, CALL)                         \
  do {                                                    \
    if ((dtype) == SJD_F32) { using T = float; CALL; }    \
    else if ((dtype) == SJD_BF16) { using T = __nv_bfloat16; CALL; } \
    else return SJD_ERR_UNSUPPORTED;                      \
  } while (0)

int launch_gemm_simt(int dtype, const void *A, int lda, const void *Wt, void *C, int ldc, int M, int N, int K,
                     int epilogue, cudaStream_t stream) {
  if (M <= 0 || N <= 0 || K <= 0) return SJD_ERR_BAD_ARG;
  SJD_DISPATCH(dtype, return gemm_simt_t<T>(A, lda, Wt, C, ldc, M, N, K, epilogue, stream));
}

int launch_embed(int dtype, const void *tok_emb, const int32_t *tok, float *x, int M, int d, int vocab,
                 cudaStream_t stream) {
  SJD_DISPATCH(dtype, SJD_CUDA(launch_kernel(embed_kernel<T>, dim3(M), dim3(256), 0, stream, reinterpret_cast<const T *>(tok_emb),
                                             tok, x, d, vocab)));
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_rmsnorm(int dtype, const float *x, const void *gain, float *h, int M, int d, float eps, cudaStream_t stream,
                   HiLoOut hilo) {
  SJD_DISPATCH(dtype, (rmsnorm_kernel<T><<<M, 256, 0, stream>>>(x, reinterpret_cast<const T *>(gain), h, d, eps, hilo)));
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_rope_append(int dtype, const float *qkv, const int32_t *in_pos, const float2 *rope_table, float *q,
                       KvLayout kv, int M, int rows_per_seq, int n_heads, QkNorm qkn, cudaStream_t stream) {
  SJD_DISPATCH(dtype, (rope_append_kernel<T><<<M, 256, 0, stream>>>(qkv, in_pos, rope_table, q, kv, rows_per_seq,
                                                                   n_heads, qkn)));
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_swiglu(const float *gu, float *act, int M, int F, cudaStream_t stream, HiLoOut hilo) {
  const size_t total = (size_t)M * F;
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  swiglu_kernel<<<blocks, 256, 0, stream>>>(gu, act, M, F, hilo);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

}  // namespace sjd

namespace sjd {
namespace {
__global__ void split_hilo_kernel(const float *__restrict__ x, HiLoOut o, size_t total) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
    store_hilo(o, i, x[i]);
}
}  // namespace

// hi/lo bf16 planes of an fp32 matrix (same row stride), for the tensor-core GEMM
int launch_split_hilo(const float *x, HiLoOut o, size_t total, cudaStream_t stream) {
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  split_hilo_kernel<<<blocks, 256, 0, stream>>>(x, o, total);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}
}  // namespace sjd
