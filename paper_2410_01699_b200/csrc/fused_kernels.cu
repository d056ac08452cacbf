// Consumer kernels of the tensor-core path.  The weight-streaming GEMM leaves one fp32 partial plane
// per K split; each kernel here adds the planes in split order (fixed order: deterministic) while doing
// the element-wise work that follows the projection in the decoder layer (Sec. 3.1 / Sec. 4.1 Step 2),
// and emits the next GEMM's activation operand directly as bf16 hi + lo planes.
#include "common.cuh"

namespace sjd {
namespace {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ void put_hilo(const HiLoOut &o, size_t idx, float v) {
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  o.base[idx] = hi;
  o.base[o.lo_offset + idx] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

__device__ __forceinline__ float sum_planes(const PlaneSet &ps, size_t idx) {
  float acc = 0.0f;
  for (int s = 0; s < ps.splits; ++s) acc += __ldg(ps.base + (size_t)s * ps.plane_stride + idx);
  return acc;
}

// x[m][:] += sum_s P[s][m][:]  (residual connection), then h = rmsnorm(x; gain) as bf16 hi/lo planes.
// One block per row; the sum of squares is reduced in a fixed tree.
constexpr int RN_THREADS = 512;
constexpr int RN_MAX_PER_THREAD = 16;   // d_model <= 8192

template <typename T>
__global__ void __launch_bounds__(RN_THREADS) resid_norm_kernel(float *__restrict__ x, PlaneSet ps, const T *__restrict__ gain,
                                                               HiLoOut h, int d, float eps) {
  __shared__ float red[RN_THREADS / 32];
  const int m = blockIdx.x, tid = threadIdx.x;
  float *row = x + (size_t)m * d;
  float v[RN_MAX_PER_THREAD];
  float ss = 0.0f;
#pragma unroll
  for (int j = 0; j < RN_MAX_PER_THREAD; ++j) {
    const int i = tid + j * RN_THREADS;
    v[j] = 0.0f;
    if (i < d) {
      float t = row[i];
      if (ps.splits > 0) t += sum_planes(ps, (size_t)m * ps.ld + i);
      v[j] = t;
      ss = fmaf(t, t, ss);
    }
  }
  ss = warp_sum(ss);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  float tot = 0.0f;
#pragma unroll
  for (int w = 0; w < RN_THREADS / 32; ++w) tot += red[w];
  const float scale = rsqrtf(tot / (float)d + eps);
#pragma unroll
  for (int j = 0; j < RN_MAX_PER_THREAD; ++j) {
    const int i = tid + j * RN_THREADS;
    if (i < d) {
      if (ps.splits > 0) row[i] = v[j];
      put_hilo(h, (size_t)m * d + i, v[j] * scale * to_f<T>(gain[i]));
    }
  }
}

// q,k,v = sum of the QKV planes; rotate q and k (pairs i, i + hd/2) by the row's absolute position;
// q -> fp32 [M][H*hd]; k, v -> cache row in_pos[m].  One block per (row, head slot).
template <typename T>
__global__ void qkv_finish_kernel(PlaneSet ps, const int32_t *__restrict__ in_pos, const float2 *__restrict__ rope,
                                  float *__restrict__ q, KvLayout kv, int rows_per_seq, int n_heads) {
  const int m = blockIdx.x, slot = blockIdx.y;
  const int pos = in_pos[m];
  if (pos < 0) return;
  const int b = m / rows_per_seq;
  const int hd = kv.head_dim, half = hd >> 1, nkv = kv.n_kv_heads;
  const int nq = n_heads * hd, nk = nkv * hd;
  const size_t rbase = (size_t)m * ps.ld;
  T *kbase = reinterpret_cast<T *>(kv.base) + (size_t)b * 2 * nkv * kv.max_seq * hd;
  T *vbase = kbase + (size_t)nkv * kv.max_seq * hd;
  if (slot < n_heads + nkv) {
    const bool is_q = slot < n_heads;
    const int col0 = is_q ? slot * hd : nq + (slot - n_heads) * hd;
    for (int j = threadIdx.x; j < half; j += blockDim.x) {
      const float2 c = rope[(size_t)pos * half + j];
      const float x1 = sum_planes(ps, rbase + col0 + j), x2 = sum_planes(ps, rbase + col0 + j + half);
      const float r1 = x1 * c.x - x2 * c.y, r2 = x2 * c.x + x1 * c.y;
      if (is_q) {
        q[(size_t)m * nq + slot * hd + j] = r1;
        q[(size_t)m * nq + slot * hd + j + half] = r2;
      } else {
        T *dst = kbase + ((size_t)(slot - n_heads) * kv.max_seq + pos) * hd;
        dst[j] = from_f<T>(r1);
        dst[j + half] = from_f<T>(r2);
      }
    }
  } else {
    const int kh = slot - n_heads - nkv;
    T *dst = vbase + ((size_t)kh * kv.max_seq + pos) * hd;
    for (int j = threadIdx.x; j < hd; j += blockDim.x) dst[j] = from_f<T>(sum_planes(ps, rbase + nq + nk + kh * hd + j));
  }
}

// act = silu(sum gate planes) * (sum up planes) as bf16 hi/lo planes; planes are [S][M][2F] (gate | up)
__global__ void swiglu_finish_kernel(PlaneSet ps, HiLoOut act, int M, int F) {
  const size_t total = (size_t)M * F;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t m = i / F, f = i % F;
    const float g = sum_planes(ps, m * ps.ld + f), u = sum_planes(ps, m * ps.ld + F + f);
    put_hilo(act, i, g / (1.0f + expf(-g)) * u);
  }
}

}  // namespace

int launch_resid_norm(int dtype, float *x, PlaneSet ps, const void *gain, HiLoOut h, int M, int d, float eps,
                      cudaStream_t stream) {
  if (d > RN_THREADS * RN_MAX_PER_THREAD) return SJD_ERR_UNSUPPORTED;
  if (dtype == SJD_F32)
    resid_norm_kernel<float><<<M, RN_THREADS, 0, stream>>>(x, ps, reinterpret_cast<const float *>(gain), h, d, eps);
  else if (dtype == SJD_BF16)
    resid_norm_kernel<__nv_bfloat16><<<M, RN_THREADS, 0, stream>>>(x, ps, reinterpret_cast<const __nv_bfloat16 *>(gain), h, d, eps);
  else
    return SJD_ERR_UNSUPPORTED;
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_qkv_finish(int dtype, PlaneSet ps, const int32_t *in_pos, const float2 *rope_table, float *q, KvLayout kv, int M,
                      int rows_per_seq, int n_heads, cudaStream_t stream) {
  const dim3 grid(M, n_heads + 2 * kv.n_kv_heads);
  if (dtype == SJD_F32)
    qkv_finish_kernel<float><<<grid, 64, 0, stream>>>(ps, in_pos, rope_table, q, kv, rows_per_seq, n_heads);
  else if (dtype == SJD_BF16)
    qkv_finish_kernel<__nv_bfloat16><<<grid, 64, 0, stream>>>(ps, in_pos, rope_table, q, kv, rows_per_seq, n_heads);
  else
    return SJD_ERR_UNSUPPORTED;
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_swiglu_finish(PlaneSet ps, HiLoOut act, int M, int F, cudaStream_t stream) {
  const size_t total = (size_t)M * F;
  const int blocks = (int)((total + 255) / 256 < 2368 ? (total + 255) / 256 : 2368);
  swiglu_finish_kernel<<<blocks, 256, 0, stream>>>(ps, act, M, F);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

}  // namespace sjd
