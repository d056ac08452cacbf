// Consumer kernels of the tensor-core path.  The weight-streaming GEMM leaves one fp32 partial plane
// per K split; each kernel here adds the planes in split order (fixed order: deterministic) while doing
// the element-wise work that follows the projection in the decoder layer (Sec. 3.1 / Sec. 4.1 Step 2),
// and emits the next GEMM's activation operand directly as bf16 hi + lo planes.
#include "common.cuh"

namespace sjd {
SJD_TIMELINE_TU(fused)
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

// Per-row RMS scale from the partial sums of squares a resid_gain launch left:
// scale(m) = 1 / sqrt(mean(x[m]^2) + eps).  The scale is a per-row scalar, so it commutes with the
// projection that follows the normalisation and is applied by that projection's consumer.
__device__ __forceinline__ float row_scale(const RowScale &rs, int m) {
  if (!rs.ss_part) return 1.0f;
  float tot = 0.0f;
  for (int j = 0; j < rs.n_part; ++j) tot += __ldg(rs.ss_part + (size_t)m * rs.n_part + j);
  return rsqrtf(tot * rs.inv_d + rs.eps);
}
// the same for a row index that is uniform over the (full) warp: lanes share the loads.  The partials
// are added in a fixed tree order, so every caller gets the same bits.
__device__ __forceinline__ float row_scale_warp(const RowScale &rs, int m) {
  if (!rs.ss_part) return 1.0f;
  const int lane = threadIdx.x & 31;
  float tot = 0.0f;
  for (int j = lane; j < rs.n_part; j += 32) tot += __ldg(rs.ss_part + (size_t)m * rs.n_part + j);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  return rsqrtf(tot * rs.inv_d + rs.eps);
}

// x[m][:] += sum_s P[s][m][:]  (residual connection); emits x * gain as bf16 hi/lo planes (the RMS
// scale is applied downstream) and one partial of sum(x^2) per 128 columns (= per warp, = per weight
// tile of the projections, which write the same partials when they fold this step into their
// epilogue).  Grid (rows, column chunks of 1024).
constexpr int RG_THREADS = 256;
constexpr int RG_COLS = RG_THREADS * 4;

template <typename T>
__global__ void __launch_bounds__(RG_THREADS) resid_gain_kernel(float *__restrict__ x, PlaneSet ps, const T *__restrict__ gain,
                                                               HiLoOut h, float *__restrict__ ss_part, int d) {
  pdl_trigger();
  SJD_TL(TL_RESID, 0, threadIdx.x == 0);
  pdl_wait();
  SJD_TL(TL_RESID, 1, threadIdx.x == 0);
  const int m = blockIdx.x, chunk = blockIdx.y, tid = threadIdx.x;
  const int c0 = chunk * RG_COLS + tid * 4;
  float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  if (c0 < d) {   // d is a multiple of 4
    const float4 t = *reinterpret_cast<const float4 *>(x + (size_t)m * d + c0);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    for (int s = 0; s < ps.splits; ++s) {
      const float4 pv = __ldg(reinterpret_cast<const float4 *>(ps.base + (size_t)s * ps.plane_stride + (size_t)m * ps.ld + c0));
      v[0] += pv.x; v[1] += pv.y; v[2] += pv.z; v[3] += pv.w;
    }
    if (ps.splits > 0) *reinterpret_cast<float4 *>(x + (size_t)m * d + c0) = make_float4(v[0], v[1], v[2], v[3]);
#pragma unroll
    for (int i = 0; i < 4; ++i) put_hilo(h, (size_t)m * d + c0 + i, v[i] * to_f<T>(gain[c0 + i]));
  }
  float ss = v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
  ss = warp_sum(ss);
  const int part = chunk * (RG_THREADS / 32) + (tid >> 5), n_part = (d + 127) / 128;
  if ((tid & 31) == 0 && part < n_part) ss_part[(size_t)m * n_part + part] = ss;
  SJD_TL(TL_RESID, 2, threadIdx.x == 0);
}

// q,k,v = scale * sum of the QKV planes; rotate q and k (pairs i, i + hd/2) by the row's absolute
// position; q -> fp32 [M][H*hd]; k, v -> cache row in_pos[m].  64 threads per (row, head slot), four
// slots per block.
template <typename T>
__global__ void qkv_finish_kernel(PlaneSet ps, RowScale rs, const int32_t *__restrict__ in_pos,
                                  const float2 *__restrict__ rope, float *__restrict__ q, KvLayout kv, int rows_per_seq,
                                  int n_heads, QkNorm qkn) {
  __shared__ float s_ss[8];   // QK-norm: per-warp sums of squares of a head (two warps per 64-thread group)
  pdl_trigger();
  SJD_TL(TL_QKV, 0, threadIdx.x == 0);
  pdl_wait();
  SJD_TL(TL_QKV, 1, threadIdx.x == 0);
  const int m = blockIdx.x, lt = threadIdx.x & 63;
  const int b = m / rows_per_seq;
  const int hd = kv.head_dim, half = hd >> 1, nkv = kv.n_kv_heads;
  const int nq = n_heads * hd, nk = nkv * hd;
  const size_t rbase = (size_t)m * ps.ld;
  T *cache = reinterpret_cast<T *>(kv.base);
  // The loads of the projection planes depend on nothing, the row's position and RMS scale are loads of their
  // own and the rotary entry depends on the position: the plane loads of a slot are issued first, so that the
  // kernel waits for two memory round trips in a row and not three.
  int pos = 0;
  float sc = 0.0f;
  bool first = true;
  // the block's 64-thread groups walk over the head slots of the row (one pass when the grid has a
  // block for every four slots, several when many rows share fewer blocks per row)
  const int stride = gridDim.y * (blockDim.x >> 6);
  for (int slot = blockIdx.y * (blockDim.x >> 6) + (threadIdx.x >> 6); slot < n_heads + 2 * nkv; slot += stride) {
    const bool is_v = slot >= n_heads + nkv;
    const bool is_q = slot < n_heads;
    // head_dim <= 128: a thread of the group owns at most one rotary pair (j, j + half) of a q or k head,
    // or the entries j and j + 64 of a v head
    const int col0 = is_q ? slot * hd : is_v ? nq + nk + (slot - n_heads - nkv) * hd : nq + (slot - n_heads) * hd;
    const int ja = lt, jb = is_v ? lt + 64 : lt + half;
    const bool has_a = is_v ? ja < hd : ja < half, has_b = is_v ? jb < hd : ja < half;
    float x1 = 0.0f, x2 = 0.0f;
    if (has_a) x1 = sum_planes(ps, rbase + col0 + ja);
    if (has_b) x2 = sum_planes(ps, rbase + col0 + jb);
    if (first) {   // uniform over the block
      pos = in_pos[m];
      sc = row_scale_warp(rs, m);   // before any thread leaves: the warp shares the loads
      first = false;
      if (pos < 0) return;
    }
    x1 *= sc;
    x2 *= sc;
    if (is_v) {
      T *dst = cache + kv_row_offset(kv, b, 1, slot - n_heads - nkv, pos);
      if (has_a) dst[ja] = from_f<T>(x1);
      if (has_b) dst[jb] = from_f<T>(x2);
      continue;
    }
    if (qkn.q_gain) {   // QK-norm: RMS over the head's entries, held by the 64 threads of this group
      const int grp = threadIdx.x >> 6;
      const float ws = warp_sum(x1 * x1 + x2 * x2);
      if ((threadIdx.x & 31) == 0) s_ss[threadIdx.x >> 5] = ws;
      asm volatile("bar.sync %0, 64;" ::"r"(grp + 1) : "memory");
      const float rinv = rsqrtf((s_ss[2 * grp] + s_ss[2 * grp + 1]) / (float)hd + qkn.eps);
      asm volatile("bar.sync %0, 64;" ::"r"(grp + 1) : "memory");   // the sums are reused by the group's next head
      if (has_a) {
        const T *gain = reinterpret_cast<const T *>(is_q ? qkn.q_gain : qkn.k_gain);
        x1 *= rinv * to_f<T>(gain[ja]);
        x2 *= rinv * to_f<T>(gain[jb]);
      }
    }
    if (!has_a) continue;
    const float2 c = rope[(size_t)pos * half + ja];
    const float r1 = x1 * c.x - x2 * c.y, r2 = x2 * c.x + x1 * c.y;
    if (is_q) {
      q[(size_t)m * nq + slot * hd + ja] = r1;
      q[(size_t)m * nq + slot * hd + jb] = r2;
    } else {
      T *dst = cache + kv_row_offset(kv, b, 0, slot - n_heads, pos);
      dst[ja] = from_f<T>(r1);
      dst[jb] = from_f<T>(r2);
    }
  }
}

// act = silu(scale * sum gate planes) * (scale * sum up planes) as bf16 hi/lo planes; planes [S][M][2F]
__global__ void swiglu_finish_kernel(PlaneSet ps, RowScale rs, HiLoOut act, int M, int F) {
  pdl_trigger();
  SJD_TL(TL_SWIGLU, 0, threadIdx.x == 0);
  pdl_wait();
  SJD_TL(TL_SWIGLU, 1, threadIdx.x == 0);
  if ((F & 3) == 0 && (ps.ld & 3) == 0 && (ps.plane_stride & 3) == 0) {
    // grid (column chunks, rows): a thread handles groups of four adjacent columns of one row
    const int m = blockIdx.y;
    const float sc = row_scale_warp(rs, m);
    const float *row = ps.base + (size_t)m * ps.ld;
    for (int f = (blockIdx.x * blockDim.x + threadIdx.x) * 4; f < F; f += gridDim.x * blockDim.x * 4) {
      float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
      for (int sp = 0; sp < ps.splits; ++sp) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(row + (size_t)sp * ps.plane_stride + f));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(row + (size_t)sp * ps.plane_stride + F + f));
        g.x += a.x; g.y += a.y; g.z += a.z; g.w += a.w;
        u.x += b.x; u.y += b.y; u.z += b.z; u.w += b.w;
      }
      const float gv[4] = {sc * g.x, sc * g.y, sc * g.z, sc * g.w}, uv[4] = {sc * u.x, sc * u.y, sc * u.z, sc * u.w};
      __nv_bfloat16 hi[4], lo[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float v = gv[i] / (1.0f + expf(-gv[i])) * uv[i];
        hi[i] = __float2bfloat16_rn(v);
        lo[i] = __float2bfloat16_rn(v - __bfloat162float(hi[i]));
      }
      const size_t idx = (size_t)m * F + f;   // multiple of 4: 8-byte aligned stores
      *reinterpret_cast<uint2 *>(act.base + idx) = *reinterpret_cast<const uint2 *>(hi);
      *reinterpret_cast<uint2 *>(act.base + act.lo_offset + idx) = *reinterpret_cast<const uint2 *>(lo);
    }
  } else {
    const size_t total = (size_t)M * F;
    const size_t nthreads = (size_t)gridDim.x * gridDim.y * blockDim.x;
    for (size_t i = ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += nthreads) {
      const size_t m = i / F, f = i % F;
      const float sc = row_scale(rs, (int)m);
      const float g = sc * sum_planes(ps, m * ps.ld + f), u = sc * sum_planes(ps, m * ps.ld + F + f);
      put_hilo(act, i, g / (1.0f + expf(-g)) * u);
    }
  }
  SJD_TL(TL_SWIGLU, 2, threadIdx.x == 0);
}

}  // namespace

int resid_gain_parts(int d) { return (d + 127) / 128; }

int launch_resid_gain(int dtype, float *x, PlaneSet ps, const void *gain, HiLoOut h, float *ss_part, int M, int d,
                      cudaStream_t stream) {
  if (d % 4 != 0) return SJD_ERR_UNSUPPORTED;
  const dim3 grid(M, (d + RG_COLS - 1) / RG_COLS);
  if (dtype == SJD_F32)
    SJD_CUDA(launch_kernel(resid_gain_kernel<float>, grid, dim3(RG_THREADS), 0, stream, x, ps,
                           reinterpret_cast<const float *>(gain), h, ss_part, d));
  else if (dtype == SJD_BF16)
    SJD_CUDA(launch_kernel(resid_gain_kernel<__nv_bfloat16>, grid, dim3(RG_THREADS), 0, stream, x, ps,
                           reinterpret_cast<const __nv_bfloat16 *>(gain), h, ss_part, d));
  else
    return SJD_ERR_UNSUPPORTED;
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_qkv_finish(int dtype, PlaneSet ps, RowScale rs, const int32_t *in_pos, const float2 *rope_table, float *q,
                      KvLayout kv, int M, int rows_per_seq, int n_heads, QkNorm qkn, cudaStream_t stream) {
  if (kv.head_dim > 128) return SJD_ERR_UNSUPPORTED;
  // a block per four head slots for a few dozen rows; fewer blocks per row (each walking more slots) as
  // the rows grow, about eight blocks per SM in all
  int per_row = (n_heads + 2 * kv.n_kv_heads + 3) / 4;
  const int cap = 1184 / M > 0 ? 1184 / M : 1;
  per_row = per_row < cap ? per_row : cap;
  const dim3 grid(M, per_row);
  if (dtype == SJD_F32)
    SJD_CUDA(launch_kernel(qkv_finish_kernel<float>, grid, dim3(256), 0, stream, ps, rs, in_pos, rope_table, q, kv,
                           rows_per_seq, n_heads, qkn));
  else if (dtype == SJD_BF16)
    SJD_CUDA(launch_kernel(qkv_finish_kernel<__nv_bfloat16>, grid, dim3(256), 0, stream, ps, rs, in_pos, rope_table, q, kv,
                           rows_per_seq, n_heads, qkn));
  else
    return SJD_ERR_UNSUPPORTED;
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_swiglu_finish(PlaneSet ps, RowScale rs, HiLoOut act, int M, int F, cudaStream_t stream) {
  // Few enough blocks that (for windows of a few dozen rows) the whole grid is resident at once and
  // leaves thread slots free: only then is the next kernel scheduled early under dependent launch.
  int per_row = (F / 4 + 255) / 256;
  const int cap = 296 / (M < 296 ? M : 296);
  per_row = per_row > cap ? (cap > 0 ? cap : 1) : per_row;
  SJD_CUDA(launch_kernel(swiglu_finish_kernel, dim3(per_row, M), dim3(256), 0, stream, ps, rs, act, M, F));
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

}  // namespace sjd
