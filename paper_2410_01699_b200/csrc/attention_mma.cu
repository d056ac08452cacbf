// Window-causal split-KV attention on tensor cores for bf16 caches (Sec. 3.2 / Sec. 4.1 Step 2: the W
// window queries attend the cached prefix plus the in-window causal block).
//
// One CTA per (query head, sequence, key range).  K and V tiles of 64 keys are staged in shared memory
// by TMA (128-byte swizzle, two 64-dim boxes per 128-dim head) through a ring of mbarrier-guarded
// stages; each warp owns 16 query rows, keeps Q (pre-scaled, split into bf16 hi + lo), the running
// max / sum and the fp32 output accumulators in registers and runs QK^T and PV as m16n8k16 bf16
// mma.sync with ldmatrix-fed operands.  A CTA always has four warps: with fewer than 64 query rows the
// warps that share 16 rows split the keys of every tile between them (KG = 2 or 4 key groups, each
// with its own running max / sum / output) and merge through shared memory at the end; one warp per
// scheduler alone cannot keep the tensor pipe and the exponentials going at the same time.  The probabilities are split hi + lo as well, so neither
// operand loses more than ~2^-17 relative.  The kernel is bound by streaming K/V once from HBM (GQA
// heads of a group share their tiles through L2).  Partials (max, sum, unnormalised output) go to the
// merge kernel of attention.cu.  Every barrier wait is bounded.
#include <cuda.h>

#include "common.cuh"

namespace sjd {
SJD_TIMELINE_TU(attn)
namespace {

constexpr int KT = 64;                 // keys per tile
constexpr int kStagesAttn = 3;
constexpr unsigned long long kWaitNsAttn = 2000000000ull;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool bar_try(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool bar_wait(uint64_t *bar, uint32_t parity) {
  if (bar_try(bar, parity)) return true;
  unsigned long long t0, t1;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (bar_try(bar, parity)) return true;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
    if (t1 - t0 > kWaitNsAttn) return false;
  }
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_addr(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_addr(bar))
      : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two floats -> packed bf16 hi pair and bf16 lo pair (lo = value - hi, rounded)
__device__ __forceinline__ void split_pair(float x, float y, uint32_t &hi, uint32_t &lo) {
  const __nv_bfloat16 hx = __float2bfloat16_rn(x), hy = __float2bfloat16_rn(y);
  const __nv_bfloat16 lx = __float2bfloat16_rn(x - __bfloat162float(hx)), ly = __float2bfloat16_rn(y - __bfloat162float(hy));
  hi = (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(lx) | ((uint32_t)__bfloat16_as_ushort(ly) << 16);
}

struct AttnParams {
  const float *q;        // [M][H*HD]
  const int32_t *in_pos; // [M]
  float *partial;        // [M][H][splits][HD + 2]
  float *out;            // [M][H*HD]: written here when splits == 1 (no merge launch needed)
  HiLoOut hilo;          // optional bf16 hi/lo planes of out (same case)
  int *status;
  int rows_per_seq, n_heads, n_kv_heads, splits;
  int plane0;            // first cache plane of this layer: planes are [b][k|v][kv_head]
  // paged cache: planes are [page][layer][k|v][kv_head], one page (KT positions) per tile
  const int32_t *page_table;   // [B][pages_per_seq]; null: contiguous
  int pages_per_seq, layer, n_layers;
};

template <int HD, int KG>
__global__ void __launch_bounds__(128) attention_mma_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams p) {
  constexpr int HALVES = HD / 64;                // 64-dim (128-byte) boxes per row
  constexpr int TILE_BYTES = KT * HD * 2;        // one of K or V
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ uint64_t bar_full[kStagesAttn];
  __shared__ int s_pos[64];
  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  pdl_trigger();
  SJD_TL(TL_ATTN, 0, threadIdx.x == 0);
  pdl_wait();   // keys/values of this step were written by the preceding kernel
  SJD_TL(TL_ATTN, 1, threadIdx.x == 0);
  const int h = blockIdx.x, b = blockIdx.y, split = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int W = p.rows_per_seq;
  const int kvh = h / (p.n_heads / p.n_kv_heads);
  const int m0 = b * W;
  const int g = lane >> 2, tq = lane & 3;
  const int n_rw = blockDim.x / (32 * KG);   // warps along the query rows
  const int rw = warp % n_rw, kg = warp / n_rw;   // this warp's 16 rows and its key group inside a tile
  constexpr int NB = KT / 8 / KG;            // 8-key blocks of a tile this warp scores
  constexpr int NK = KT / 16 / KG;           // 16-key blocks it multiplies with V

  if (tid < 64) s_pos[tid] = tid < W ? p.in_pos[m0 + tid] : -1;
  if (tid == 0) {
    for (int s = 0; s < kStagesAttn; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bar_full[s])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  int len = 0;
  for (int i = 0; i < W; ++i) len = max(len, s_pos[i] + 1);
  int chunk = (len + p.splits - 1) / p.splits;
  chunk = (chunk + KT - 1) / KT * KT;
  const int k_begin = split * chunk;
  const int k_end = min(len, k_begin + chunk);
  const int n_tiles = k_end > k_begin ? (k_end - k_begin + KT - 1) / KT : 0;
  const int plane_k = p.plane0 + (b * 2 + 0) * p.n_kv_heads + kvh;
  const int plane_v = p.plane0 + (b * 2 + 1) * p.n_kv_heads + kvh;

  auto issue = [&](int t) {   // thread 0: load tile t into its stage
    const int s = t % kStagesAttn;
    uint8_t *dst = smem + s * STAGE_BYTES;
    int key0 = k_begin + t * KT, pk = plane_k, pv = plane_v;
    if (p.page_table != nullptr) {   // k_begin is a multiple of KT: tile t is exactly one page
      const int page = __ldg(p.page_table + b * p.pages_per_seq + key0 / KT);
      pk = ((page * p.n_layers + p.layer) * 2 + 0) * p.n_kv_heads + kvh;
      pv = pk + p.n_kv_heads;
      key0 = 0;
    }
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&bar_full[s])), "r"(STAGE_BYTES)
                 : "memory");
#pragma unroll
    for (int hf = 0; hf < HALVES; ++hf) {
      tma_load_3d(dst + hf * (KT * 128), &kv_map, hf * 64, key0, pk, &bar_full[s]);
      tma_load_3d(dst + TILE_BYTES + hf * (KT * 128), &kv_map, hf * 64, key0, pv, &bar_full[s]);
    }
  };
  if (tid == 0)
    for (int t = 0; t < n_tiles && t < kStagesAttn; ++t) issue(t);

  // this thread's two query rows
  const int r0 = rw * 16 + g, r1 = r0 + 8;
  const int pos0 = r0 < W ? s_pos[r0] : -1, pos1 = r1 < W ? s_pos[r1] : -1;
  // Q fragments, pre-scaled by log2(e) / sqrt(HD), split hi / lo
  uint32_t qh[HD / 16][4], ql[HD / 16][4];
  {
    const float sc = 1.4426950408889634f * rsqrtf((float)HD);
    const float *q0 = p.q + ((size_t)(m0 + r0) * p.n_heads + h) * HD;
    const float *q1 = p.q + ((size_t)(m0 + r1) * p.n_heads + h) * HD;
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
      const int c = ks * 16 + tq * 2;
      float2 a = make_float2(0.f, 0.f), bq = a, cq = a, dq = a;
      if (pos0 >= 0) {
        a = *reinterpret_cast<const float2 *>(q0 + c);
        cq = *reinterpret_cast<const float2 *>(q0 + c + 8);
      }
      if (pos1 >= 0) {
        bq = *reinterpret_cast<const float2 *>(q1 + c);
        dq = *reinterpret_cast<const float2 *>(q1 + c + 8);
      }
      split_pair(a.x * sc, a.y * sc, qh[ks][0], ql[ks][0]);
      split_pair(bq.x * sc, bq.y * sc, qh[ks][1], ql[ks][1]);
      split_pair(cq.x * sc, cq.y * sc, qh[ks][2], ql[ks][2]);
      split_pair(dq.x * sc, dq.y * sc, qh[ks][3], ql[ks][3]);
    }
  }

  float o[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};

  bool ok = true;
  for (int t = 0; t < n_tiles; ++t) {
    const int s = t % kStagesAttn;
    const bool got = bar_wait(&bar_full[s], (uint32_t)((t / kStagesAttn) & 1));
    if (!__syncthreads_and(got)) { ok = false; break; }
    const uint32_t kbase = smem_addr(smem + s * STAGE_BYTES), vbase = kbase + TILE_BYTES;
    const int key0 = k_begin + t * KT;

    // ---- S = Q K^T  (16 rows x 64 keys per warp)
    float sacc[NB][4];
#pragma unroll
    for (int i = 0; i < NB; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.0f;
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
      const int half = ks >> 2, c0 = (ks & 3) * 2;
      // all key fragments of this k-step first, then one pass of MMAs per Q plane: consecutive MMAs
      // go to different accumulators, so none waits for the one before it
      uint32_t kf[NB][2];
#pragma unroll
      for (int nb = 0; nb < NB; nb += 2) {
        const int row = (kg * NB + nb) * 8 + (lane & 7) + ((lane >> 4) & 1) * 8;
        const int chunkc = c0 + ((lane >> 3) & 1);
        ldmatrix_x4(kbase + half * (KT * 128) + row * 128 + ((chunkc ^ (row & 7)) << 4), kf[nb][0], kf[nb][1], kf[nb + 1][0],
                    kf[nb + 1][1]);
      }
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) mma_bf16(sacc[nb], qh[ks], kf[nb][0], kf[nb][1]);
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) mma_bf16(sacc[nb], ql[ks], kf[nb][0], kf[nb][1]);
    }
    // ---- mask, online softmax (base 2)
    float tmax0 = -INFINITY, tmax1 = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      const int j = key0 + (kg * NB + nb) * 8 + tq * 2;
      if (!(j <= pos0 && j < k_end)) sacc[nb][0] = -INFINITY;
      if (!(j + 1 <= pos0 && j + 1 < k_end)) sacc[nb][1] = -INFINITY;
      if (!(j <= pos1 && j < k_end)) sacc[nb][2] = -INFINITY;
      if (!(j + 1 <= pos1 && j + 1 < k_end)) sacc[nb][3] = -INFINITY;
      tmax0 = fmaxf(tmax0, fmaxf(sacc[nb][0], sacc[nb][1]));
      tmax1 = fmaxf(tmax1, fmaxf(sacc[nb][2], sacc[nb][3]));
    }
    tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 1));
    tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 2));
    tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 1));
    tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 2));
    const float mn0 = fmaxf(m_run[0], tmax0), mn1 = fmaxf(m_run[1], tmax1);
    const float al0 = mn0 > -INFINITY ? exp2f(m_run[0] - mn0) : 1.0f;   // exp2f(-inf) = 0 for a fresh row
    const float al1 = mn1 > -INFINITY ? exp2f(m_run[1] - mn1) : 1.0f;
    const float sub0 = mn0 > -INFINITY ? mn0 : 0.0f, sub1 = mn1 > -INFINITY ? mn1 : 0.0f;
    m_run[0] = mn0;
    m_run[1] = mn1;
    float ls0 = 0.0f, ls1 = 0.0f;
    uint32_t ph[NK][4], pl[NK][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      const float p0 = exp2f(sacc[nb][0] - sub0), p1 = exp2f(sacc[nb][1] - sub0);
      const float p2 = exp2f(sacc[nb][2] - sub1), p3 = exp2f(sacc[nb][3] - sub1);
      ls0 += p0 + p1;
      ls1 += p2 + p3;
      const int kk = nb >> 1, hi8 = (nb & 1) * 2;   // A fragment regs: {row g, row g+8} x {keys 0-7, keys 8-15}
      split_pair(p0, p1, ph[kk][hi8], pl[kk][hi8]);
      split_pair(p2, p3, ph[kk][hi8 + 1], pl[kk][hi8 + 1]);
    }
    l_run[0] = l_run[0] * al0 + ls0;
    l_run[1] = l_run[1] * al1 + ls1;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      o[i][0] *= al0; o[i][1] *= al0;
      o[i][2] *= al1; o[i][3] *= al1;
    }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < NK; ++kk) {
#pragma unroll
      for (int c8 = 0; c8 < HD / 8; c8 += 8) {   // eight output column blocks at a time, same ordering idea
        uint32_t vf[8][2];
#pragma unroll
        for (int cd = 0; cd < 8; cd += 2) {
          const int row = (kg * NK + kk) * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int chunkc = c8 + cd + ((lane >> 4) & 1);
          ldmatrix_x4_trans(vbase + (chunkc >> 3) * (KT * 128) + row * 128 + (((chunkc & 7) ^ (row & 7)) << 4), vf[cd][0],
                            vf[cd][1], vf[cd + 1][0], vf[cd + 1][1]);
        }
#pragma unroll
        for (int cd = 0; cd < 8; ++cd) mma_bf16(o[c8 + cd], ph[kk], vf[cd][0], vf[cd][1]);
#pragma unroll
        for (int cd = 0; cd < 8; ++cd) mma_bf16(o[c8 + cd], pl[kk], vf[cd][0], vf[cd][1]);
      }
    }
    __syncthreads();   // every warp is done with this stage
    if (tid == 0 && t + kStagesAttn < n_tiles) issue(t + kStagesAttn);
  }
  if (!ok) {
    if (tid == 0) atomicExch(p.status, 4);
    // leave no copy in flight: wait (bounded) for the stages that were armed
    if (tid == 0)
      for (int t = 0; t < n_tiles && t < kStagesAttn; ++t) bar_wait(&bar_full[t % kStagesAttn], 0);
    return;
  }

  SJD_TL(TL_ATTN, 2, threadIdx.x == 0);
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
  if (KG > 1) {
    // ---- merge the key groups of each 16-row band: groups 1.. leave (max, sum, output) in the (now
    // idle) tile ring, group 0 folds them into its own.  Every tile was consumed before the last
    // barrier of the loop, so the ring is free.
    constexpr int REC = HD + 2;   // floats per row record
    float *xch = reinterpret_cast<float *>(smem);
    if (kg > 0) {
      float *dst = xch + ((size_t)((kg - 1) * n_rw + rw) * 16) * REC;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        float *row = dst + (g + rr * 8) * REC;
        if (tq == 0) {
          row[0] = m_run[rr];
          row[1] = l_run[rr];
        }
#pragma unroll
        for (int i = 0; i < HD / 8; ++i)
          *reinterpret_cast<float2 *>(row + 2 + i * 8 + tq * 2) = make_float2(o[i][rr * 2], o[i][rr * 2 + 1]);
      }
    }
    __syncthreads();
    if (kg > 0) return;
#pragma unroll
    for (int og = 1; og < KG; ++og) {
      const float *src = xch + ((size_t)((og - 1) * n_rw + rw) * 16) * REC;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const float *row = src + (g + rr * 8) * REC;
        const float m_o = row[0], l_o = row[1];
        const float mn = fmaxf(m_run[rr], m_o);
        const float a_s = mn > -INFINITY ? exp2f(m_run[rr] - mn) : 1.0f;   // both empty: keep zeros
        const float a_o = mn > -INFINITY ? exp2f(m_o - mn) : 0.0f;
        m_run[rr] = mn;
        l_run[rr] = l_run[rr] * a_s + l_o * a_o;
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) {
          const float2 v = *reinterpret_cast<const float2 *>(row + 2 + i * 8 + tq * 2);
          o[i][rr * 2] = o[i][rr * 2] * a_s + v.x * a_o;
          o[i][rr * 2 + 1] = o[i][rr * 2 + 1] * a_s + v.y * a_o;
        }
      }
    }
  }
  if (p.splits == 1) {
    // ---- a single key range: normalise and write the output rows (and their hi/lo planes) directly
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = rr == 0 ? r0 : r1;
      if (r >= W) continue;
      const float inv = l_run[rr] > 0.0f ? 1.0f / l_run[rr] : 0.0f;   // inactive rows: zeros
      const size_t base = ((size_t)(m0 + r) * p.n_heads + h) * HD;
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) {
        const float v0 = o[i][rr * 2] * inv, v1 = o[i][rr * 2 + 1] * inv;
        const size_t idx = base + i * 8 + tq * 2;
        *reinterpret_cast<float2 *>(p.out + idx) = make_float2(v0, v1);
        if (p.hilo.base) {
          uint32_t hi, lo;
          split_pair(v0, v1, hi, lo);
          *reinterpret_cast<uint32_t *>(p.hilo.base + idx) = hi;
          *reinterpret_cast<uint32_t *>(p.hilo.base + p.hilo.lo_offset + idx) = lo;
        }
      }
    }
    return;
  }
  // ---- partial record per (row, head, split): [max (natural log units), sum, o[HD]]
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int r = rr == 0 ? r0 : r1;
    if (r >= W) continue;
    float *dst = p.partial + (((size_t)(m0 + r) * p.n_heads + h) * p.splits + split) * (HD + 2);
    if (tq == 0) {
      dst[0] = m_run[rr] > -INFINITY ? m_run[rr] * 0.6931471805599453f : -INFINITY;
      dst[1] = l_run[rr];
    }
#pragma unroll
    for (int i = 0; i < HD / 8; ++i)
      *reinterpret_cast<float2 *>(dst + 2 + i * 8 + tq * 2) = make_float2(o[i][rr * 2], o[i][rr * 2 + 1]);
  }
}

typedef CUresult (*EncodeTiledFn3)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// bf16 cache [planes][max_seq][head_dim] as boxes of 64 keys x 64 dims, 128-byte swizzle
int make_kv_tensor_map(TensorMap *out, const void *base, long planes, long max_seq, int head_dim) {
  static EncodeTiledFn3 fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn3>(sym);
  }
  if (!fn) return SJD_ERR_UNSUPPORTED;
  if (((uintptr_t)base & 15u) != 0 || (head_dim != 64 && head_dim != 128)) return SJD_ERR_UNSUPPORTED;
  cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)max_seq, (cuuint64_t)planes};
  cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)max_seq * head_dim * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)KT, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base),
                        dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SJD_OK : SJD_ERR_CUDA;
}

bool attention_mma_supported(int head_dim, int rows_per_seq) { return (head_dim == 64 || head_dim == 128) && rows_per_seq <= 64; }

// With splits > 1 the kernel leaves partial records and the caller merges them with the combine kernel of
// attention.cu; with a single key range it writes `out` (and `hilo`) itself and no merge is needed.
int launch_attention_mma(const TensorMap &kv_map, int plane0, KvLayout kv, const float *q, const int32_t *in_pos,
                         float *partial,
                         float *out, HiLoOut hilo, int *status, int M, int rows_per_seq, int n_heads, int n_kv_heads,
                         int head_dim, int splits, cudaStream_t stream) {
  if (!attention_mma_supported(head_dim, rows_per_seq) || M % rows_per_seq != 0) return SJD_ERR_UNSUPPORTED;
  AttnParams p;
  p.q = q;
  p.in_pos = in_pos;
  p.partial = partial;
  p.out = out;
  p.hilo = hilo;
  p.status = status;
  p.rows_per_seq = rows_per_seq;
  p.n_heads = n_heads;
  p.n_kv_heads = n_kv_heads;
  p.splits = splits;
  p.plane0 = plane0;
  static_assert(KT == KV_PAGE, "one key tile per cache page");
  p.page_table = kv.page_table;
  p.pages_per_seq = kv.pages_per_seq;
  p.layer = kv.layer;
  p.n_layers = kv.n_layers;
  const int threads = 128;   // four warps: 16-row bands x key groups
  const int kg = rows_per_seq <= 16 ? 4 : rows_per_seq <= 32 ? 2 : 1;
  const dim3 grid(n_heads, M / rows_per_seq, splits);
  const CUtensorMap &km = reinterpret_cast<const CUtensorMap &>(kv_map);
  const size_t smem = (size_t)kStagesAttn * 2 * KT * head_dim * 2 + 1024;
  auto launch = [&](auto kernel) -> int {
    SJD_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    SJD_CUDA(launch_kernel(kernel, grid, dim3(threads), smem, stream, km, p));
    SJD_CHECK_LAUNCH();
    return SJD_OK;
  };
  if (head_dim == 128) {
    if (kg == 4) return launch(attention_mma_kernel<128, 4>);
    if (kg == 2) return launch(attention_mma_kernel<128, 2>);
    return launch(attention_mma_kernel<128, 1>);
  }
  if (kg == 4) return launch(attention_mma_kernel<64, 4>);
  if (kg == 2) return launch(attention_mma_kernel<64, 2>);
  return launch(attention_mma_kernel<64, 1>);
}

}  // namespace sjd
