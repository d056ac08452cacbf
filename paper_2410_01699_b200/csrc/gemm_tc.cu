// Weight-streaming projection GEMM for sm_100a:  P[s][m][n] = sum_{k in split s} X[m][k] * W[n][k]
// (Sec. 4.1 Step 2: the one forward pass over the window; every projection of the decoder).
//
// Shape of the problem: M = batch * window is 8..128 rows, the weight matrices (bf16) are tens to
// hundreds of MB and are read exactly once per step, so the kernel is bound by HBM bandwidth and its
// job is to keep every SM's TMA queue full.  Larger M (batches of images with wide windows, up to
// 1024 rows) is cut into token slabs of at most 128 rows; the CTAs of the slabs of one weight tile
// are neighbours in the grid, so the tile comes from HBM once and from L2 for the other slabs.  With
// several slabs the kernel is bound by the tensor pipe (both activation planes are multiplied) and, in
// this tiling, by shared-memory bandwidth: a 128 x 256 MMA tile moves 96 KB through shared memory per 512
// tensor clocks.  (Measured and removed: two adjacent weight tiles per CTA against one activation tile,
// 10-15 % slower than two independent CTAs per SM.)
//   * W is the 128-row operand of tcgen05.mma (M = 128), the tokens are the N dimension.  The fp32
//     activations arrive split into two bf16 planes, hi = bf16(x) and lo = bf16(x - hi); both planes
//     are columns of the same MMA (N = 2 * Mp), and the epilogue adds the two halves: activations keep
//     ~16 bits of mantissa at no cost in weight bytes.  (Multiplying the hi plane alone, i.e. plain
//     bf16 activations, would halve the tensor work of the many-row case but misses the 2e-2 logits
//     tolerance at d_model 4096 already after two layers: 4.0e-2.  So both planes, always, and the
//     useful tensor throughput of the many-row case cannot pass half the peak.)
//   * One CTA per (128-row weight tile, K split); two CTAs are resident per SM.  A launch covers up to
//     three weight matrices that share the activation operand (Q|K|V, gate|up), so their tiles form
//     one grid.  With more than one K split every CTA writes an fp32 partial plane; the consumer
//     kernel (residual + RMSNorm, RoPE + cache append, SwiGLU, or a plain sum) adds the planes in
//     split order: deterministic, no atomics, no serial reduction tail inside the GEMM.
//   * Warp 0 issues TMA loads (128B-swizzled 128x64 W tiles with an evict-first L2 policy, plus the
//     activation tiles) into a ring of shared-memory stages guarded by mbarriers; warp 1 issues the
//     MMAs into a TMEM accumulator and commits to the stage's "empty" barrier; warps 2-5 drain the
//     accumulator with tcgen05.ld and store.
//   * Every wait is bounded: after ~2 s a role records an error in the status word and leaves; the
//     CTA still frees its TMEM.
#include <cuda.h>
#include <string.h>

#include "common.cuh"

namespace sjd {
SJD_TIMELINE_TU(gemm)
namespace {

constexpr int TILE_N = 128;   // weight rows per tile (MMA M)
constexpr int TILE_K = 64;    // bf16 elements per k-block = one 128-byte swizzle atom
constexpr int UMMA_K = 16;
constexpr int W_TILE_BYTES = TILE_N * TILE_K * 2;
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
// tunables (defaults chosen by measurement on B200)
#ifndef SJD_GEMM_SMEM_BUDGET
#define SJD_GEMM_SMEM_BUDGET (100 * 1024)   // ring bytes per CTA when two CTAs share an SM
#endif
#ifndef SJD_GEMM_DEEP_RING
#define SJD_GEMM_DEEP_RING 1                // double the ring when the grid has at most one CTA per SM
#endif
#ifndef SJD_GEMM_L2_PROMO
#define SJD_GEMM_L2_PROMO CU_TENSOR_MAP_L2_PROMOTION_L2_256B
#endif
#ifndef SJD_GEMM_MIN_KB
#define SJD_GEMM_MIN_KB 8                   // fewest k-blocks (of 16 KB of weights) a CTA should stream (8: the O projection runs 32 x 8 CTAs whose whole share fits the prefetched ring; 3.51 against 3.54 ms per step with 16)
#endif
#ifndef SJD_GEMM_CTAS_PER_SM
#define SJD_GEMM_CTAS_PER_SM 2
#endif
constexpr int kSmemBudget = SJD_GEMM_SMEM_BUDGET;
constexpr unsigned long long kWaitNs = 2000000000ull;

struct GemmParams {
  void *out;              // fp32 planes [splits][M][ldc], or bf16 [M][ldc] when store_bf16
  size_t plane_stride;    // elements between planes
  int ldc;
  int M;                  // valid token rows
  int Mp;                 // token rows of one slab, a multiple of 16 (MMA N = 2 * Mp: hi and lo plane)
  int n_slabs;            // token slabs; CTA blockIdx.x = weight tile * n_slabs + slab
  int x_lo_row;           // row of the lo plane inside the activation tensor map
  int k_blocks, splits;   // K / 64, K splits (gridDim.y)
  int tile_end[3];        // matrix j owns tiles [tile_end[j-1], tile_end[j])
  int col_off[3];         // first output column of matrix j
  int stages;
  int store_bf16;
  int *status;            // device status word (non-zero = a bounded wait ran out)
  const float *ss_part;   // optional [M][n_part] partial sums of squares: rows are scaled by
  int n_part;             //   1 / sqrt(sum_j ss_part[m][j] * inv_d + eps) before they are stored
  float inv_d, eps;
  int tile_rows;          // weight rows a tile really holds (<= 128; the rest of the MMA's 128 rows is idle)
  int n_out[3];           // output features of matrix j (the last tile of a matrix may be partial)
  // gate|up mode (template GU): tile t holds rows [t*tile_rows, (t+1)*tile_rows) of the gate matrix in MMA
  // rows 0.. and the same rows of the up matrix in MMA rows 64..; the epilogue stores
  // silu(gate) * up as bf16 hi/lo planes [M][F]
  __nv_bfloat16 *act_hi;
  size_t act_lo_off;
  int F;
};

// ---------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false if the barrier did not flip within kWaitNs.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > kWaitNs) return false;
  }
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_nohint(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                          // 128-byte swizzle
  return d;
}
// instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t *r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// AND of a predicate over the 128 epilogue threads (named barrier 1): keeps their control flow uniform
__device__ __forceinline__ bool epilogue_all(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

// ---------------------------------------------------------------------------------- kernel
// GU: the gate|up launch that applies SwiGLU in its epilogue
template <bool GU>
__global__ void __launch_bounds__(kThreads, 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap w_map0, const __grid_constant__ CUtensorMap w_map1,
               const __grid_constant__ CUtensorMap w_map2, const __grid_constant__ CUtensorMap x_map, const GemmParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_acc_full;
  __shared__ uint32_t s_tmem_base;
  __shared__ float s_scale[TILE_N];   // per-row output scales of this CTA's token slab (epilogue)

  constexpr int WT = 1;   // weight tiles (accumulators) per CTA
  constexpr int XP = 2;   // activation planes multiplied: hi and lo
  pdl_trigger();   // the next kernel in the stream may be scheduled as soon as every CTA got here
  SJD_TL(TL_GEMM, 0, threadIdx.x == 0);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = (int)blockIdx.x / p.n_slabs, split = blockIdx.y;
  const int tile = unit * WT;                         // first weight tile of this CTA
  const int m_base = ((int)blockIdx.x - unit * p.n_slabs) * p.Mp;   // first token row of this CTA's slab
  const int NN = XP * p.Mp;                          // MMA N
  const int x_tile_bytes = NN * TILE_K * 2;
  const int w_bytes = WT * W_TILE_BYTES;
  const int stage_bytes = w_bytes + x_tile_bytes;
  const int R = p.tile_rows;
  const uint32_t stage_tx = (uint32_t)((GU ? 2 : WT) * R * TILE_K * 2 + x_tile_bytes);   // bytes the copies of a stage deliver
  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  // which weight matrix this tile belongs to
  const int mat = GU ? 0 : (tile < p.tile_end[0] ? 0 : (tile < p.tile_end[1] ? 1 : 2));
  const CUtensorMap *w_map = mat == 0 ? &w_map0 : (mat == 1 ? &w_map1 : &w_map2);
  const int tile_in_mat = tile - (mat == 0 ? 0 : p.tile_end[mat - 1]);
  // this CTA's k-blocks
  const int kb_begin = (int)(((long)split * p.k_blocks) / p.splits);
  const int kb_end = (int)(((long)(split + 1) * p.k_blocks) / p.splits);
  const int n_kb = kb_end - kb_begin;

  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < WT * NN) tmem_cols <<= 1;

  if (tid == 0) {
    tma_prefetch_desc(w_map);
    tma_prefetch_desc(&x_map);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bar_full[s], 1);
      mbar_init(&bar_empty[s], 1);
    }
    mbar_init(&bar_acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      // The weights do not depend on the preceding kernel: fill the ring with W tiles right away,
      // then wait for the predecessor before fetching the activation tiles it produced.
      const int pre = n_kb < p.stages ? n_kb : p.stages;
      for (int i = 0; i < pre; ++i) {
        mbar_expect_tx(&bar_full[i], stage_tx);
        if (GU) {
          tma_load_2d(smem + i * stage_bytes, &w_map0, (kb_begin + i) * TILE_K, tile * R, &bar_full[i], policy);
          tma_load_2d(smem + i * stage_bytes + W_TILE_BYTES / 2, &w_map1, (kb_begin + i) * TILE_K, tile * R, &bar_full[i],
                      policy);
        } else {
#pragma unroll
          for (int j = 0; j < WT; ++j)
            tma_load_2d(smem + i * stage_bytes + j * W_TILE_BYTES, w_map, (kb_begin + i) * TILE_K, (tile_in_mat + j) * R,
                        &bar_full[i], policy);
        }
      }
      SJD_TL(TL_GEMM, 3, true);
      pdl_wait();
      SJD_TL(TL_GEMM, 1, true);
      for (int i = 0; i < pre; ++i) {
        uint8_t *dst = smem + i * stage_bytes;
        const int kcol = (kb_begin + i) * TILE_K;
        tma_load_2d_nohint(dst + w_bytes, &x_map, kcol, m_base, &bar_full[i]);
        if (XP == 2)
          tma_load_2d_nohint(dst + w_bytes + x_tile_bytes / 2, &x_map, kcol, p.x_lo_row + m_base, &bar_full[i]);
      }
      int s = pre == p.stages ? 0 : pre;
      uint32_t ph = pre == p.stages ? 1u : 0u;
      bool ok = true;
      int it = pre;
      for (; it < n_kb; ++it) {
        if (!mbar_wait(&bar_empty[s], ph ^ 1u)) { ok = false; break; }
        uint8_t *dst = smem + s * stage_bytes;
        const int kcol = (kb_begin + it) * TILE_K;
        mbar_expect_tx(&bar_full[s], stage_tx);
        if (GU) {
          tma_load_2d(dst, &w_map0, kcol, tile * R, &bar_full[s], policy);
          tma_load_2d(dst + W_TILE_BYTES / 2, &w_map1, kcol, tile * R, &bar_full[s], policy);
        } else {
#pragma unroll
          for (int j = 0; j < WT; ++j)
            tma_load_2d(dst + j * W_TILE_BYTES, w_map, kcol, (tile_in_mat + j) * R, &bar_full[s], policy);
        }
        tma_load_2d_nohint(dst + w_bytes, &x_map, kcol, m_base, &bar_full[s]);
        if (XP == 2)
          tma_load_2d_nohint(dst + w_bytes + x_tile_bytes / 2, &x_map, kcol, p.x_lo_row + m_base, &bar_full[s]);
        if (++s == p.stages) { s = 0; ph ^= 1u; }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        // leave no copy in flight: wait (bounded) for the stages armed most recently
        const int armed = it < p.stages ? it : p.stages;
        for (int j = it - armed; j < it; ++j) mbar_wait(&bar_full[j % p.stages], (uint32_t)((j / p.stages) & 1));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(NN);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int it = 0; it < n_kb; ++it) {
        if (!mbar_wait(&bar_full[s], ph)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + s * stage_bytes);
        const uint32_t b_addr = a_addr + w_bytes;
#pragma unroll
        for (int k = 0; k < TILE_K / UMMA_K; ++k) {
          const uint64_t bdesc = umma_desc_sw128(b_addr + k * UMMA_K * 2);
  #pragma unroll
        for (int j = 0; j < WT; ++j)
            umma_bf16(tmem_base + j * NN, umma_desc_sw128(a_addr + j * W_TILE_BYTES + k * UMMA_K * 2), bdesc, idesc,
                      !(it == 0 && k == 0));
        }
        umma_commit(&bar_empty[s]);   // frees the stage once these MMAs have read it
        if (++s == p.stages) { s = 0; ph ^= 1u; }
      }
      if (ok) umma_commit(&bar_acc_full);
      else atomicExch(p.status, 2);
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (2..5)
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;          // weight row inside the tile
    const bool ok = epilogue_all(mbar_wait(&bar_acc_full, 0));
    if (ok) {
      tc_fence_after();
      pdl_wait();   // the planes may still be read, and the row scales written, by the preceding kernel
      float *plane = reinterpret_cast<float *>(p.out) + (size_t)split * p.plane_stride;
      __nv_bfloat16 *out_bf16 = reinterpret_cast<__nv_bfloat16 *>(p.out);
      if (p.ss_part || GU) {   // RMS scale of each token row, once per CTA (epilogue thread e: row m_base + e)
        const int e = tid - 64, m = m_base + e;
        float sc = 1.0f;
        if (p.ss_part && e < p.Mp && m < p.M) {
          float tot = 0.0f;
          for (int jj = 0; jj < p.n_part; ++jj) tot += __ldg(p.ss_part + (size_t)m * p.n_part + jj);
          sc = rsqrtf(tot * p.inv_d + p.eps);
        }
        s_scale[e] = sc;
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
      if (GU) {
        // MMA rows 0..63 hold gate features, rows 64..127 the same features of the up matrix.  The warps
        // that read the up rows (TMEM lane quarters 2, 3) pass their values through shared memory (the
        // ring is idle by now) to the warps that read the gate rows, which finish the activation.
        // Every epilogue warp parks its 32 accumulator rows (scaled) in shared memory, row-major with an odd
        // stride; after one barrier the 128 threads share the activation work: thread t finishes feature
        // t % 64 for every second token, so that a warp's stores cover 32 adjacent features of one token.
        float *ex = reinterpret_cast<float *>(smem);   // [128][Mp + 1]
        const int ldx = p.Mp + 1;
        const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        for (int m0 = 0; m0 < p.Mp; m0 += 16) {
          uint32_t hi[16], lo[16];
          tmem_ld16_issue(t_addr + m0, hi);
          tmem_ld16_issue(t_addr + p.Mp + m0, lo);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i)
            ex[row * ldx + m0 + i] = (__uint_as_float(hi[i]) + __uint_as_float(lo[i])) * s_scale[m0 + i];
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int e = tid - 64, fr = e & 63;
        const int f = tile * R + fr;
        if (fr < R && f < p.F) {
          for (int mm = e >> 6; mm < p.Mp; mm += 2) {
            const int m = m_base + mm;
            if (m >= p.M) break;
            const float g = ex[fr * ldx + mm], u = ex[(64 + fr) * ldx + mm];
            const float v = g / (1.0f + expf(-g)) * u;
            const __nv_bfloat16 vh = __float2bfloat16_rn(v);
            p.act_hi[(size_t)m * p.F + f] = vh;
            p.act_hi[p.act_lo_off + (size_t)m * p.F + f] = __float2bfloat16_rn(v - __bfloat162float(vh));
          }
        }
      } else {
#pragma unroll
      for (int j = 0; j < WT; ++j)                               // accumulator
      for (int m0 = 0; m0 < p.Mp; m0 += 16) {                    // first token row of the chunk
        const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + j * NN;
        const int n_local = (tile_in_mat + j) * R + row;
        const int n = p.col_off[mat] + n_local;
        const bool live = row < R && n_local < p.n_out[mat];
        uint32_t hi[16], lo[16];
        tmem_ld16_issue(t_addr + m0, hi);
        if (XP == 2) {
          tmem_ld16_issue(t_addr + p.Mp + m0, lo);
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) lo[i] = 0u;
        }
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int m = m_base + m0 + i;
          if (live && m < p.M) {
            float v = __uint_as_float(hi[i]) + __uint_as_float(lo[i]);
            if (p.ss_part) v *= s_scale[m0 + i];
            if (p.store_bf16) out_bf16[(size_t)m * p.ldc + n] = __float2bfloat16_rn(v);
            else plane[(size_t)m * p.ldc + n] = v;
          }
        }
      }
      }
    } else if (tid == 64) {
      atomicExch(p.status, 3);
    }
    SJD_TL(TL_GEMM, 2, tid == 64);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// plain sum of split planes (sjd_gemm): out[m][n] (+)= sum_s P[s][m][n]
__global__ void sum_planes_kernel(const float *__restrict__ planes, size_t plane_stride, int splits, float *__restrict__ out,
                                  size_t total, int accumulate) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    float acc = 0.0f;
    for (int s = 0; s < splits; ++s) acc += planes[(size_t)s * plane_stride + i];
    out[i] = accumulate ? out[i] + acc : acc;
  }
}

}  // namespace

// bf16 row-major [rows][cols] matrix viewed as boxes of box_rows x 64 columns with 128-byte swizzle
int make_tensor_map_bf16(TensorMap *out, const void *base, long rows, long cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return SJD_ERR_UNSUPPORTED;
  if (((uintptr_t)base & 15u) != 0 || (cols * 2) % 16 != 0 || box_rows < 1 || box_rows > 256) return SJD_ERR_UNSUPPORTED;
  static_assert(sizeof(TensorMap) == sizeof(CUtensorMap), "tensor map size");
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)TILE_K, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base),
                        dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        SJD_GEMM_L2_PROMO, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SJD_OK : SJD_ERR_CUDA;
}

bool gemm_tc_supported(int M, int N, int K) { return M >= 1 && M <= 1024 && N % TILE_N == 0 && K % TILE_K == 0; }

// How M token rows are laid over the MMA N dimension (at most 256 columns per accumulator, two per token
// row: hi and lo plane): slabs of at most 128 rows.
GemmTcPlan gemm_tc_plan(int M) {
  GemmTcPlan pl;
  pl.n_slabs = (M + 127) / 128;
  const int per = (M + pl.n_slabs - 1) / pl.n_slabs;
  pl.slab_rows = (per + 15) / 16 * 16;
  return pl;
}

// K splits for a launch of `tiles` weight tiles: a single wave of the resident CTAs (two per SM), at least 16 k-blocks (256 KB of weights) per CTA so that
// set-up and drain stay small next to the streaming
int gemm_tc_splits(const GemmTcPlan &pl, int tiles, int k_blocks, int n_sms) {
  const int ctas = tiles * pl.n_slabs;
  int s = (SJD_GEMM_CTAS_PER_SM * n_sms) / (ctas > 0 ? ctas : 1);
  const int cap = k_blocks / SJD_GEMM_MIN_KB > 1 ? k_blocks / SJD_GEMM_MIN_KB : 1;
  s = s > cap ? cap : s;
  s = s > 16 ? 16 : s;
  return s < 1 ? 1 : s;
}

int launch_gemm_tc(const GemmTcCall &g, cudaStream_t stream) {
  if (g.n_mats < 1 || g.n_mats > 3 || g.splits < 1) return SJD_ERR_BAD_ARG;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  const bool gu = g.act_hi != nullptr;
  const int R = g.tile_rows > 0 ? g.tile_rows : TILE_N;
  if (R > TILE_N || (gu && (R > TILE_N / 2 || g.n_mats != 2 || g.n_out[0] != g.n_out[1] || g.splits != 1)))
    return SJD_ERR_BAD_ARG;
  int tiles = 0;
  for (int j = 0; j < 3; ++j) {
    if (j < g.n_mats && !(gu && j == 1)) {
      if (g.M < 1 || g.M > 1024 || g.K % TILE_K != 0 || g.n_out[j] < 1) return SJD_ERR_UNSUPPORTED;
      if (R == TILE_N && g.n_out[j] % TILE_N != 0) return SJD_ERR_UNSUPPORTED;
      tiles += (g.n_out[j] + R - 1) / R;
    }
    p.tile_end[j] = tiles;
    p.col_off[j] = j < g.n_mats ? g.col_off[j] : 0;
    p.n_out[j] = j < g.n_mats ? g.n_out[j] : 0;
  }
  if (g.store_bf16 && g.splits != 1) return SJD_ERR_BAD_ARG;
  p.out = g.out;
  p.plane_stride = g.plane_stride;
  p.ldc = g.ldc;
  const GemmTcPlan pl = gemm_tc_plan(g.M);
  p.M = g.M;
  p.Mp = pl.slab_rows;
  p.n_slabs = pl.n_slabs;
  p.x_lo_row = g.x_lo_row;
  p.k_blocks = g.K / TILE_K;
  p.splits = g.splits;
  p.store_bf16 = g.store_bf16;
  p.status = g.status;
  p.ss_part = g.ss_part;
  p.n_part = g.n_part;
  p.inv_d = g.inv_d;
  p.eps = g.eps;
  p.tile_rows = R;
  p.act_hi = g.act_hi;
  p.act_lo_off = g.act_lo_off;
  p.F = gu ? g.n_out[0] : 0;
  const int stage_bytes = W_TILE_BYTES + 2 * p.Mp * TILE_K * 2;
  const int ctas = tiles * p.n_slabs;
  // one CTA per SM or fewer: give each the deeper ring
  const int budget =
      (SJD_GEMM_DEEP_RING && g.n_sms > 0 && ctas * g.splits <= g.n_sms) ? 2 * kSmemBudget : kSmemBudget;
  int stages = budget / stage_bytes;
  stages = stages > kMaxStages ? kMaxStages : stages;
  if (stages < 2) return SJD_ERR_UNSUPPORTED;
  p.stages = stages;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  const CUtensorMap &w0 = reinterpret_cast<const CUtensorMap &>(*g.w_map[0]);
  const CUtensorMap &w1 = reinterpret_cast<const CUtensorMap &>(*g.w_map[g.n_mats > 1 ? 1 : 0]);
  const CUtensorMap &w2 = reinterpret_cast<const CUtensorMap &>(*g.w_map[g.n_mats > 2 ? 2 : 0]);
  const CUtensorMap &xm = reinterpret_cast<const CUtensorMap &>(*g.x_map);
  // opt in to > 48 KB of dynamic shared memory, once per device
  static bool configured[64] = {};
  int dev = 0;
  SJD_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SJD_ERR_UNSUPPORTED;
  if (!configured[dev]) {
    const int max_dyn = 2 * kSmemBudget + 2048;
    SJD_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn));
    SJD_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn));
    configured[dev] = true;
  }
  const dim3 grid(ctas, g.splits);
  if (gu)
    SJD_CUDA(launch_kernel(gemm_tc_kernel<true>, grid, dim3(kThreads), smem, stream, w0, w1, w2, xm, p));
  else
    SJD_CUDA(launch_kernel(gemm_tc_kernel<false>, grid, dim3(kThreads), smem, stream, w0, w1, w2, xm, p));
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

int launch_sum_planes(const float *planes, size_t plane_stride, int splits, float *out, size_t total, int accumulate,
                      cudaStream_t stream) {
  const int blocks = (int)((total + 255) / 256 < 2368 ? (total + 255) / 256 : 2368);
  sum_planes_kernel<<<blocks, 256, 0, stream>>>(planes, plane_stride, splits, out, total, accumulate);
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

}  // namespace sjd
