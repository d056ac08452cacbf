// Weight-streaming projection GEMM for sm_100a:  out[m][n] (epilogue)= sum_k X[m][k] * W[n][k]
// (Sec. 4.1 Step 2: the one forward pass over the window; every projection of the decoder).
//
// Shape of the problem: M = batch * window is 8..128 rows, the weight matrix W [N][K] (bf16) is tens
// to hundreds of MB and is read exactly once per step, so the kernel is bound by HBM bandwidth and its
// job is to keep every SM's TMA queue full.
//   * W is the 128-row operand of tcgen05.mma (M = 128), the tokens are the N dimension.  The fp32
//     activations arrive split into two bf16 planes, hi = bf16(x) and lo = bf16(x - hi); both planes
//     are columns of the same MMA (N = 2 * Mp), and the epilogue adds the two halves: activations keep
//     ~16 bits of mantissa at no cost in bytes.
//   * One persistent CTA per SM.  The (tile, k-block) units are split evenly over the CTAs (stream-K);
//     a CTA whose range covers only part of a tile's K range writes an fp32 partial and takes a
//     ticket; the last CTA of a tile adds the partials in CTA order (fixed order: deterministic) and
//     runs the epilogue.  No floating-point atomics.
//   * Warp 0 issues TMA loads (128B-swizzled 128x64 W tiles with an evict-first L2 policy, plus the
//     activation tiles) into a ring of shared-memory stages guarded by mbarriers; warp 1 issues the
//     MMAs into one of two TMEM accumulators and commits to the stage's "empty" barrier; warps 2-5
//     drain the accumulator with tcgen05.ld while the next segment's MMAs run.
//   * Every wait is bounded: after ~2 s a role records an error in the status word and leaves; the
//     CTA still frees its TMEM.
#include <cuda.h>

#include "common.cuh"

namespace sjd {
namespace {

constexpr int TILE_N = 128;   // weight rows per tile (MMA M)
constexpr int TILE_K = 64;    // bf16 elements per k-block = one 128-byte swizzle atom
constexpr int UMMA_K = 16;
constexpr int W_TILE_BYTES = TILE_N * TILE_K * 2;
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr unsigned long long kWaitNs = 2000000000ull;

struct GemmParams {
  void *out;              // fp32 or bf16 [M][ldc]
  int ldc;
  int M;                  // valid token rows
  int Mp;                 // token rows padded to a multiple of 16 (MMA N = 2 * Mp)
  int x_lo_row;           // row of the lo plane inside the activation tensor map
  int n_tiles, k_blocks;  // N / 128, K / 64
  int stages;
  int epilogue;
  float *partials;        // [gridDim.x][2][2 * Mp][128]
  int *tickets;           // [n_tiles], zero on entry and on exit
  int *status;            // device status word (non-zero = a bounded wait ran out)
};

// ---------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

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

// ---------------------------------------------------------------------------------- work split
struct Split {
  long total, q, r;   // units, units per CTA (floor), CTAs with one extra
  __device__ void init(long units, int ctas) {
    total = units;
    q = units / ctas;
    r = units % ctas;
  }
  __device__ long begin(int c) const { return (long)c * q + (c < r ? c : r); }
  __device__ int owner(long u) const {
    const long b = r * (q + 1);
    if (u < b) return (int)(u / (q + 1));
    return (int)(r + (u - b) / (q > 0 ? q : 1));
  }
};

template <int EPI>
__device__ __forceinline__ void store_out(const GemmParams &p, int m, int n, float v) {
  if (m >= p.M) return;
  const size_t idx = (size_t)m * p.ldc + n;
  if (EPI == EPI_STORE_F32) reinterpret_cast<float *>(p.out)[idx] = v;
  else if (EPI == EPI_ADD_F32) reinterpret_cast<float *>(p.out)[idx] += v;
  else reinterpret_cast<__nv_bfloat16 *>(p.out)[idx] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------------- kernel
template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map, const GemmParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_acc_full[2], bar_acc_empty[2];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_last;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int NN = 2 * p.Mp;                                   // MMA N
  const int x_tile_bytes = NN * TILE_K * 2;
  const int stage_bytes = W_TILE_BYTES + x_tile_bytes;
  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  Split sp;
  sp.init((long)p.n_tiles * p.k_blocks, n_cta);
  const long u_begin = sp.begin(cta), u_end = sp.begin(cta + 1);

  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * NN) tmem_cols <<= 1;

  if (tid == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&bar_full[s], 1);
      mbar_init(&bar_empty[s], 1);
    }
    mbar_init(&bar_acc_full[0], 1);
    mbar_init(&bar_acc_full[1], 1);
    mbar_init(&bar_acc_empty[0], 4);
    mbar_init(&bar_acc_empty[1], 4);
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
    if (lane == 0 && u_begin < u_end) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      long it = 0;
      bool ok = true;
      for (long u = u_begin; u < u_end && ok; ++u, ++it) {
        const int tile = (int)(u / p.k_blocks), kb = (int)(u % p.k_blocks);
        const int s = (int)(it % p.stages);
        const uint32_t ph = (uint32_t)((it / p.stages) & 1);
        if (!mbar_wait(&bar_empty[s], ph ^ 1u)) { ok = false; break; }
        uint8_t *dst = smem + (size_t)s * stage_bytes;
        mbar_expect_tx(&bar_full[s], (uint32_t)stage_bytes);
        tma_load_2d(dst, &w_map, kb * TILE_K, tile * TILE_N, &bar_full[s], policy);
        tma_load_2d_nohint(dst + W_TILE_BYTES, &x_map, kb * TILE_K, 0, &bar_full[s]);
        tma_load_2d_nohint(dst + W_TILE_BYTES + x_tile_bytes / 2, &x_map, kb * TILE_K, p.x_lo_row, &bar_full[s]);
      }
      if (!ok) {
        atomicExch(p.status, 1);
        // leave no copy in flight: wait (bounded) for the stages armed most recently
        const long armed = it < p.stages ? it : p.stages;
        for (long j = it - armed; j < it; ++j) mbar_wait(&bar_full[j % p.stages], (uint32_t)((j / p.stages) & 1));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && u_begin < u_end) {
      const uint32_t idesc = umma_idesc_bf16(NN);
      long it = 0;
      int seg = 0;
      bool ok = true;
      for (long u = u_begin; u < u_end && ok; ++seg) {
        const int kb0 = (int)(u % p.k_blocks);
        const long seg_end = min(u_end, u - kb0 + p.k_blocks);
        const int buf = seg & 1;
        if (!mbar_wait(&bar_acc_empty[buf], (uint32_t)(((seg >> 1) & 1) ^ 1))) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_addr = tmem_base + (uint32_t)(buf * NN);
        bool first = true;
        for (; u < seg_end; ++u, ++it) {
          const int s = (int)(it % p.stages);
          const uint32_t ph = (uint32_t)((it / p.stages) & 1);
          if (!mbar_wait(&bar_full[s], ph)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
          const uint32_t b_addr = a_addr + W_TILE_BYTES;
#pragma unroll
          for (int k = 0; k < TILE_K / UMMA_K; ++k) {
            umma_bf16(d_addr, umma_desc_sw128(a_addr + k * UMMA_K * 2), umma_desc_sw128(b_addr + k * UMMA_K * 2), idesc,
                      !(first && k == 0));
          }
          first = false;
          umma_commit(&bar_empty[s]);   // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(&bar_acc_full[buf]);
      }
      if (!ok) atomicExch(p.status, 2);
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (2..5)
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;          // weight row inside the tile
    int seg = 0;
    bool ok = true;
    for (long u = u_begin; u < u_end && ok; ++seg) {
      const int tile = (int)(u / p.k_blocks), kb0 = (int)(u % p.k_blocks);
      const long seg_end = min(u_end, u - kb0 + p.k_blocks);
      const int kb1 = kb0 + (int)(seg_end - u);
      const bool full_tile = (kb0 == 0 && kb1 == p.k_blocks);
      const int buf = seg & 1;
      if (!epilogue_all(mbar_wait(&bar_acc_full[buf], (uint32_t)((seg >> 1) & 1)))) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * NN);
      const int n = tile * TILE_N + row;
      if (full_tile) {
        for (int m0 = 0; m0 < p.Mp; m0 += 16) {
          float hi[16], lo[16];
          tmem_ld16(t_addr + m0, hi);
          tmem_ld16(t_addr + p.Mp + m0, lo);
#pragma unroll
          for (int i = 0; i < 16; ++i) store_out<EPI>(p, m0 + i, n, hi[i] + lo[i]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
      } else {
        // partial K range: park the fp32 partial, take a ticket; the last arrival reduces the tile
        const int which = kb0 > 0 ? 0 : 1;
        float *slot = p.partials + ((size_t)(cta * 2 + which) * NN) * TILE_N;
        for (int c0 = 0; c0 < NN; c0 += 16) {
          float v[16];
          tmem_ld16(t_addr + c0, v);
#pragma unroll
          for (int i = 0; i < 16; ++i) __stcg(&slot[(size_t)(c0 + i) * TILE_N + row], v[i]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
        __threadfence();
        // all four epilogue warps must have stored before the ticket is taken
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int c_lo = sp.owner((long)tile * p.k_blocks), c_hi = sp.owner((long)(tile + 1) * p.k_blocks - 1);
        if (tid == 64) {
          __threadfence();
          const int old = atomicAdd(&p.tickets[tile], 1);
          s_last = (old == c_hi - c_lo);
          if (s_last) p.tickets[tile] = 0;
          __threadfence();
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (s_last) {
          for (int m0 = 0; m0 < p.Mp; m0 += 16) {
            float acc[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = 0.0f;
            for (int half = 0; half < 2; ++half) {
              for (int c = c_lo; c <= c_hi; ++c) {
                const int wch = sp.begin(c) > (long)tile * p.k_blocks ? 0 : 1;
                const float *src = p.partials + ((size_t)(c * 2 + wch) * NN) * TILE_N;
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] += __ldcg(&src[(size_t)(half * p.Mp + m0 + i) * TILE_N + row]);
              }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) store_out<EPI>(p, m0 + i, n, acc[i]);
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");   // s_last is reused by the next segment
      }
      u = seg_end;
    }
    if (!ok) atomicExch(p.status, 3);
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
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SJD_OK : SJD_ERR_CUDA;
}

bool gemm_tc_supported(int M, int N, int K) { return M >= 1 && M <= 128 && N % TILE_N == 0 && K % TILE_K == 0; }

size_t gemm_tc_partial_floats(int n_ctas, int max_rows) {
  const int mp = (max_rows + 15) / 16 * 16;
  return (size_t)n_ctas * 2 * (2 * mp) * TILE_N;
}

int launch_gemm_tc(const TensorMap &w_map, const TensorMap &x_map, int x_lo_row, void *out, int ldc, int M, int N, int K,
                   int epilogue, float *partials, int *tickets, int *status, int n_ctas, cudaStream_t stream) {
  if (!gemm_tc_supported(M, N, K)) return SJD_ERR_UNSUPPORTED;
  GemmParams p;
  p.out = out;
  p.ldc = ldc;
  p.M = M;
  p.Mp = (M + 15) / 16 * 16;
  p.x_lo_row = x_lo_row;
  p.n_tiles = N / TILE_N;
  p.k_blocks = K / TILE_K;
  p.epilogue = epilogue;
  p.partials = partials;
  p.tickets = tickets;
  p.status = status;
  const int stage_bytes = W_TILE_BYTES + 2 * p.Mp * TILE_K * 2;
  int stages = (200 * 1024) / stage_bytes;
  stages = stages > kMaxStages ? kMaxStages : stages;
  if (stages < 2) return SJD_ERR_UNSUPPORTED;
  p.stages = stages;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  const CUtensorMap &wm = reinterpret_cast<const CUtensorMap &>(w_map);
  const CUtensorMap &xm = reinterpret_cast<const CUtensorMap &>(x_map);
#define SJD_LAUNCH_TC(E)                                                                                         \
  do {                                                                                                           \
    SJD_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));   \
    gemm_tc_kernel<E><<<n_ctas, kThreads, smem, stream>>>(wm, xm, p);                                            \
  } while (0)
  if (epilogue == EPI_STORE_F32) SJD_LAUNCH_TC(EPI_STORE_F32);
  else if (epilogue == EPI_ADD_F32) SJD_LAUNCH_TC(EPI_ADD_F32);
  else if (epilogue == EPI_STORE_T) SJD_LAUNCH_TC(EPI_STORE_T);
  else return SJD_ERR_BAD_ARG;
#undef SJD_LAUNCH_TC
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

}  // namespace sjd
