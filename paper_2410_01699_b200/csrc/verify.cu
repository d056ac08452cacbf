// Fused verify-and-resample kernel (Sec. 4.1 Step 3, Eqs. 1-3) and the window slide of Step 4.
//
// One thread block per window row.  A block
//   1. (only when the draft's law is a logits row whose statistics are not cached) stages the
//      previous-iteration row in shared memory and computes its top-k threshold and softmax
//      denominator;
//   2. stages this iteration's row, finds the top-k threshold with an exact MSB-first radix select
//      on order-preserving keys (ties at the threshold are all kept), computes the softmax
//      denominator as per-chunk partial sums in token order;
//   3. evaluates p(d)/q(d) against the Philox uniform (Eq. 1), draws the re-draft token from p by
//      inverse CDF (Eq. 3) and, if the row rejected, the residual token from max(0, p - q) (Eq. 2);
//   4. publishes a 32-byte record.  The last block of a sequence to finish (an atomic ticket, no
//      waiting) scans the records left to right, fixes the accepted prefix and slides the window
//      (Step 4, Sec. 4.2).
// Logits are read once from HBM; later passes hit the shared-memory copy.  Rows too large for
// shared memory are re-read through L2.  No floating-point atomics: every sum has a fixed order.
//
// bf16 rows of at most 65536 entries take a leaner route (fast_row): the block holds the row in
// registers (eight 16-byte vectors per thread), finds the maximum with packed bf16 instructions,
// histograms once the distance of every entry below the maximum in bf16 codes (exact for the 4095
// codes next to it), walks that histogram per warp to the exact threshold, and forms chunk sums,
// prefix and inverse-CDF searches from registers with every table search done by each warp for itself
// (about a dozen block barriers per row).  Rows with NaN/+inf, without a finite entry, with the
// K-th largest entry more than 4095 codes below the maximum (e.g. a positive maximum and a negative
// threshold) or next to +-0 use the general route above; both routes produce the same threshold and
// the same weights.  Longer bf16 rows (the 184320-entry head) take the same route streamed: a full block
// passes the row through its registers in segments of 65536 entries, once per phase (long_statistics).
#include <float.h>

#include <type_traits>

#include "common.cuh"

namespace sjd {
SJD_TIMELINE_TU(verify)
namespace {

#ifndef SJD_VERIFY_MIN_BLOCKS
#define SJD_VERIFY_MIN_BLOCKS 4   // resident blocks per SM the 256-thread variant is compiled for (64 registers)
#endif
constexpr int kMaxChunks = 1024;   // 32 vectors of 16 bytes per chunk
constexpr int kMaxThreads = 1024;

// ------------------------------------------------------------------------------------ elements
template <typename T>
struct Elt;

template <>
struct Elt<float> {
  static constexpr int VEC = 4;
  static constexpr int KEYBITS = 32;
  static constexpr uint32_t NEG_INF = 0xFF800000u;
  __device__ static __forceinline__ uint32_t get(const uint4 &v, int t) {
    return t == 0 ? v.x : t == 1 ? v.y : t == 2 ? v.z : v.w;
  }
  __device__ static __forceinline__ void set(uint4 &v, int t, uint32_t b) {
    if (t == 0) v.x = b; else if (t == 1) v.y = b; else if (t == 2) v.z = b; else v.w = b;
  }
  __device__ static __forceinline__ uint32_t load_bits(const float *p) { return __float_as_uint(__ldg(p)); }
  __device__ static __forceinline__ bool bad(uint32_t b) {
    return (b & 0x7FFFFFFFu) > 0x7F800000u || b == 0x7F800000u;
  }
  __device__ static __forceinline__ uint32_t key(uint32_t b) { return (b & 0x80000000u) ? ~b : (b | 0x80000000u); }
  __device__ static __forceinline__ uint32_t unkey(uint32_t k) { return (k & 0x80000000u) ? (k ^ 0x80000000u) : ~k; }
  __device__ static __forceinline__ float val(uint32_t b) { return __uint_as_float(b); }
  __device__ static __forceinline__ uint32_t bits(float x) { return __float_as_uint(x); }
};

template <>
struct Elt<__nv_bfloat16> {
  static constexpr int VEC = 8;
  static constexpr int KEYBITS = 16;
  static constexpr uint32_t NEG_INF = 0xFF80u;
  __device__ static __forceinline__ uint32_t word(const uint4 &v, int i) {
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
  }
  __device__ static __forceinline__ uint32_t get(const uint4 &v, int t) {
    return (word(v, t >> 1) >> ((t & 1) * 16)) & 0xFFFFu;
  }
  __device__ static __forceinline__ void set(uint4 &v, int t, uint32_t b) {
    const uint32_t sh = (t & 1) * 16;
    const uint32_t m = ~(0xFFFFu << sh);
    const int i = t >> 1;
    if (i == 0) v.x = (v.x & m) | (b << sh);
    else if (i == 1) v.y = (v.y & m) | (b << sh);
    else if (i == 2) v.z = (v.z & m) | (b << sh);
    else v.w = (v.w & m) | (b << sh);
  }
  __device__ static __forceinline__ uint32_t load_bits(const __nv_bfloat16 *p) {
    return (uint32_t)__ldg(reinterpret_cast<const unsigned short *>(p));
  }
  __device__ static __forceinline__ bool bad(uint32_t b) { return (b & 0x7FFFu) > 0x7F80u || b == 0x7F80u; }
  __device__ static __forceinline__ uint32_t key(uint32_t b) { return (b & 0x8000u) ? (~b & 0xFFFFu) : (b | 0x8000u); }
  __device__ static __forceinline__ uint32_t unkey(uint32_t k) { return (k & 0x8000u) ? (k ^ 0x8000u) : (~k & 0xFFFFu); }
  __device__ static __forceinline__ float val(uint32_t b) { return __uint_as_float(b << 16); }
  __device__ static __forceinline__ uint32_t bits(float x) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x)); }
};

// ------------------------------------------------------------------------------------ scratch
struct Scratch {
  double chunk_excl[kMaxChunks + 1];  // exclusive prefix of chunk sums; [NC] = total
  float chunk_sum[kMaxChunks];
  alignas(16) uint32_t hist12[4096];              // register-resident route: histogram of code distances below the row maximum
  uint32_t hist[256];
  uint32_t redu[32];
  uint32_t d_bits[2];                 // register-resident route: bits of the q / p row's entry at the draft token
  uint32_t sel_bin, count_above, bad;
  int sel_chunk, last_chunk;
  int tok;
  float tok_w;
  int is_last;
  // new window slots whose token is drawn from a logits row (Sec. 4.2 (c), (d)): filled by draw_fresh_slots,
  // consumed by finalize_sequence; row -1: no row, the slot is a uniform random token; kind SJD_Q_ROW: a row
  // of this pass's buffer, SJD_Q_RING: a slot of the ring of retained rows
  int fresh_tok[64], fresh_row[64], fresh_kind[64];
  float fresh_q[64];
};

// A logits row seen as 16-byte vectors aligned in global memory: vector j holds elements
// j*VEC - off .. j*VEC - off + VEC - 1; elements outside [0, V) read as -inf.
template <typename T>
struct Row {
  const T *g;
  const T *g2;   // classifier-free guidance: the unconditional stream's row (g is the conditional one), or null
  float gw;      // guidance weight
  int V, off, NV;
  const uint4 *s;  // shared-memory copy (sanitised), or null

  __device__ void init(const T *row, int v, const T *row_uncond = nullptr, float weight = 0.0f) {
    g = row;
    g2 = row_uncond;
    gw = weight;
    V = v;
    off = (int)(((uintptr_t)row & 15u) / sizeof(T));
    NV = (off + v + Elt<T>::VEC - 1) / Elt<T>::VEC;
    s = nullptr;
  }
  // bits of element i as the verification sees it: the stored logit, or under guidance the mix
  // l_u + w * (l_c - l_u) (one subtraction, one fused multiply-add in fp32) rounded to the storage dtype
  __device__ __forceinline__ uint32_t raw_bits(int i) const {
    const uint32_t b = Elt<T>::load_bits(g + i);
    if (!g2) return b;
    const float c = Elt<T>::val(b), u = Elt<T>::val(Elt<T>::load_bits(g2 + i));
    return Elt<T>::bits(fmaf(gw, c - u, u));
  }
  // sanitised vector straight from global memory
  __device__ __forceinline__ uint4 load_global(int j, uint32_t &bad) const {
    using E = Elt<T>;
    const int i0 = j * E::VEC - off;
    uint4 v;
    if (!g2 && i0 >= 0 && i0 + E::VEC <= V) {
      v = __ldg(reinterpret_cast<const uint4 *>(g + i0));
    } else {
      v = make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int t = 0; t < E::VEC; ++t) {
        const int i = i0 + t;
        E::set(v, t, (i >= 0 && i < V) ? raw_bits(i) : E::NEG_INF);
      }
    }
#pragma unroll
    for (int t = 0; t < E::VEC; ++t) {
      if (E::bad(E::get(v, t))) {
        E::set(v, t, E::NEG_INF);
        bad = 1;
      }
    }
    return v;
  }
  __device__ __forceinline__ uint4 vec(int j) const {
    uint32_t ignore = 0;
    return s ? s[j] : load_global(j, ignore);
  }
  // sanitised bits of element i (0 <= i < V)
  __device__ __forceinline__ uint32_t element(int i) const {
    if (s) {   // the staged copy is already sanitised
      if (sizeof(T) == 2) return (uint32_t) reinterpret_cast<const unsigned short *>(s)[i + off];
      return reinterpret_cast<const uint32_t *>(s)[i + off];
    }
    const uint32_t b = raw_bits(i);
    return Elt<T>::bad(b) ? Elt<T>::NEG_INF : b;
  }
};

// weight of one element under a row's statistics: exp((x - xmax)/T) inside the top-k set, else 0
// 2^x for x <= 0 (hardware approximation, 2 ulp; results below the normal range flush to 0)
__device__ __forceinline__ float exp2_neg(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <typename T>
struct PWeight {
  uint32_t tau_key;
  float xmax, scale;   // scale = log2(e) / T
  bool degenerate;  // no finite entry: all mass on token 0
  __device__ void init(const RowStats &st, float inv_temperature) {
    tau_key = st.tau_key;
    xmax = st.xmax;
    scale = inv_temperature * 1.4426950408889634f;
    degenerate = !(st.xmax > -FLT_MAX);
  }
  __device__ __forceinline__ float one(uint32_t bits, int idx) const {
    if (degenerate) return idx == 0 ? 1.0f : 0.0f;
    return Elt<T>::key(bits) >= tau_key ? exp2_neg((Elt<T>::val(bits) - xmax) * scale) : 0.0f;
  }
};

template <typename T>
struct PRowWeights {  // functor: weights of vector j of a row
  Row<T> row;
  PWeight<T> pw;
  __device__ __forceinline__ void operator()(int j, float *w) const {
    const uint4 v = row.vec(j);
    const int i0 = j * Elt<T>::VEC - row.off;
#pragma unroll
    for (int t = 0; t < Elt<T>::VEC; ++t) w[t] = pw.one(Elt<T>::get(v, t), i0 + t);
  }
};

template <typename T>
struct ResidualWeights {  // functor: max(0, p - q) for vector j (in the p row's vector space)
  Row<T> prow, qrow;
  PWeight<T> pw, qw;
  float inv_zp, inv_zq;
  int kind, draft, V;
  __device__ __forceinline__ void operator()(int j, float *w) const {
    using E = Elt<T>;
    const uint4 v = prow.vec(j);
    const int i0 = j * E::VEC - prow.off;
    uint4 qv = make_uint4(0, 0, 0, 0);
    const bool qvec = (kind == SJD_Q_ROW) && (qrow.off == prow.off);
    if (qvec) qv = qrow.vec(j);
#pragma unroll
    for (int t = 0; t < E::VEC; ++t) {
      const int i = i0 + t;
      const float p = pw.one(E::get(v, t), i) * inv_zp;
      float q;
      if (kind == SJD_Q_ROW) {
        const bool in = (i >= 0 && i < V);
        const uint32_t qb = qvec ? E::get(qv, t) : (in ? qrow.element(i) : E::NEG_INF);
        q = qw.one(qb, i) * inv_zq;
      } else if (kind == SJD_Q_UNIFORM) {
        q = 1.0f / (float)V;
      } else {
        q = (i == draft) ? 1.0f : 0.0f;
      }
      w[t] = (i >= 0 && i < V) ? fmaxf(0.0f, p - q) : 0.0f;
    }
  }
};

// ------------------------------------------------------------------------------------ radix select
// warp 0: locate, from the top, the histogram bin holding the `remaining`-th largest key
__device__ void find_bin(Scratch &sc, uint32_t remaining) {
  const int lane = threadIdx.x & 31;
  uint32_t c[8], tot = 0;
#pragma unroll
  for (int b = 0; b < 8; ++b) {
    c[b] = sc.hist[lane * 8 + b];
    tot += c[b];
  }
  uint32_t incl = tot;  // sum over lanes >= lane
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += y;
  }
  const uint32_t above = incl - tot;
  const bool hit = (above < remaining) && (remaining <= incl);
  const uint32_t ballot = __ballot_sync(0xffffffffu, hit);
  if (ballot == 0) {  // remaining exceeds the population: keep everything
    if (lane == 0) {
      sc.sel_bin = 0;
      sc.count_above = incl - c[0];
    }
    return;
  }
  if (hit) {
    uint32_t acc = above;
#pragma unroll
    for (int b = 7; b >= 0; --b) {
      const uint32_t nxt = acc + c[b];
      if (acc < remaining && remaining <= nxt) {
        sc.sel_bin = lane * 8 + b;
        sc.count_above = acc;
      }
      acc = nxt;
    }
  }
}

// Stage the row (optional), histogram the top digit, find the largest key.  Returns max key.
template <typename T>
__device__ uint32_t stage_first_pass(Row<T> &row, uint4 *stage, Scratch &sc, bool need_hist) {
  using E = Elt<T>;
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int i = tid; i < 256; i += nt) sc.hist[i] = 0;
  if (tid == 0) sc.bad = 0;
  __syncthreads();
  uint32_t kmax = 0, bad = 0;
  for (int j0 = tid; j0 < row.NV; j0 += 4 * nt) {
    uint4 v[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int j = j0 + r * nt;
      if (j < row.NV) v[r] = row.load_global(j, bad);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int j = j0 + r * nt;
      if (j < row.NV) {
        if (stage) stage[j] = v[r];
#pragma unroll
        for (int t = 0; t < E::VEC; ++t) {
          const uint32_t k = E::key(E::get(v[r], t));
          kmax = max(kmax, k);
          if (need_hist) atomicAdd(&sc.hist[k >> (E::KEYBITS - 8)], 1u);
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  if ((tid & 31) == 0) sc.redu[tid >> 5] = kmax;
  if (bad) sc.bad = 1;
  __syncthreads();
  if (stage) row.s = stage;
  kmax = 0;
  for (int w = 0; w < (nt >> 5); ++w) kmax = max(kmax, sc.redu[w]);
  return kmax;
}

// Exact key of the top_k-th largest element (histogram of digit 0 already in sc.hist).
template <typename T>
__device__ uint32_t select_threshold(const Row<T> &row, Scratch &sc, uint32_t top_k) {
  using E = Elt<T>;
  const int tid = threadIdx.x, nt = blockDim.x;
  uint32_t prefix = 0, remaining = top_k;
  constexpr int PASSES = E::KEYBITS / 8;
  for (int pass = 0; pass < PASSES; ++pass) {
    const int shift = E::KEYBITS - 8 * (pass + 1);
    if (pass > 0) {
      for (int i = tid; i < 256; i += nt) sc.hist[i] = 0;
      __syncthreads();
      const uint32_t hi_mask_shift = shift + 8;
      for (int j = tid; j < row.NV; j += nt) {
        const uint4 v = row.vec(j);
#pragma unroll
        for (int t = 0; t < E::VEC; ++t) {
          const uint32_t k = E::key(E::get(v, t));
          if ((k >> hi_mask_shift) == (prefix >> hi_mask_shift)) atomicAdd(&sc.hist[(k >> shift) & 255u], 1u);
        }
      }
      __syncthreads();
    }
    if (tid < 32) find_bin(sc, remaining);
    __syncthreads();
    prefix |= sc.sel_bin << shift;
    remaining -= sc.count_above;
    __syncthreads();
  }
  return prefix;
}

// ------------------------------------------------------------------------------------ sums & sampling
__device__ void chunk_prefix(int NC, Scratch &sc);

// Per-chunk sums of the functor's weights in token order, then their exclusive prefix in fp64.
template <int VEC, typename F>
__device__ void chunk_sums(const F &f, int NV, Scratch &sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  const int NC = (NV + 31) >> 5;
  for (int c = warp; c < NC; c += nw) {
    const int j = c * 32 + lane;
    float s = 0.0f;
    if (j < NV) {
      float w[VEC];
      f(j, w);
#pragma unroll
      for (int t = 0; t < VEC; ++t) s += w[t];
    }
    float incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) sc.chunk_sum[c] = incl;
  }
  __syncthreads();
  chunk_prefix(NC, sc);
}

// Exclusive prefix of sc.chunk_sum[0..NC) in fp64 (warp 0), total in sc.chunk_excl[NC].
__device__ void chunk_prefix(int NC, Scratch &sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (warp == 0) {
    const int per = (NC + 31) >> 5;
    const int lo = min(NC, lane * per), hi = min(NC, lo + per);
    double loc = 0.0;
    for (int c = lo; c < hi; ++c) loc += (double)sc.chunk_sum[c];
    double incl = loc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    double run = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane == 0) run = 0.0;
    for (int c = lo; c < hi; ++c) {
      sc.chunk_excl[c] = run;
      run += (double)sc.chunk_sum[c];
    }
    if (lane == 31) sc.chunk_excl[NC] = incl;
  }
  __syncthreads();
}

// Inverse CDF in token order over the functor's weights (chunk_sums must have run with the same
// functor): smallest index i with w_i > 0 and cumsum_i > u * total.  Result in sc.tok / sc.tok_w.
template <int VEC, typename F>
__device__ void sample_icdf(const F &f, int NV, int off, Scratch &sc, float u) {
  const int tid = threadIdx.x, lane = tid & 31, nt = blockDim.x;
  const int NC = (NV + 31) >> 5;
  const double total = sc.chunk_excl[NC];
  const double target = (double)u * total;
  if (tid == 0) {
    sc.sel_chunk = 0x7fffffff;
    sc.last_chunk = -1;
    sc.tok = 0;
    sc.tok_w = 0.0f;
  }
  __syncthreads();
  for (int c = tid; c < NC; c += nt) {
    if (sc.chunk_sum[c] > 0.0f) {
      atomicMax(&sc.last_chunk, c);
      if (sc.chunk_excl[c] <= target && target < sc.chunk_excl[c + 1]) atomicMin(&sc.sel_chunk, c);
    }
  }
  __syncthreads();
  if (tid < 32) {
    int c = sc.sel_chunk;
    const bool fallback = (c == 0x7fffffff);
    if (fallback) c = sc.last_chunk;
    if (c >= 0) {
      const int j = c * 32 + lane;
      float w[VEC];
      float s = 0.0f;
#pragma unroll
      for (int t = 0; t < VEC; ++t) w[t] = 0.0f;
      if (j < NV) {
        f(j, w);
#pragma unroll
        for (int t = 0; t < VEC; ++t) s += w[t];
      }
      float incl = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      float excl = __shfl_up_sync(0xffffffffu, incl, 1);
      if (lane == 0) excl = 0.0f;
      const double base = sc.chunk_excl[c];
      const bool cond = !fallback && (base + (double)incl > target);
      const uint32_t ballot = __ballot_sync(0xffffffffu, cond);
      const uint32_t pos = __ballot_sync(0xffffffffu, s > 0.0f);
      int sel_lane;
      bool take_last = false;
      if (ballot != 0) {
        sel_lane = __ffs(ballot) - 1;
      } else {
        sel_lane = 31 - __clz(pos);  // pos != 0 because the chunk sum is positive
        take_last = true;
      }
      if (lane == sel_lane) {
        double acc = base + (double)excl;
        int found = -1, last = -1;
#pragma unroll
        for (int t = 0; t < VEC; ++t) {
          if (w[t] > 0.0f) {
            acc += (double)w[t];
            last = t;
            if (found < 0 && !take_last && acc > target) found = t;
          }
        }
        const int t_sel = found >= 0 ? found : last;
        float wsel = 0.0f;
#pragma unroll
        for (int t = 0; t < VEC; ++t)
          if (t == t_sel) wsel = w[t];
        sc.tok = j * VEC + t_sel - off;
        sc.tok_w = wsel;
      }
    }
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------ packed bf16 helpers
__device__ __forceinline__ __nv_bfloat162 as_bf2(uint32_t w) { return *reinterpret_cast<__nv_bfloat162 *>(&w); }
// order-preserving keys of both halves of a packed bf16 pair (same map as Elt<bf16>::key per half)
__device__ __forceinline__ uint32_t key_pair(uint32_t w) {
  const uint32_t neg = ((w >> 15) & 0x00010001u) * 0xFFFFu;   // 0xFFFF in the halves whose sign bit is set
  return w ^ (neg | 0x80008000u);
}
__device__ __forceinline__ uint32_t word_of(const uint4 &v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }

// One 16-byte vector of a row under classifier-free guidance: per entry l_u + w * (l_c - l_u) with one
// subtraction and one fused multiply-add in fp32, rounded to bf16 (the same arithmetic as Row::raw_bits).
__device__ __forceinline__ uint4 mix_vec_bf16(const uint4 &c, const uint4 &u, float w) {
  uint32_t o[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t cx = word_of(c, k), ux = word_of(u, k);
    const float c0 = __uint_as_float(cx << 16), c1 = __uint_as_float(cx & 0xFFFF0000u);
    const float u0 = __uint_as_float(ux << 16), u1 = __uint_as_float(ux & 0xFFFF0000u);
    const __nv_bfloat162 m = __floats2bfloat162_rn(fmaf(w, c0 - u0, u0), fmaf(w, c1 - u1, u1));
    o[k] = *reinterpret_cast<const uint32_t *>(&m);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}
// vector j of a bf16 row (16-byte aligned), mixed with the unconditional stream's row when there is one
__device__ __forceinline__ uint4 rr_load_vec(const uint4 *g, const uint4 *g2, float w, int j) {
  const uint4 c = __ldg(g + j);
  return g2 ? mix_vec_bf16(c, __ldg(g2 + j), w) : c;
}

// ------------------------------------------------------------------------------------ register-resident row, few barriers
// The whole treatment of one window row (Eqs. 1-3) for bf16 rows a block can hold in registers, laid
// out warp by warp: warp w owns chunks 8w .. 8w+7 (32 vectors each, the chunks of chunk_sums), lane l
// holds vector l of each.  Every search over shared tables (histogram bins, chunk prefix) is done
// by each warp for itself instead of by one warp between two barriers, so a row costs about a dozen
// block barriers.  Returns false (block-uniform) when the row needs the general route; nothing it
// has published by then differs from what that route writes.
struct RegRow {
  uint4 v[8];
};

__device__ __forceinline__ uint4 reg_slot(const RegRow &r, int i) {   // i is warp-uniform
  uint4 o = r.v[0];
#pragma unroll
  for (int k = 1; k < 8; ++k)
    if (i == k) o = r.v[k];
  return o;
}

// load + maximum; publishes the entry at index d (if any) in sc.d_bits.  One barrier.  Returns the
// block-wide maximum key; 0xFFFF if the row holds a NaN.
__device__ uint32_t rr_load_max(RegRow &row, const uint4 *g, const uint4 *g2, float gw, int NV, int d, int d_slot,
                                Scratch &sc, bool zero_hist) {
  using E = Elt<__nv_bfloat16>;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nt = blockDim.x, nw = nt >> 5;
  const int j0 = warp * 256 + lane;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int j = j0 + i * 32;
    row.v[i] = j < NV ? rr_load_vec(g, g2, gw, j) : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
  }
  if (zero_hist)
    for (int i = tid; i < 1024; i += nt) reinterpret_cast<uint4 *>(sc.hist12)[i] = make_uint4(0u, 0u, 0u, 0u);
  __nv_bfloat162 m2 = as_bf2(row.v[0].x);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
#pragma unroll
    for (int w = 0; w < 4; ++w) m2 = __hmax2_nan(m2, as_bf2(word_of(row.v[i], w)));
  }
  if (tid == 0 && d >= 0) {   // the entry at the draft token: one more load (a cache hit) instead of a search through the registers
    const unsigned short *e = reinterpret_cast<const unsigned short *>(g);
    uint32_t bits = (uint32_t)__ldg(e + d);
    if (g2) {
      const float c = E::val(bits), u = E::val((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(g2) + d));
      bits = E::bits(fmaf(gw, c - u, u));
    }
    sc.d_bits[d_slot] = bits;
  }
  const __nv_bfloat16 m1 = __hmax_nan(__low2bfloat16(m2), __high2bfloat16(m2));
  const uint32_t mbits = (uint32_t)__bfloat16_as_ushort(m1);
  uint32_t kmax = (mbits & 0x7FFFu) > 0x7F80u ? 0xFFFFu : E::key(mbits);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) sc.redu[warp] = kmax;
  __syncthreads();
  kmax = 0;
  for (int w = 0; w < nw; ++w) kmax = max(kmax, sc.redu[w]);
  return kmax;
}

// Exact key of the K-th largest entry: one histogram pass over the distance (in bf16 codes) of every
// entry below the row's maximum, exact for the 4095 codes next to the maximum (32 binades: for a
// positive maximum, every positive value that matters) and lumped beyond; then every warp walks
// the histogram from the top for itself.  One barrier.  false: the K-th largest lies in the lump
// (or next to +-0), the general route decides.
// `z_hist` (optional): the softmax denominator from the histogram alone -- all entries of a bin share one
// value, so Z = sum over the kept bins of count * 2^((value - max) * scale) -- for rows whose chunk
// sums nobody needs (the previous-iteration row when its statistics are not cached).
// histogram pass of rr_select over the vectors held in `row` (those with local index below NV)
__device__ __forceinline__ void rr_hist_add(const RegRow &row, int NV, uint32_t kmax, Scratch &sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int j0 = warp * 256 + lane;
  const uint32_t kmax2 = kmax | (kmax << 16);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (j0 + i * 32 < NV) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint32_t dist = kmax2 - key_pair(word_of(row.v[i], w));   // per half, no borrow: keys <= kmax
        // every entry is counted, the far ones in the last bin (skipping them under a predicate was measured
        // slower: the predicate becomes a branch, and the cost of a shared-memory reduction does not depend
        // on how many lanes take part or on how many of them hit the same counter)
        atomicAdd(&sc.hist12[min(dist & 0xFFFFu, 4095u)], 1u);
        atomicAdd(&sc.hist12[min(dist >> 16, 4095u)], 1u);
      }
    }
  }
}

// walk of rr_select over the finished histogram (every warp for itself)
__device__ __forceinline__ bool rr_walk(uint32_t kmax, uint32_t K, Scratch &sc, uint32_t &tau_key, float scale,
                                        double *z_hist) {
  using E = Elt<__nv_bfloat16>;
  const int lane = threadIdx.x & 31;
  // The walk: 32 adjacent bins per step (conflict-free).  A step that does not reach the K-th entry costs one
  // load and one warp-wide integer sum; only the step that does is scanned.  For z_hist every lane
  // accumulates the mass of its own bins and the warp adds the lanes up once, at the end.
  uint32_t acc = 0;
  float zl = 0.0f;
  const float xmax = E::val(E::unkey(kmax));
  for (int base = 0; base < 4096; base += 32) {
    const uint32_t c = sc.hist12[base + lane];
    const uint32_t bin = (uint32_t)(base + lane);
    const uint32_t tot = __reduce_add_sync(0xffffffffu, c);
    if (acc + tot < K) {
      if (z_hist && c != 0 && bin <= kmax) zl += (float)c * exp2_neg((E::val(E::unkey(kmax - bin)) - xmax) * scale);
      acc += tot;
      continue;
    }
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    const uint32_t ballot = __ballot_sync(0xffffffffu, acc + incl >= K);   // non-zero: this step reaches K
    const int last = __ffs(ballot) - 1;
    if (z_hist) {   // mass of this step's bins down to (and including) the threshold bin
      if (lane <= last && c != 0 && bin <= kmax) zl += (float)c * exp2_neg((E::val(E::unkey(kmax - bin)) - xmax) * scale);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) zl += __shfl_xor_sync(0xffffffffu, zl, o);
      *z_hist = (double)zl;
    }
    const uint32_t tbin = (uint32_t)(base + last);
    if (tbin >= 4095u) return false;
    tau_key = kmax - tbin;
    return !(tau_key == 0x7FFFu || tau_key == 0x8000u);
  }
  return false;
}

__device__ __forceinline__ bool rr_select(const RegRow &row, int NV, uint32_t kmax, uint32_t K, Scratch &sc,
                                          uint32_t &tau_key, float scale, double *z_hist) {
  rr_hist_add(row, NV, kmax, sc);
  __syncthreads();
  return rr_walk(kmax, K, sc, tau_key, scale, z_hist);
}

// chunk sums of a weight functor evaluated on registers -> sc.chunk_sum.  One barrier.
// Every lane holds eight slot sums; the warp adds them up transposed (each exchange halves the number of
// slots a lane still carries: 4 + 2 + 1 + 1 + 1 shuffles instead of 8 x 5), in a fixed order.
// `chunk0`: chunk index of this block's first vector (rows streamed in segments), NC then counts the whole row's chunks.
template <typename F>
__device__ __forceinline__ void rr_chunk_sums(const F &wf, int NV, Scratch &sc, int chunk0 = 0, int n_chunks = -1) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NC = n_chunks >= 0 ? n_chunks : (NV + 31) >> 5;
  float s[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float w[8];
    wf(i, w);
    s[i] = ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
  }
  const bool b4 = (lane & 16) != 0, b3 = (lane & 8) != 0, b2 = (lane & 4) != 0;
  float a[4], c[2];
#pragma unroll
  for (int k = 0; k < 4; ++k) {   // lanes 16..31 keep slots 4..7, lanes 0..15 slots 0..3
    const float send = b4 ? s[k] : s[k + 4], keep = b4 ? s[k + 4] : s[k];
    a[k] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
  }
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const float send = b3 ? a[k] : a[k + 2], keep = b3 ? a[k + 2] : a[k];
    c[k] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
  }
  float e;
  {
    const float send = b2 ? c[0] : c[1], keep = b2 ? c[1] : c[0];
    e = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  }
  e += __shfl_xor_sync(0xffffffffu, e, 2);
  e += __shfl_xor_sync(0xffffffffu, e, 1);
  const int slot = (lane >> 2) & 7;   // bit 4 -> slot bit 2, bit 3 -> bit 1, bit 2 -> bit 0
  if ((lane & 3) == 0 && chunk0 + warp * 8 + slot < NC) sc.chunk_sum[chunk0 + warp * 8 + slot] = e;
  __syncthreads();
}

// Per-warp view of the fp64 prefix over sc.chunk_sum: lane L owns chunks [L*per, (L+1)*per).
struct WarpPrefix {
  double excl, incl, total;
  int per;
};
__device__ __forceinline__ WarpPrefix rr_prefix(int NC, const Scratch &sc) {
  const int lane = threadIdx.x & 31;
  WarpPrefix wp;
  wp.per = (NC + 31) >> 5;
  const int lo = min(NC, lane * wp.per), hi = min(NC, lo + wp.per);
  double loc = 0.0;
  for (int c = lo; c < hi; ++c) loc += (double)sc.chunk_sum[c];
  double incl = loc;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  wp.incl = incl;
  wp.excl = incl - loc;
  wp.total = __shfl_sync(0xffffffffu, incl, 31);
  return wp;
}

// Inverse CDF (token order) over weights held in registers: every warp finds the chunk, the warp that
// owns it finds the entry (same rules as sample_icdf) and publishes it.  One barrier.
// wf(c, w): this lane's eight weights of chunk c, asked of the warp that owns the chunk (chunk c of a row
// streamed in segments of 8 * blockDim vectors belongs to warp (c mod 8 * warps) / 8).
template <typename F>
__device__ void rr_icdf(const F &wf, int NV, const WarpPrefix &wp, float u, Scratch &sc, int &tok, float &tok_w) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NC = (NV + 31) >> 5;
  const int seg_chunks = (int)(blockDim.x >> 5) * 8;
  const double target = (double)u * wp.total;
  const int lo = min(NC, lane * wp.per), hi = min(NC, lo + wp.per);
  // inside this lane's group: first chunk with positive mass whose interval holds the target; last positive chunk
  int c_hit = -1, c_last = -1;
  double base_hit = 0.0, base_last = 0.0, run = wp.excl;
  for (int c = lo; c < hi; ++c) {
    const float cs = sc.chunk_sum[c];
    const double nxt = run + (double)cs;
    if (cs > 0.0f) {
      if (c_hit < 0 && run <= target && target < nxt) {
        c_hit = c;
        base_hit = run;
      }
      c_last = c;
      base_last = run;
    }
    run = nxt;
  }
  const uint32_t hit = __ballot_sync(0xffffffffu, c_hit >= 0);
  const uint32_t pos = __ballot_sync(0xffffffffu, c_last >= 0);
  bool fallback = false;
  int c;
  double base;
  if (hit) {
    const int src = __ffs(hit) - 1;
    c = __shfl_sync(0xffffffffu, c_hit, src);
    base = __shfl_sync(0xffffffffu, base_hit, src);
  } else if (pos) {
    const int src = 31 - __clz(pos);
    c = __shfl_sync(0xffffffffu, c_last, src);
    base = __shfl_sync(0xffffffffu, base_last, src);
    fallback = true;
  } else {
    c = -1;
    base = 0.0;
  }
  if (c < 0) {
    if (tid == 0) {
      sc.tok = 0;
      sc.tok_w = 0.0f;
    }
  } else if (warp == ((c % seg_chunks) >> 3)) {
    float w[8];
    wf(c, w);
    float sum = 0.0f;
#pragma unroll
    for (int t = 0; t < 8; ++t) sum += w[t];
    float incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    float excl = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane == 0) excl = 0.0f;
    const bool cond = !fallback && (base + (double)incl > target);
    const uint32_t ballot = __ballot_sync(0xffffffffu, cond);
    const uint32_t posl = __ballot_sync(0xffffffffu, sum > 0.0f);
    int sel_lane;
    bool take_last = false;
    if (ballot != 0) {
      sel_lane = __ffs(ballot) - 1;
    } else {
      sel_lane = posl ? 31 - __clz(posl) : 0;
      take_last = true;
    }
    if (lane == sel_lane) {
      double acc = base + (double)excl;
      int found = -1, last = -1;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        if (w[t] > 0.0f) {
          acc += (double)w[t];
          last = t;
          if (found < 0 && !take_last && acc > target) found = t;
        }
      }
      const int t_sel = found >= 0 ? found : (last >= 0 ? last : 0);
      float wsel = 0.0f;
#pragma unroll
      for (int t = 0; t < 8; ++t)
        if (t == t_sel) wsel = w[t];
      sc.tok = (c * 32 + lane) * 8 + t_sel;
      sc.tok_w = wsel;
    }
  }
  __syncthreads();
  tok = sc.tok;
  tok_w = sc.tok_w;
}

// weights of the eight entries of one vector whose entries below the threshold have been replaced by
// -inf (rr_mask_below): 2^((x - max) * scale) as one fused multiply-add and one exp2 per entry
__device__ __forceinline__ void rr_p_weights(const uint4 &v, float xmax, float scale, float *w) {
  const float c0 = -xmax * scale;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t x = word_of(v, k);
    w[2 * k] = exp2_neg(fmaf(__uint_as_float(x << 16), scale, c0));
    w[2 * k + 1] = exp2_neg(fmaf(__uint_as_float(x & 0xFFFF0000u), scale, c0));
  }
}

// entries below the threshold (a value other than +-0) become -inf, two per instruction pair
__device__ __forceinline__ void rr_mask_below(RegRow &row, float tau_f) {
  const __nv_bfloat16 t1 = __float2bfloat16_rn(tau_f);   // exact: the threshold is an entry of the row
  const __nv_bfloat162 t2 = __halves2bfloat162(t1, t1);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t *w = reinterpret_cast<uint32_t *>(&row.v[i]);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t m = __hge2_mask(as_bf2(w[k]), t2);
      w[k] = (w[k] & m) | (0xFF80FF80u & ~m);
    }
  }
}

struct RowFast {   // statistics of a row on this route
  RowStats st;
  float tau_f;
  float d_weight;   // unnormalised weight of the entry at the draft token
  double z_hist;    // denominator from the histogram (rows processed without chunk sums), else < 0
};

// statistics of one row: 4 barriers.  false: general route.
// `want_chunks`: mask the entries below the threshold in `row` and leave the chunk sums of the row's
// weights in sc.chunk_sum (needed to sample from the row).
__device__ bool rr_statistics(RegRow &row, const __nv_bfloat16 *g, const __nv_bfloat16 *g2, float gw, int V, int d,
                              int d_slot, int top_k, float inv_t, Scratch &sc, RowFast &out, bool want_chunks) {
  using E = Elt<__nv_bfloat16>;
  const int NV = V >> 3;
  const bool need_select = top_k < V;
  const uint32_t kmax = rr_load_max(row, reinterpret_cast<const uint4 *>(g), reinterpret_cast<const uint4 *>(g2), gw, NV, d,
                                    d_slot, sc, need_select);
  if (kmax >= 0xFF80u || kmax <= 0x007Fu) return false;
  SJD_TL(TL_VERIFY, 20, threadIdx.x == 0);   // row loaded, maximum known
  uint32_t tau_key = 0;
  const float scale = inv_t * 1.4426950408889634f;
  const bool from_hist = need_select && !want_chunks;
  out.z_hist = -1.0;
  if (need_select && !rr_select(row, NV, kmax, (uint32_t)top_k, sc, tau_key, scale, from_hist ? &out.z_hist : nullptr))
    return false;
  SJD_TL(TL_VERIFY, 23, threadIdx.x == 0);   // threshold known
  out.st.tau_key = tau_key;
  out.st.xmax = E::val(E::unkey(kmax));
  out.st.flags = 0;
  out.tau_f = need_select ? E::val(E::unkey(tau_key)) : -INFINITY;
  const float xmax = out.st.xmax, tau_f = out.tau_f;
  if (from_hist) {
    __syncthreads();   // sc.d_bits is read below; the walk above read the histogram the next row clears
  } else {
    if (need_select) rr_mask_below(row, tau_f);
    rr_chunk_sums([&](int i, float *w) { rr_p_weights(row.v[i], xmax, scale, w); }, NV, sc);
  }
  SJD_TL(TL_VERIFY, 24, threadIdx.x == 0);   // chunk sums written
  const float dv = E::val(sc.d_bits[d_slot]);
  out.d_weight = (d >= 0 && dv >= tau_f) ? exp2_neg((dv - xmax) * scale) : 0.0f;
  return true;
}

// ------------------------------------------------------------------------------------ rows longer than the registers
// bf16 rows of more than 8 * blockDim vectors (V = 184320: 23040 vectors against 8192) take the same phases with
// the row streamed through the registers one segment of 8 * blockDim vectors at a time; every phase reads the
// row again (it was written by the preceding kernel and sits in L2): maximum, histogram, masked weights and
// chunk sums.  The chunk numbering is the one of a row held at once (chunk = 32 consecutive vectors), so the
// prefix and the search over sc.chunk_sum are shared; the search re-reads the one chunk it ends in.
__device__ __forceinline__ void seg_load(RegRow &row, const uint4 *g, const uint4 *g2, float gw, int NV, int seg) {
  const int j0 = seg * 8 * (int)blockDim.x + (int)(threadIdx.x >> 5) * 256 + (int)(threadIdx.x & 31);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int j = j0 + i * 32;
    row.v[i] = j < NV ? rr_load_vec(g, g2, gw, j) : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
  }
}
// vector j of the row with the entries below the threshold replaced by -inf (what rr_mask_below leaves in a RegRow)
__device__ __forceinline__ uint4 load_masked_vec(const uint4 *g, const uint4 *g2, float gw, int NV, int j, float tau_f) {
  if (j >= NV) return make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
  const uint4 v = rr_load_vec(g, g2, gw, j);
  const __nv_bfloat16 t1 = __float2bfloat16_rn(tau_f);
  const __nv_bfloat162 t2 = __halves2bfloat162(t1, t1);
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t m = __hge2_mask(as_bf2(w[k]), t2);
    w[k] = (w[k] & m) | (0xFF80FF80u & ~m);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// rr_statistics for a streamed row.  Barriers: 1 (maximum) + 1 (histogram) + one per segment (chunk sums).
__device__ bool long_statistics(const __nv_bfloat16 *g, const __nv_bfloat16 *g2, float gw, int V, int d, int d_slot, int top_k,
                                float inv_t, Scratch &sc, RowFast &out, bool want_chunks) {
  using E = Elt<__nv_bfloat16>;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nt = blockDim.x, nw = nt >> 5;
  const int NV = V >> 3, NC = (NV + 31) >> 5;
  const int seg_v = 8 * nt, n_seg = (NV + seg_v - 1) / seg_v;
  const uint4 *gv = reinterpret_cast<const uint4 *>(g), *gv2 = reinterpret_cast<const uint4 *>(g2);
  const bool need_select = top_k < V;
  RegRow row;
  // ---- maximum (and the entry at the draft token)
  if (need_select)
    for (int i = tid; i < 1024; i += nt) reinterpret_cast<uint4 *>(sc.hist12)[i] = make_uint4(0u, 0u, 0u, 0u);
  __nv_bfloat162 m2 = as_bf2(0xFF80FF80u);
  for (int seg = 0; seg < n_seg; ++seg) {
    seg_load(row, gv, gv2, gw, NV, seg);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int w = 0; w < 4; ++w) m2 = __hmax2_nan(m2, as_bf2(word_of(row.v[i], w)));
    }
  }
  if (tid == 0 && d >= 0) {
    uint32_t bits = (uint32_t)__ldg(reinterpret_cast<const unsigned short *>(g) + d);
    if (g2) {
      const float c = E::val(bits), u = E::val((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(g2) + d));
      bits = E::bits(fmaf(gw, c - u, u));
    }
    sc.d_bits[d_slot] = bits;
  }
  const __nv_bfloat16 m1 = __hmax_nan(__low2bfloat16(m2), __high2bfloat16(m2));
  const uint32_t mbits = (uint32_t)__bfloat16_as_ushort(m1);
  uint32_t kmax = (mbits & 0x7FFFu) > 0x7F80u ? 0xFFFFu : E::key(mbits);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) sc.redu[warp] = kmax;
  __syncthreads();
  kmax = 0;
  for (int w = 0; w < nw; ++w) kmax = max(kmax, sc.redu[w]);
  if (kmax >= 0xFF80u || kmax <= 0x007Fu) return false;
  // ---- threshold
  uint32_t tau_key = 0;
  const float scale = inv_t * 1.4426950408889634f;
  const bool from_hist = need_select && !want_chunks;
  out.z_hist = -1.0;
  if (need_select) {
    for (int seg = 0; seg < n_seg; ++seg) {
      seg_load(row, gv, gv2, gw, NV, seg);
      rr_hist_add(row, NV - seg * seg_v, kmax, sc);
    }
    __syncthreads();
    if (!rr_walk(kmax, (uint32_t)top_k, sc, tau_key, scale, from_hist ? &out.z_hist : nullptr)) return false;
  }
  out.st.tau_key = tau_key;
  out.st.xmax = E::val(E::unkey(kmax));
  out.st.flags = 0;
  out.tau_f = need_select ? E::val(E::unkey(tau_key)) : -INFINITY;
  const float xmax = out.st.xmax, tau_f = out.tau_f;
  if (from_hist) {
    __syncthreads();   // sc.d_bits is read below; the walk above read the histogram the next row clears
  } else {
    for (int seg = 0; seg < n_seg; ++seg) {
      seg_load(row, gv, gv2, gw, NV, seg);
      if (need_select) rr_mask_below(row, tau_f);
      rr_chunk_sums([&](int i, float *w) { rr_p_weights(row.v[i], xmax, scale, w); }, NV, sc, seg * nw * 8, NC);
    }
  }
  const float dv = E::val(sc.d_bits[d_slot]);
  out.d_weight = (d >= 0 && dv >= tau_f) ? exp2_neg((dv - xmax) * scale) : 0.0f;
  return true;
}

// The logits rows of window slot k of image b: this iteration's (p) and the one the draft was drawn from
// (q, row qr of the other buffer); under guidance the unconditional stream's rows beside them (else null).
template <typename T>
struct RowRefs {
  const T *p, *p2, *q, *q2;
  const RowStats *qstats;   // statistics of the q row (valid when the launch has them cached)
};
// q_ring: the draft's law is a retained row (Sec. 4.2 (d)): qr is then a slot of the ring, whose rows are
// stored as the verification saw them (already mixed under guidance)
template <typename T>
__device__ __forceinline__ RowRefs<T> row_refs(const VerifyParams &p, int b, int k, int qr, int cur, bool q_ring = false) {
  const int sb = p.paired ? 2 * b : b;
  RowRefs<T> rr;
  rr.p = reinterpret_cast<const T *>(p.logits[cur]) + ((size_t)sb * p.W + k) * p.V;
  rr.p2 = p.paired ? rr.p + (size_t)p.W * p.V : nullptr;
  if (q_ring) {
    rr.q = reinterpret_cast<const T *>(p.ring) + ((size_t)b * p.ring_len + qr) * p.V;
    rr.q2 = nullptr;
    rr.qstats = p.ring_stats + (size_t)b * p.ring_len + qr;
  } else {
    rr.q = reinterpret_cast<const T *>(p.logits[cur ^ 1]) + ((size_t)sb * p.W + qr) * p.V;
    rr.q2 = p.paired ? rr.q + (size_t)p.W * p.V : nullptr;
    rr.qstats = p.stats[cur ^ 1] + (size_t)b * p.W + qr;
  }
  return rr;
}

template <bool STREAM_OK>
__device__ void rr_residual(const VerifyParams &p, const RegRow *row_in, const RowRefs<__nv_bfloat16> &rows, int kind, int d,
                            const RowStats &ps, const RowStats &qs, float u_res, Scratch &sc, int &tok, uint32_t &flags);


constexpr int kResampleDeferred = -2;   // RowOut.resample_tok of a rejected row whose Eq. 2 draw is still to be made

// STREAM_OK: the instantiation for full blocks, which also takes rows too long for the registers
template <bool STREAM_OK>
__device__ bool fast_row_bf16(const VerifyParams &p, Scratch &sc, int r, int b, int kind, int d, int qr, int cur,
                              const RowRefs<__nv_bfloat16> &rows, float inv_t, float u_acc, float u_res,
                              float u_draft, RowOut &ro) {
  using E = Elt<__nv_bfloat16>;
  const int tid = threadIdx.x;
  const int V = p.V, NV = V >> 3, NC = (NV + 31) >> 5;
  const bool streamed = STREAM_OK && NV > 8 * (int)blockDim.x;   // too long for the registers: see long_statistics
  if (NV > 8 * (int)blockDim.x && (!STREAM_OK || NC > kMaxChunks)) return false;
  const bool d_ok = d >= 0 && d < V;
  const int dd = d_ok ? d : -1;
  const float scale = inv_t * 1.4426950408889634f;
  RegRow row;

  // ---- the law of the draft
  RowStats qs;
  qs.tau_key = 0; qs.xmax = 0.0f; qs.z = 1.0f; qs.flags = 0;
  float q_d;
  if (kind == SJD_Q_ROW) {
    if (p.prev_stats_valid) {
      qs = *rows.qstats;
      if (qs.flags != 0 || !(qs.xmax > -FLT_MAX) || qs.tau_key == 0x7FFFu || qs.tau_key == 0x8000u) return false;
      uint32_t bits = E::NEG_INF;
      if (d_ok) {
        bits = E::load_bits(rows.q + d);
        if (rows.q2) {
          const float cq = E::val(bits), uq = E::val(E::load_bits(rows.q2 + d));
          bits = E::bits(fmaf(p.guidance, cq - uq, uq));
        }
      }
      if (E::bad(bits)) return false;
      q_d = d_ok ? (E::key(bits) >= qs.tau_key ? exp2_neg((E::val(bits) - qs.xmax) * scale) : 0.0f) / qs.z : 1.0f;
    } else {
      RowFast qfast;
      if (!(streamed ? long_statistics(rows.q, rows.q2, p.guidance, V, dd, 0, p.top_k, inv_t, sc, qfast, false)
                     : rr_statistics(row, rows.q, rows.q2, p.guidance, V, dd, 0, p.top_k, inv_t, sc, qfast, false)))
        return false;
      qs = qfast.st;
      qs.z = (float)(qfast.z_hist >= 0.0 ? qfast.z_hist : rr_prefix(NC, sc).total);
      if (tid == 0) p.stats[cur ^ 1][r] = qs;
      q_d = d_ok ? qfast.d_weight / qs.z : 1.0f;
    }
  } else if (kind == SJD_Q_UNIFORM) {
    q_d = 1.0f / (float)V;
  } else {
    q_d = 1.0f;
  }

  SJD_TL(TL_VERIFY, 10, tid == 0);
  // ---- this iteration's distribution (entries below the threshold are -inf in `row` from here on)
  RowFast pfast;
  if (!(streamed ? long_statistics(rows.p, rows.p2, p.guidance, V, dd, 1, p.top_k, inv_t, sc, pfast, true)
                 : rr_statistics(row, rows.p, rows.p2, p.guidance, V, dd, 1, p.top_k, inv_t, sc, pfast, true)))
    return false;
  const WarpPrefix wpp = rr_prefix(NC, sc);
  RowStats ps = pfast.st;
  ps.z = (float)wpp.total;
  if (tid == 0) p.stats[cur][r] = ps;
  const float p_d = d_ok ? pfast.d_weight / ps.z : 0.0f;
  const float xmax_p = ps.xmax;
  SJD_TL(TL_VERIFY, 11, tid == 0);

  // ---- Eq. 1
  float ratio;
  if (q_d > 0.0f) ratio = p_d / q_d;
  else ratio = p_d > 0.0f ? INFINITY : 0.0f;
  const float thr = fminf(1.0f, ratio);
  const bool accept = u_acc < thr;
  uint32_t flags = 0;
  if (thr < 1.0f && fabsf(u_acc - thr) < 1e-4f) flags |= SJD_FLAG_NEAR_TIE_ACCEPT;

  // ---- Eq. 3: re-draft from p
  auto p_w = [&](int i, float *w) { rr_p_weights(reg_slot(row, i), xmax_p, scale, w); };
  int redraft_tok;
  float redraft_w;
  if (streamed) {
    const uint4 *pg = reinterpret_cast<const uint4 *>(rows.p), *pg2 = reinterpret_cast<const uint4 *>(rows.p2);
    const float tau_f = pfast.tau_f;
    rr_icdf([&](int c, float *w) {
      rr_p_weights(load_masked_vec(pg, pg2, p.guidance, NV, c * 32 + (tid & 31), tau_f), xmax_p, scale, w);
    }, NV, wpp, u_draft, sc, redraft_tok, redraft_w);
  } else {
    rr_icdf([&](int c, float *w) { p_w(c & 7, w); }, NV, wpp, u_draft, sc, redraft_tok, redraft_w);
  }
  const float redraft_p = redraft_w / ps.z;
  SJD_TL(TL_VERIFY, 12, tid == 0);

  // ---- Eq. 2.  Only the first rejected row of a sequence needs it.  In a grid of several waves a rejected row
  // leaves it to the block that scans the sequence (32 draws per launch instead of up to B * W); in a grid
  // that is resident at once (one sequence: latency matters, throughput does not) every rejected row draws
  // its token now, in parallel with the others.
  int resample_tok = accept ? -1 : kResampleDeferred;
  if (!accept && !p.defer_residual && p.schedule != SJD_SCHEDULE_JACOBI) {
    __syncthreads();
    rr_residual<STREAM_OK>(p, streamed ? nullptr : &row, rows, kind, d, ps, qs, u_res, sc, resample_tok, flags);
  }
  ro.p_draft = p_d; ro.q_draft = q_d; ro.thr = thr; ro.accept = accept ? 1 : 0;
  ro.redraft_tok = redraft_tok; ro.redraft_p = redraft_p; ro.resample_tok = resample_tok;
  ro.flags = flags;
  if (p.schedule == SJD_SCHEDULE_JACOBI) {   // deterministic criterion: the slot is fixed if its token did not change
    const bool same = d_ok && redraft_tok == d;
    ro.thr = same ? 1.0f : 0.0f;
    ro.accept = same ? 1 : 0;
    ro.resample_tok = same ? -1 : redraft_tok;   // the first changed slot is fixed to its new token
    ro.flags = 0;
  }
  return true;
}

template <typename T, bool STREAM_OK>
__device__ __forceinline__ bool fast_row(const VerifyParams &p, Scratch &sc, int r, int b, int kind, int d, int qr, int cur,
                                         const RowRefs<T> &rows, float inv_t, float u_acc, float u_res, float u_draft,
                                         RowOut &ro) {
  if constexpr (std::is_same<T, __nv_bfloat16>::value)
    return fast_row_bf16<STREAM_OK>(p, sc, r, b, kind, d, qr, cur, rows, inv_t, u_acc, u_res, u_draft, ro);
  else
    return false;
}

// Eq. 2 on a p row held in registers (entries below its threshold may already have been replaced by
// -inf): residual weights max(0, p - q), their chunk sums and the inverse-CDF draw; the q row is read
// from global memory (L2) vector by vector as it is needed.  Block-wide; returns the token and flags.
// row_in == null: the p row is too long for the registers and is streamed from global memory as well (only in
// the instantiation for full blocks, STREAM_OK: smaller blocks never meet such a row).
template <bool STREAM_OK>
__device__ void rr_residual(const VerifyParams &p, const RegRow *row_in, const RowRefs<__nv_bfloat16> &rows, int kind, int d,
                            const RowStats &ps, const RowStats &qs, float u_res, Scratch &sc, int &tok, uint32_t &flags) {
  using E = Elt<__nv_bfloat16>;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = p.V, NV = V >> 3, NC = (NV + 31) >> 5;
  const float scale = (1.0f / p.temperature) * 1.4426950408889634f;
  const uint4 *qg = reinterpret_cast<const uint4 *>(rows.q), *qg2 = reinterpret_cast<const uint4 *>(rows.q2);
  const float tau_p = ps.tau_key ? E::val(E::unkey(ps.tau_key)) : -INFINITY;
  const float tau_q = qs.tau_key ? E::val(E::unkey(qs.tau_key)) : -INFINITY;
  const int j0 = warp * 256 + lane;
  // probabilities straight from one fused multiply-add per entry: p_i = 2^(x_i * scale + c) with
  // c = -max * scale - log2(Z); entries below the threshold contribute nothing
  const float cp = -ps.xmax * scale - log2f(ps.z), cq = -qs.xmax * scale - log2f(qs.z);
  const float q_uniform = 1.0f / (float)V;
  auto r_vec = [&](const uint4 &pv, int j, float *w) {   // max(0, p - q) of the eight entries of vector j
    uint4 qv = make_uint4(0, 0, 0, 0);
    if (kind == SJD_Q_ROW && j < NV) qv = rr_load_vec(qg, qg2, p.guidance, j);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t px = word_of(pv, k), qx = word_of(qv, k);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float pval = __uint_as_float(h ? px & 0xFFFF0000u : px << 16);
        const float pp = pval >= tau_p ? exp2_neg(fmaf(pval, scale, cp)) : 0.0f;   // fillers (-inf) give 0
        float qq;
        if (kind == SJD_Q_ROW) {
          const float qval = __uint_as_float(h ? qx & 0xFFFF0000u : qx << 16);
          qq = qval >= tau_q ? exp2_neg(fmaf(qval, scale, cq)) : 0.0f;
        } else if (kind == SJD_Q_UNIFORM) {
          qq = q_uniform;
        } else {
          qq = (j * 8 + k * 2 + h == d) ? 1.0f : 0.0f;
        }
        w[2 * k + h] = fmaxf(0.0f, pp - qq);
      }
    }
  };
  auto p_vec = [&](const uint4 &pv, float *w) {   // the p row's own weights (empty residual: sample from p)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t px = word_of(pv, k);
      const float lo = __uint_as_float(px << 16), hi = __uint_as_float(px & 0xFFFF0000u);
      w[2 * k] = lo >= tau_p ? exp2_neg((lo - ps.xmax) * scale) : 0.0f;
      w[2 * k + 1] = hi >= tau_p ? exp2_neg((hi - ps.xmax) * scale) : 0.0f;
    }
  };
  float wsel;
  if (STREAM_OK && row_in == nullptr) {
    // ---- a row streamed in segments (see long_statistics): chunk sums segment by segment, the search re-reads
    // the vectors of the chunk it ends in
    const uint4 *pg = reinterpret_cast<const uint4 *>(rows.p), *pg2 = reinterpret_cast<const uint4 *>(rows.p2);
    const int nw = blockDim.x >> 5, seg_v = 8 * (int)blockDim.x, n_seg = (NV + seg_v - 1) / seg_v;
    const uint4 filler = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
    RegRow seg_row;
    for (int seg = 0; seg < n_seg; ++seg) {
      seg_load(seg_row, pg, pg2, p.guidance, NV, seg);
      rr_chunk_sums([&](int i, float *w) { r_vec(seg_row.v[i], seg * seg_v + j0 + i * 32, w); }, NV, sc, seg * nw * 8, NC);
    }
    WarpPrefix wr = rr_prefix(NC, sc);
    if (wr.total > 0.0) {
      rr_icdf([&](int c, float *w) {
        const int j = c * 32 + lane;
        r_vec(j < NV ? rr_load_vec(pg, pg2, p.guidance, j) : filler, j, w);
      }, NV, wr, u_res, sc, tok, wsel);
    } else {
      flags |= SJD_FLAG_RESIDUAL_EMPTY;
      __syncthreads();
      for (int seg = 0; seg < n_seg; ++seg) {
        seg_load(seg_row, pg, pg2, p.guidance, NV, seg);
        rr_chunk_sums([&](int i, float *w) { p_vec(seg_row.v[i], w); }, NV, sc, seg * nw * 8, NC);
      }
      wr = rr_prefix(NC, sc);
      rr_icdf([&](int c, float *w) {
        const int j = c * 32 + lane;
        p_vec(j < NV ? rr_load_vec(pg, pg2, p.guidance, j) : filler, w);
      }, NV, wr, u_res, sc, tok, wsel);
    }
    return;
  }
  const RegRow &row = *row_in;
  auto r_w = [&](int i, float *w) { r_vec(reg_slot(row, i), j0 + i * 32, w); };
  rr_chunk_sums(r_w, NV, sc);
  WarpPrefix wr = rr_prefix(NC, sc);
  if (wr.total > 0.0) {
    rr_icdf([&](int c, float *w) { r_w(c & 7, w); }, NV, wr, u_res, sc, tok, wsel);
  } else {
    flags |= SJD_FLAG_RESIDUAL_EMPTY;
    auto p_w = [&](int i, float *w) { p_vec(reg_slot(row, i), w); };
    __syncthreads();
    rr_chunk_sums(p_w, NV, sc);
    wr = rr_prefix(NC, sc);
    rr_icdf([&](int c, float *w) { p_w(c & 7, w); }, NV, wr, u_res, sc, tok, wsel);
  }
}

// Eq. 2 for the first rejected row of sequence b, when that row left it open (register-resident route,
// grids of more than one wave): run by every thread of the sequence's last block before the window slide.
// The row's statistics and those of its draft's law were published by the block that verified it; the p
// row is read again into registers (it is still in L2).
template <bool STREAM_OK>
__device__ void deferred_residual_bf16(const VerifyParams &p, int b, uint32_t step, int cur, Scratch &sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int W = p.W, NV = p.V >> 3;
  const int w_eff = p.w_eff ? p.w_eff[p.paired ? 2 * b : b] : W;
  RowOut *ro = p.row_out + (size_t)b * W;
  if (tid < 32) {
    int first = w_eff;
    for (int k = lane; k < w_eff; k += 32)
      if (!__ldcg(&ro[k].accept)) first = min(first, k);
    first = __reduce_min_sync(0xffffffffu, first);
    if (lane == 0) sc.sel_chunk = (first < w_eff && __ldcg(&ro[first].resample_tok) == kResampleDeferred) ? first : -1;
  }
  __syncthreads();
  const int a = sc.sel_chunk;
  __syncthreads();
  if (a < 0) return;
  const int r = b * W + a;
  const int sb = p.paired ? 2 * b : b;   // the sequence whose state holds the window (both streams hold the same)
  const int kind_raw = p.q_kind ? p.q_kind[sb * W + a] : SJD_Q_ROW;
  const int kind = kind_raw == SJD_Q_RING ? SJD_Q_ROW : kind_raw;
  const int d = p.draft[sb * W + a];
  const int qr = p.q_row ? p.q_row[sb * W + a] : a;
  const int base = p.e2e ? p.st.n[sb] : (p.base_pos ? p.base_pos[b] : 0);
  const Philox4 rnd = philox4x32_10((uint32_t)(base + a), step, p.seq_base + (uint32_t)b, kStreamVerify, p.seed_lo,
                                    p.seed_hi);
  const float u_res = u24(rnd.w[1]);
  const RowRefs<__nv_bfloat16> rows = row_refs<__nv_bfloat16>(p, b, a, qr, cur, kind_raw == SJD_Q_RING);
  const uint4 *pg = reinterpret_cast<const uint4 *>(rows.p), *pg2 = reinterpret_cast<const uint4 *>(rows.p2);
  auto load_stats = [](const RowStats *g) {
    const uint4 u = __ldcg(reinterpret_cast<const uint4 *>(g));
    RowStats st;
    st.tau_key = u.x; st.xmax = __uint_as_float(u.y); st.z = __uint_as_float(u.z); st.flags = u.w;
    return st;
  };
  const RowStats ps = load_stats(&p.stats[cur][r]);
  RowStats qs;
  qs.tau_key = 0; qs.xmax = 0.0f; qs.z = 1.0f; qs.flags = 0;
  if (kind == SJD_Q_ROW) qs = load_stats(rows.qstats);
  uint32_t flags = 0;
  int tok;
  if (STREAM_OK && NV > 8 * (int)blockDim.x) {   // a row streamed in segments
    rr_residual<STREAM_OK>(p, nullptr, rows, kind, d, ps, qs, u_res, sc, tok, flags);
  } else {
    RegRow row;
    const int j0 = warp * 256 + lane;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int j = j0 + i * 32;
      row.v[i] = j < NV ? rr_load_vec(pg, pg2, p.guidance, j) : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
    }
    rr_residual<STREAM_OK>(p, &row, rows, kind, d, ps, qs, u_res, sc, tok, flags);
  }
  if (tid == 0) {
    ro[a].resample_tok = tok;
    ro[a].flags = __ldcg(&ro[a].flags) | flags;
    __threadfence();
  }
  __syncthreads();
}

// Threshold + denominator of one row; leaves chunk sums of the row's weights in the scratch.
template <typename T>
__device__ RowStats row_statistics(Row<T> &row, uint4 *stage, Scratch &sc, int top_k, float inv_t,
                                   PRowWeights<T> &f) {
  using E = Elt<T>;
  const bool need_select = top_k < row.V;
  const uint32_t kmax = stage_first_pass<T>(row, stage, sc, need_select);
  RowStats st;
  st.flags = sc.bad ? SJD_FLAG_NONFINITE : 0u;
  st.tau_key = need_select ? select_threshold<T>(row, sc, (uint32_t)top_k) : 0u;
  st.xmax = E::val(E::unkey(kmax));
  f.row = row;
  f.pw.init(st, inv_t);
  chunk_sums<E::VEC>(f, row.NV, sc);
  st.z = (float)sc.chunk_excl[(row.NV + 31) >> 5];
  return st;
}

// ------------------------------------------------------------------------------------ initialisation (c)
// Sec. 4.2 (c): every slot that enters the window draws its token from the distribution predicted at its left
// neighbour: the most recent logits row of the nearest position to the left that has been through a pass,
// which is row min(t - 1 - n, W_eff - 1) of this pass (n: fixed tokens before the pass).  Run by every
// thread of the sequence's last block before the slide; one inverse-CDF draw over the row per new slot
// (the chunk sums are shared by consecutive slots that draw from the same row).
template <typename T>
__device__ void draw_fresh_slots(const VerifyParams &p, int b, uint32_t step, int cur, Scratch &sc) {
  using E = Elt<T>;
  const int tid = threadIdx.x, lane = tid & 31;
  const int W = p.W;
  const int sb = p.paired ? 2 * b : b;
  const int w_eff = p.w_eff ? p.w_eff[sb] : W;
  const RowOut *ro = p.row_out + (size_t)b * W;
  if (tid < 32) {
    int first = w_eff;
    for (int k = lane; k < w_eff; k += 32)
      if (!__ldcg(&ro[k].accept)) first = min(first, k);
    first = __reduce_min_sync(0xffffffffu, first);
    if (lane == 0) sc.sel_chunk = first;
  }
  __syncthreads();
  const int a = sc.sel_chunk;
  __syncthreads();
  const int m = (a < w_eff) ? a + 1 : w_eff;
  const int base = p.st.n[sb], n2 = base + m;
  const int prompt_len = p.st.prompt_lens[sb];
  const int w2 = max(0, min(W, prompt_len + p.st.n_generate - n2));
  int kept = (a < w_eff) ? min(w_eff - a - 1, w2) : 0;
  if (p.schedule == SJD_SCHEDULE_NO_REFINE) kept = 0;
  const float inv_t = 1.0f / p.temperature;
  int have = -1;   // row whose chunk sums are in the scratch
  for (int s = kept; s < w2; ++s) {
    const int t_pos = n2 + s;
    // k: row of this pass's buffer (>= 0), or -2 - slot for a slot of the ring, or -1: no row
    int k = -1;
    if (p.st.init == SJD_INIT_RESAMPLE_LEFT) {
      if (w_eff > 0) k = min(t_pos - 1 - base, w_eff - 1);
    } else {   // (d): the position one grid row above; its most recent row is in this pass's buffer if it was
               // inside the window just verified, else in the ring (every image position passes through a window)
      const int src = t_pos - p.st.grid_stride;
      if (src >= prompt_len) {
        if (src >= base) k = src - base < w_eff ? src - base : -1;
        else if (p.ring) k = -2 - src % p.ring_len;
      }
    }
    if (k == -1) {
      if (tid == 0) sc.fresh_row[s] = -1;
      continue;
    }
    const bool from_ring = k < -1;
    const int slot = from_ring ? -2 - k : k;
    const RowRefs<T> rows = row_refs<T>(p, b, from_ring ? 0 : slot, from_ring ? slot : 0, cur, from_ring);
    const RowStats *sp = from_ring ? rows.qstats : &p.stats[cur][(size_t)b * W + slot];
    const uint4 su = __ldcg(reinterpret_cast<const uint4 *>(sp));
    RowStats st;
    st.tau_key = su.x; st.xmax = __uint_as_float(su.y); st.z = __uint_as_float(su.z); st.flags = su.w;
    PRowWeights<T> f;
    if (from_ring) f.row.init(rows.q, p.V);
    else f.row.init(rows.p, p.V, rows.p2, p.guidance);
    f.pw.init(st, inv_t);
    if (k != have) {
      chunk_sums<E::VEC>(f, f.row.NV, sc);
      have = k;
    }
    const Philox4 rnd = philox4x32_10((uint32_t)t_pos, step, p.seq_base + (uint32_t)b, kStreamInit, p.seed_lo, p.seed_hi);
    sample_icdf<E::VEC>(f, f.row.NV, f.row.off, sc, u24(rnd.w[0]));
    if (tid == 0) {
      sc.fresh_tok[s] = sc.tok;
      sc.fresh_q[s] = sc.tok_w / st.z;
      sc.fresh_row[s] = slot;
      sc.fresh_kind[s] = from_ring ? SJD_Q_RING : SJD_Q_ROW;
    }
    __syncthreads();
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------ finalize
// Run by every thread of the last block of sequence b: accept scan (warp 0), then the commit, the
// window slide and the next inputs in parallel over the window slots.  Under guidance "sequence b" is
// image b: its window is kept twice, in the state of the conditional stream (sequence 2b) and of the
// unconditional one (2b + 1); both copies are read from the first and written identically, except that
// each stream's fixed tokens (and so its next first input) go to its own token array.
__device__ void finalize_sequence(const VerifyParams &p, int b, uint32_t step, Scratch &sc) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
  const int W = p.W;
  const int sb = p.paired ? 2 * b : b, n_streams = p.paired ? 2 : 1;
  const int w_eff = p.w_eff ? p.w_eff[sb] : W;
  const RowOut *ro = p.row_out + (size_t)b * W;
  const int32_t *old_draft = p.draft + (size_t)sb * W;
  const sjd_step_out &o = p.out;
  if (tid < 32) {
    int first = w_eff;
    for (int k = lane; k < w_eff; k += 32)
      if (!__ldcg(&ro[k].accept)) first = min(first, k);
    const int a = __reduce_min_sync(0xffffffffu, first);
    uint32_t fl = 0;
    for (int k = lane; k < w_eff; k += 32) {
      const uint32_t rf = __ldcg(&ro[k].flags);
      fl |= rf & SJD_FLAG_NONFINITE;
      if (k <= a) fl |= rf & SJD_FLAG_NEAR_TIE_ACCEPT;   // the rows the left-to-right scan looks at
      if (k == a) fl |= rf & SJD_FLAG_RESIDUAL_EMPTY;
    }
    fl = __reduce_or_sync(0xffffffffu, fl);
    if (lane == 0) {
      sc.sel_chunk = a;
      sc.sel_bin = fl;
    }
  }
  __syncthreads();
  const int a = sc.sel_chunk;
  uint32_t flags = sc.sel_bin;
  const int m = (a < w_eff) ? a + 1 : w_eff;
  const int base = p.e2e ? p.st.n[sb] : (p.base_pos ? p.base_pos[b] : 0);
  const int n2 = base + m;

  // fixed tokens: accepted drafts, then the resampled one
  for (int i = tid; i < W; i += nt) {
    int tok = -1;
    if (i < a) tok = old_draft[i];
    else if (i == a && a < w_eff) tok = __ldcg(&ro[a].resample_tok);
    if (o.committed) o.committed[(size_t)b * W + i] = tok;
    if (p.e2e && i < m)
      for (int s2 = 0; s2 < n_streams; ++s2) p.st.committed[(size_t)(sb + s2) * p.st.max_seq + base + i] = tok;
  }

  int w2 = 0, kept = 0;
  if (p.e2e) {
    const int total = p.st.prompt_lens[sb] + p.st.n_generate;
    w2 = max(0, min(W, total - n2));
    kept = (a < w_eff) ? min(w_eff - a - 1, w2) : 0;
    if (p.schedule == SJD_SCHEDULE_NO_REFINE) kept = 0;   // every slot of the new window is initialised afresh
    if (n2 >= total) flags |= SJD_FLAG_DONE;
  } else {
    kept = (a < w_eff && p.schedule != SJD_SCHEDULE_NO_REFINE) ? (w_eff - a - 1) : 0;
    w2 = kept;
  }
  int32_t *nd = p.e2e ? p.st.draft + (size_t)sb * W : nullptr;
  // A copied slot may read a slot filled just before it (and a token fixed above), so the copy
  // initialisations fill the window in order on one thread; everything else goes slot-parallel.
  const bool serial = p.e2e && p.st.init != SJD_INIT_RANDOM;
  if (serial) __syncthreads();   // the fixed tokens above are read below
  for (int s = serial ? 0 : tid; s < W && (!serial || tid == 0); s += serial ? 1 : nt) {
    int tok = -1, kind = -1, qrow = 0;
    float q = 0.0f;
    if (s < kept) {
      const int k = a + 1 + s;
      tok = __ldcg(&ro[k].redraft_tok);
      q = __ldcg(&ro[k].redraft_p);
      kind = SJD_Q_ROW;
      qrow = k;
    } else if (s < w2 && (p.st.init == SJD_INIT_RESAMPLE_LEFT || p.st.init == SJD_INIT_RESAMPLE_ABOVE) &&
               sc.fresh_row[s] >= 0) {  // Sec. 4.2 (c), (d)
      tok = sc.fresh_tok[s];
      q = sc.fresh_q[s];
      kind = sc.fresh_kind[s];
      qrow = sc.fresh_row[s];
    } else if (s < w2) {  // freshly initialised slot (end-to-end mode only), Sec. 4.2
      const int t_pos = n2 + s;
      const int stride = p.st.init == SJD_INIT_COPY_ABOVE ? p.st.grid_stride
                         : p.st.init == SJD_INIT_COPY_LEFT ? 1 : 0;
      const int src = t_pos - stride;
      if (p.st.init != SJD_INIT_RANDOM && stride > 0 && src >= p.st.prompt_lens[sb]) {
        tok = src < n2 ? p.st.committed[(size_t)sb * p.st.max_seq + src] : nd[src - n2];
        kind = SJD_Q_ONEHOT;
        q = 1.0f;
      } else {
        const Philox4 r = philox4x32_10((uint32_t)t_pos, step, p.seq_base + (uint32_t)b, kStreamInit,
                                        p.seed_lo, p.seed_hi);
        tok = (int)(((uint64_t)r.w[0] * (uint64_t)p.V) >> 32);
        kind = SJD_Q_UNIFORM;
        q = 1.0f / (float)p.V;
      }
    }
    if (p.e2e) {
      for (int s2 = 0; s2 < n_streams; ++s2) {
        const size_t at = (size_t)(sb + s2) * W + s;
        p.st.draft[at] = tok;
        p.st.q_kind[at] = kind;
        p.st.q_row[at] = qrow;
        p.st.q_draft[at] = q;
      }
    }
    if (o.draft) o.draft[(size_t)b * W + s] = tok;
    if (o.q_kind) o.q_kind[(size_t)b * W + s] = kind;
    if (o.q_draft) o.q_draft[(size_t)b * W + s] = q;
  }
  __syncthreads();   // the new window and the fixed tokens are read below
  if (p.e2e) {
    for (int s2 = 0; s2 < n_streams; ++s2) {
      int32_t *it = p.st.in_tok + (size_t)(sb + s2) * W;
      int32_t *ip = p.st.in_pos + (size_t)(sb + s2) * W;
      for (int k = tid; k < W; k += nt) {
        const bool act = k < w2;
        it[k] = act ? (k == 0 ? p.st.committed[(size_t)(sb + s2) * p.st.max_seq + n2 - 1] : nd[k - 1]) : 0;
        ip[k] = act ? n2 - 1 + k : -1;
      }
    }
  }
  if (tid == 0) {
    if (p.e2e) {
      for (int s2 = 0; s2 < n_streams; ++s2) {
        p.st.n[sb + s2] = n2;
        p.st.w_eff[sb + s2] = w2;
      }
    }
    if (p.n_prev) {   // what the retaining copy after this launch goes by (Sec. 4.2 (d))
      p.n_prev[b] = base;
      p.w_prev[b] = w_eff;
    }
    if (o.n_accepted) o.n_accepted[b] = a;
    if (o.n_committed) o.n_committed[b] = m;
    if (o.total_committed) o.total_committed[b] = n2;
    if (o.flags) o.flags[b] = flags;
  }
}

// ------------------------------------------------------------------------------------ kernel
// STREAM: the instantiation launched for bf16 rows too long for the registers of a block (see long_statistics)
template <typename T, int MAXT, bool STREAM = false>
__global__ void __launch_bounds__(MAXT, MAXT <= 256 ? SJD_VERIFY_MIN_BLOCKS : 1) verify_rows_kernel(const VerifyParams p) {
  using E = Elt<T>;
  extern __shared__ uint4 dyn_smem[];
  __shared__ Scratch sc;
  uint4 *stage = p.staged ? dyn_smem : nullptr;
  pdl_trigger();
  SJD_TL(TL_VERIFY, 0, threadIdx.x == 0);
  pdl_wait();   // the logits come from the preceding kernel
  SJD_TL(TL_VERIFY, 1, threadIdx.x == 0);

  const int r = blockIdx.x;
  const int b = r / p.W, k = r % p.W;
  const int sb = p.paired ? 2 * b : b;   // sequence whose state describes the window (under guidance both streams' do)
  const int rs = sb * p.W + k;
  const int tid = threadIdx.x;
  const int w_eff = p.w_eff ? p.w_eff[sb] : p.W;
  const uint32_t step = p.step_ptr ? *p.step_ptr : p.step;
  const int cur = p.step_ptr ? (int)(step & 1u) : 0;
  const float inv_t = 1.0f / p.temperature;

  if (k < w_eff) {
    // (the Jacobi schedule compares tokens and uses no q: treat every draft as a copied one)
    const int kind_raw = p.q_kind ? p.q_kind[rs] : SJD_Q_ROW;
    const bool q_ring = kind_raw == SJD_Q_RING;   // a retained row: the same law as a row of the other buffer
    const int kind = p.schedule == SJD_SCHEDULE_JACOBI ? SJD_Q_ONEHOT : (q_ring ? SJD_Q_ROW : kind_raw);
    const int d = p.draft[rs];
    const bool d_ok = d >= 0 && d < p.V;
    const int qr = p.q_row ? p.q_row[rs] : k;
    const int base = p.e2e ? p.st.n[sb] : (p.base_pos ? p.base_pos[b] : 0);
    const Philox4 rnd = philox4x32_10((uint32_t)(base + k), step, p.seq_base + (uint32_t)b, kStreamVerify,
                                      p.seed_lo, p.seed_hi);
    const float u_acc = u24(rnd.w[0]), u_res = u24(rnd.w[1]);
    float u_draft = u24(rnd.w[2]);
    const bool jacobi = p.schedule == SJD_SCHEDULE_JACOBI;
    if (jacobi)   // Sec. 3.2: the draw of a position uses the same uniform in every pass (step index 0)
      u_draft = u24(philox4x32_10((uint32_t)(base + k), 0u, p.seq_base + (uint32_t)b, kStreamVerify, p.seed_lo, p.seed_hi).w[2]);
    const RowRefs<T> rows = row_refs<T>(p, b, k, qr, cur, q_ring);

    RowOut fast_out;
    const bool fast_done = p.fast && (((uintptr_t)rows.q | (uintptr_t)rows.p) & 15u) == 0 &&
                           fast_row<T, STREAM>(p, sc, r, b, kind, d, qr, cur, rows, inv_t, u_acc, u_res, u_draft, fast_out);
    if (fast_done) {
      if (tid == 0) p.row_out[r] = fast_out;
    } else {
    __syncthreads();
    // ---- the law of the draft
    Row<T> qrow;
    qrow.init(rows.q, p.V, rows.q2, p.guidance);
    RowStats qs;
    qs.tau_key = 0; qs.xmax = 0.0f; qs.z = 1.0f; qs.flags = 0;
    PRowWeights<T> qf;
    float q_d;
    if (kind == SJD_Q_ROW) {
      if (p.prev_stats_valid) {
        qs = *rows.qstats;
      } else {
        qs = row_statistics<T>(qrow, stage, sc, p.top_k, inv_t, qf);
        if (tid == 0) p.stats[cur ^ 1][r] = qs;
        __syncthreads();
        qrow.s = nullptr;  // the staging buffer is about to be reused
      }
      qf.row = qrow;
      qf.pw.init(qs, inv_t);
      q_d = d_ok ? qf.pw.one(qrow.element(d), d) / qs.z : 1.0f;
    } else if (kind == SJD_Q_UNIFORM) {
      q_d = 1.0f / (float)p.V;
    } else {
      q_d = 1.0f;
    }

    SJD_TL(TL_VERIFY, 10, tid == 0);   // the draft's law is known
    // ---- this iteration's distribution
    Row<T> prow;
    prow.init(rows.p, p.V, rows.p2, p.guidance);
    PRowWeights<T> pf;
    const RowStats ps = row_statistics<T>(prow, stage, sc, p.top_k, inv_t, pf);
    if (tid == 0) p.stats[cur][r] = ps;
    const float p_d = d_ok ? pf.pw.one(prow.element(d), d) / ps.z : 0.0f;

    SJD_TL(TL_VERIFY, 11, tid == 0);   // this row's statistics are known
    // ---- Eq. 1
    float ratio;
    if (q_d > 0.0f) ratio = p_d / q_d;
    else ratio = p_d > 0.0f ? INFINITY : 0.0f;
    float thr = fminf(1.0f, ratio);
    bool accept = u_acc < thr;
    uint32_t flags = ps.flags | (kind == SJD_Q_ROW ? qs.flags : 0u);
    if (thr < 1.0f && fabsf(u_acc - thr) < 1e-4f) flags |= SJD_FLAG_NEAR_TIE_ACCEPT;

    // ---- Eq. 3: re-draft from p (used if an earlier row rejects)
    sample_icdf<E::VEC>(pf, prow.NV, prow.off, sc, u_draft);
    const int redraft_tok = sc.tok;
    const float redraft_p = sc.tok_w / ps.z;
    __syncthreads();

    SJD_TL(TL_VERIFY, 12, tid == 0);   // re-draft token drawn
    // ---- Eq. 2: residual resample (used if this is the first rejected row)
    int resample_tok = -1;
    if (jacobi) {   // deterministic criterion instead of Eqs. 1-2
      accept = d_ok && redraft_tok == d;
      thr = accept ? 1.0f : 0.0f;
      flags &= ~SJD_FLAG_NEAR_TIE_ACCEPT;
      resample_tok = accept ? -1 : redraft_tok;
    } else if (!accept) {
      ResidualWeights<T> rf;
      rf.prow = prow; rf.qrow = qrow; rf.pw = pf.pw; rf.qw = qf.pw;
      rf.inv_zp = 1.0f / ps.z; rf.inv_zq = 1.0f / qs.z;
      rf.kind = kind; rf.draft = d; rf.V = p.V;
      if (kind != SJD_Q_ROW) rf.qw = pf.pw;
      chunk_sums<E::VEC>(rf, prow.NV, sc);
      if (sc.chunk_excl[(prow.NV + 31) >> 5] > 0.0) {
        sample_icdf<E::VEC>(rf, prow.NV, prow.off, sc, u_res);
      } else {
        flags |= SJD_FLAG_RESIDUAL_EMPTY;
        __syncthreads();
        chunk_sums<E::VEC>(pf, prow.NV, sc);
        sample_icdf<E::VEC>(pf, prow.NV, prow.off, sc, u_res);
      }
      resample_tok = sc.tok;
    }
    SJD_TL(TL_VERIFY, 13, tid == 0);   // residual token drawn
    if (tid == 0) {
      RowOut ro;
      ro.p_draft = p_d; ro.q_draft = q_d; ro.thr = thr; ro.accept = accept ? 1 : 0;
      ro.redraft_tok = redraft_tok; ro.redraft_p = redraft_p; ro.resample_tok = resample_tok; ro.flags = flags;
      p.row_out[r] = ro;
    }
    }   // general route
  }

  // ---- ticket: the last block of the sequence slides the window
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const int old = atomicAdd(&p.seq_counter[b], 1);
    sc.is_last = (old == p.W - 1);
  }
  __syncthreads();
  if (!sc.is_last) return;
  __threadfence();
  SJD_TL(TL_VERIFY, 14, tid == 0);
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    if (p.fast && p.defer_residual) deferred_residual_bf16<STREAM>(p, b, step, cur, sc);
  }
  if (p.e2e && (p.st.init == SJD_INIT_RESAMPLE_LEFT || p.st.init == SJD_INIT_RESAMPLE_ABOVE))
    draw_fresh_slots<T>(p, b, step, cur, sc);
  finalize_sequence(p, b, step, sc);
  SJD_TL(TL_VERIFY, 15, tid == 0);
  __syncthreads();
  if (tid == 0) {
    p.seq_counter[b] = 0;
    __threadfence();
    const int done = atomicAdd(p.done_counter, 1);
    if (done == p.B - 1) {  // every block has read the step index by now
      *p.done_counter = 0;
      if (p.step_ptr) *p.step_ptr = step + 1u;
    }
  }
}

// Sec. 4.2 (d): keep the rows of the window just verified (as the verification saw them: mixed under
// guidance) and their statistics in the ring, slot = position % ring_len; one block per (row, image).
template <typename T>
__global__ void retain_rows_kernel(const VerifyParams p) {
  pdl_trigger();
  pdl_wait();
  const int k = blockIdx.x, b = blockIdx.y;
  if (k >= p.w_prev[b]) return;
  const uint32_t step = *p.step_ptr - 1u;          // the verification before this kernel has bumped the index
  const int cur = (int)(step & 1u);
  const int slot = (p.n_prev[b] + k) % p.ring_len;
  Row<T> row;
  const RowRefs<T> rows = row_refs<T>(p, b, k, 0, cur);
  row.init(rows.p, p.V, rows.p2, p.guidance);
  T *dst = reinterpret_cast<T *>(p.ring) + ((size_t)b * p.ring_len + slot) * p.V;
  unsigned short *d16 = reinterpret_cast<unsigned short *>(dst);
  uint32_t *d32 = reinterpret_cast<uint32_t *>(dst);
  for (int i = threadIdx.x; i < p.V; i += blockDim.x) {
    const uint32_t bits = row.raw_bits(i);
    if (sizeof(T) == 2) d16[i] = (unsigned short)bits;
    else d32[i] = bits;
  }
  if (threadIdx.x == 0) p.ring_stats[(size_t)b * p.ring_len + slot] = p.stats[cur][(size_t)b * p.W + k];
}

}  // namespace

int launch_retain_rows(const VerifyParams &p, int dtype, cudaStream_t stream) {
  if (!p.ring || !p.ring_stats || p.ring_len < 1 || !p.n_prev || !p.w_prev || !p.step_ptr) return SJD_ERR_BAD_ARG;
  const dim3 grid(p.W, p.B);
  if (dtype == SJD_F32) SJD_CUDA(launch_kernel(retain_rows_kernel<float>, grid, dim3(256), 0, stream, p));
  else if (dtype == SJD_BF16) SJD_CUDA(launch_kernel(retain_rows_kernel<__nv_bfloat16>, grid, dim3(256), 0, stream, p));
  else return SJD_ERR_UNSUPPORTED;
  SJD_CHECK_LAUNCH();
  return SJD_OK;
}

size_t verify_scratch_bytes(int batch, int window) {
  if (batch <= 0 || window <= 0) return 0;
  const size_t rows = (size_t)batch * window;
  size_t b = 0;
  b += 2 * rows * sizeof(RowStats);
  b += rows * sizeof(RowOut);
  b += ((size_t)batch + 1) * sizeof(int32_t);
  return (b + 255) / 256 * 256;
}

template <typename T>
static int launch_verify_t(const VerifyParams &p_in, cudaStream_t stream) {
  VerifyParams p = p_in;
  constexpr int VEC = Elt<T>::VEC;
  const long nv_max = ((long)p.V + 2 * VEC - 2) / VEC + 1;
  if ((nv_max + 31) / 32 > kMaxChunks) return SJD_ERR_CAPACITY;
  const size_t stage_bytes = (size_t)nv_max * 16;
  p.staged = stage_bytes <= 160 * 1024 ? 1 : 0;
  int threads = nv_max <= 1024 ? 128 : nv_max <= 4096 ? 256 : nv_max <= 16384 ? 512 : 1024;
  // rows a block can hold in registers, eight vectors per thread
  p.fast = 0;
  // (longer rows, up to kMaxChunks chunks, stream through the registers of a full block in segments)
  const bool in_registers = p.V / VEC <= 8 * kMaxThreads;
  if (std::is_same<T, __nv_bfloat16>::value && (p.staged || !in_registers) && p.V % VEC == 0 &&
      ((uintptr_t)p.logits[0] & 15u) == 0 && ((uintptr_t)p.logits[1] & 15u) == 0) {
    p.fast = 1;
    threads = in_registers ? (p.V / VEC + 255) / 256 * 32 : kMaxThreads;
    threads = threads < 64 ? 64 : threads;
    // no staging buffer: the rows live in registers; the odd row that needs the general route (a NaN, a
    // threshold out of the histogram's reach) re-reads global memory instead, and more blocks fit an SM
    p.staged = 0;
    // more blocks than can be resident at once: rejected rows leave the Eq. 2 draw to the sequence's last block
    static int n_sms = 0;
    if (n_sms == 0) {
      int dev = 0, v = 0;
      if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess)
        n_sms = v;
    }
    const int resident = (n_sms > 0 ? n_sms : 148) * (threads <= 256 ? SJD_VERIFY_MIN_BLOCKS : 1);
    p.defer_residual = p.B * p.W > resident ? 1 : 0;
  }
  const size_t dyn = p.staged ? stage_bytes : 0;
  auto launch = [&](auto kernel) -> int {
    // static scratch (about 30 KB) + the staged row: opt in as soon as the sum can pass 48 KB
    if (dyn > 16 * 1024) SJD_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn));
    SJD_CUDA(launch_kernel(kernel, dim3(p.B * p.W), dim3(threads), dyn, stream, p));
    SJD_CHECK_LAUNCH();
    return SJD_OK;
  };
  if (threads <= 256) return launch(verify_rows_kernel<T, 256>);
  if (p.fast && !in_registers) return launch(verify_rows_kernel<T, kMaxThreads, true>);
  return launch(verify_rows_kernel<T, kMaxThreads>);
}

int launch_verify(const VerifyParams &p, int dtype, cudaStream_t stream) {
  if (dtype == SJD_F32) return launch_verify_t<float>(p, stream);
  if (dtype == SJD_BF16) return launch_verify_t<__nv_bfloat16>(p, stream);
  return SJD_ERR_UNSUPPORTED;
}

}  // namespace sjd
