// Aggregation kernels: out[r] = rs_r * sum_k s_k * X[idx[k]] over one segment of a CSR (forward)
// or CSC (backward) structure.  This is the pull loop of Algorithm 1 of the paper; the register
// accumulation with one store per row follows the idea of Algorithm 3, and cutting the source
// vertices into blocks whose rows of X stay L2-resident is Algorithm 2 with L2 in the role of
// the CPU cache (one launch per block, later launches adding to the output).
//
// Work decomposition
//   light segments (length <= heavy_threshold): every warp owns rows_per_warp consecutive
//     segments and reads their indices as one contiguous stream of 32-edge batches (one edge
//     per lane, next batch prefetched), so short rows share coalesced index loads.  Lanes are
//     spread along the feature dimension with 16-, 8- or 4-byte vector loads.  When a row slice
//     needs fewer than 32 vectors the warp is cut into groups of G lanes and the groups take
//     different edges of the same segment; their partial sums are combined by a fixed shuffle
//     tree.  U load steps per lane are in flight before the first add.
//   heavy segments: one thread block per segment; the first blocks of the same launch (as many
//     as the device keeps resident) loop over the heavy list, which is ordered longest first;
//     the 8 warps take interleaved batches of 32 edges and combine in shared memory in warp
//     order.
// Every output element is produced by one thread in an order fixed by the launch shape, so the
// result is deterministic and needs no atomics in either direction.
#ifndef DG_AGGREGATE_KERNELS_CUH_
#define DG_AGGREGATE_KERNELS_CUH_
#include "dg_internal.cuh"

namespace dg {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kBlock = kWarpsPerBlock * 32;
constexpr unsigned kFull = 0xffffffffu;

// Accumulators are fp32 vectors of VEC floats; f8 is the 8-wide one (two float4).
struct f8 { float4 lo, hi; };
template <int VEC> struct Vec;
template <> struct Vec<1> { using T = float; };
template <> struct Vec<2> { using T = float2; };
template <> struct Vec<4> { using T = float4; };
template <> struct Vec<8> { using T = f8; };

// Storage type of the gathered matrix: fp32, or bf16 (halves every gathered byte; the sums
// stay fp32).  Pack<E, VEC>::Load is what one lane loads for VEC consecutive elements.
struct F32 { static constexpr int kBytes = 4; };
struct BF16 { static constexpr int kBytes = 2; };
template <typename E, int VEC> struct Pack { using Load = typename Vec<VEC>::T; };
template <> struct Pack<BF16, 2> { using Load = uint32_t; };
template <> struct Pack<BF16, 4> { using Load = uint2; };
template <> struct Pack<BF16, 8> { using Load = uint4; };

__device__ __forceinline__ float ldg_vec(const char* p, float) {
  return __ldg(reinterpret_cast<const float*>(p));
}
__device__ __forceinline__ float2 ldg_vec(const char* p, float2) {
  return __ldg(reinterpret_cast<const float2*>(p));
}
__device__ __forceinline__ float4 ldg_vec(const char* p, float4) {
  return __ldg(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ uint32_t ldg_vec(const char* p, uint32_t) {
  return __ldg(reinterpret_cast<const uint32_t*>(p));
}
__device__ __forceinline__ uint2 ldg_vec(const char* p, uint2) {
  return __ldg(reinterpret_cast<const uint2*>(p));
}
__device__ __forceinline__ uint4 ldg_vec(const char* p, uint4) {
  return __ldg(reinterpret_cast<const uint4*>(p));
}
// a 32-bit word holds two bf16 values: the low half is the element with the lower index
__device__ __forceinline__ float bf_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
// element i of a matrix stored as E
template <typename E> __device__ __forceinline__ float ld_elem(const void* X, size_t i);
template <> __device__ __forceinline__ float ld_elem<F32>(const void* X, size_t i) {
  return __ldg(reinterpret_cast<const float*>(X) + i);
}
template <> __device__ __forceinline__ float ld_elem<BF16>(const void* X, size_t i) {
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(X) + i) << 16);
}
// 1 / (in-degree + 1) of vertex r, from the CSR row pointer
__device__ __forceinline__ float self_factor(const int64_t* self_ptr, int64_t r) {
  return 1.0f / (float)(__ldg(self_ptr + r + 1) - __ldg(self_ptr + r) + 1);
}
__device__ __forceinline__ float ld_vec(const float* p, float) { return *p; }
__device__ __forceinline__ float2 ld_vec(const float* p, float2) {
  return *reinterpret_cast<const float2*>(p);
}
__device__ __forceinline__ float4 ld_vec(const float* p, float4) {
  return *reinterpret_cast<const float4*>(p);
}
__device__ __forceinline__ f8 ld_vec(const float* p, f8) {
  f8 v;
  v.lo = *reinterpret_cast<const float4*>(p);
  v.hi = *reinterpret_cast<const float4*>(p + 4);
  return v;
}
__device__ __forceinline__ void zero(uint32_t& a) { a = 0u; }
__device__ __forceinline__ void zero(uint2& a) { a.x = a.y = 0u; }
__device__ __forceinline__ void zero(uint4& a) { a.x = a.y = a.z = a.w = 0u; }
__device__ __forceinline__ void zero(float& a) { a = 0.f; }
__device__ __forceinline__ void zero(float2& a) { a.x = a.y = 0.f; }
__device__ __forceinline__ void zero(float4& a) { a.x = a.y = a.z = a.w = 0.f; }
__device__ __forceinline__ void add(float& a, const float& v) { a += v; }
__device__ __forceinline__ void add(float2& a, const float2& v) { a.x += v.x; a.y += v.y; }
__device__ __forceinline__ void add(float4& a, const float4& v) {
  a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
}
__device__ __forceinline__ void zero(f8& a) { zero(a.lo); zero(a.hi); }
__device__ __forceinline__ void add(f8& a, const f8& v) { add(a.lo, v.lo); add(a.hi, v.hi); }
// packed bf16 loads into fp32 accumulators
__device__ __forceinline__ void add(float2& a, uint32_t v) { a.x += bf_lo(v); a.y += bf_hi(v); }
__device__ __forceinline__ void add(float4& a, uint2 v) {
  a.x += bf_lo(v.x); a.y += bf_hi(v.x); a.z += bf_lo(v.y); a.w += bf_hi(v.y);
}
__device__ __forceinline__ void add(f8& a, uint4 v) {
  add(a.lo, make_uint2(v.x, v.y));
  add(a.hi, make_uint2(v.z, v.w));
}
__device__ __forceinline__ void fma(float2& a, float s, uint32_t v) {
  a.x = fmaf(s, bf_lo(v), a.x); a.y = fmaf(s, bf_hi(v), a.y);
}
__device__ __forceinline__ void fma(float4& a, float s, uint2 v) {
  a.x = fmaf(s, bf_lo(v.x), a.x); a.y = fmaf(s, bf_hi(v.x), a.y);
  a.z = fmaf(s, bf_lo(v.y), a.z); a.w = fmaf(s, bf_hi(v.y), a.w);
}
__device__ __forceinline__ void fma(f8& a, float s, uint4 v) {
  fma(a.lo, s, make_uint2(v.x, v.y));
  fma(a.hi, s, make_uint2(v.z, v.w));
}
__device__ __forceinline__ void fma(float& a, float s, const float& v) { a = fmaf(s, v, a); }
__device__ __forceinline__ void fma(float2& a, float s, const float2& v) {
  a.x = fmaf(s, v.x, a.x); a.y = fmaf(s, v.y, a.y);
}
__device__ __forceinline__ void fma(float4& a, float s, const float4& v) {
  a.x = fmaf(s, v.x, a.x); a.y = fmaf(s, v.y, a.y);
  a.z = fmaf(s, v.z, a.z); a.w = fmaf(s, v.w, a.w);
}
__device__ __forceinline__ void scale(float& a, float s) { a *= s; }
__device__ __forceinline__ void scale(float2& a, float s) { a.x *= s; a.y *= s; }
__device__ __forceinline__ void scale(float4& a, float s) { a.x *= s; a.y *= s; a.z *= s; a.w *= s; }
__device__ __forceinline__ void scale(f8& a, float s) { scale(a.lo, s); scale(a.hi, s); }
__device__ __forceinline__ float shfl_xor(float a, int m) { return __shfl_xor_sync(kFull, a, m); }
__device__ __forceinline__ float2 shfl_xor(float2 a, int m) {
  return make_float2(__shfl_xor_sync(kFull, a.x, m), __shfl_xor_sync(kFull, a.y, m));
}
__device__ __forceinline__ float4 shfl_xor(float4 a, int m) {
  return make_float4(__shfl_xor_sync(kFull, a.x, m), __shfl_xor_sync(kFull, a.y, m),
                     __shfl_xor_sync(kFull, a.z, m), __shfl_xor_sync(kFull, a.w, m));
}
__device__ __forceinline__ f8 shfl_xor(f8 a, int m) {
  f8 r;
  r.lo = shfl_xor(a.lo, m);
  r.hi = shfl_xor(a.hi, m);
  return r;
}
__device__ __forceinline__ void stcs_vec(float* p, float v) { __stcs(p, v); }
__device__ __forceinline__ void stcs_vec(float* p, float2 v) { __stcs(reinterpret_cast<float2*>(p), v); }
__device__ __forceinline__ void stcs_vec(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }
__device__ __forceinline__ void stcs_vec(float* p, f8 v) {
  __stcs(reinterpret_cast<float4*>(p), v.lo);
  __stcs(reinterpret_cast<float4*>(p + 4), v.hi);
}
__device__ __forceinline__ void st_smem(float* p, f8 v) {
  p[0] = v.lo.x; p[1] = v.lo.y; p[2] = v.lo.z; p[3] = v.lo.w;
  p[4] = v.hi.x; p[5] = v.hi.y; p[6] = v.hi.z; p[7] = v.hi.w;
}
__device__ __forceinline__ void st_smem(float* p, float v) { p[0] = v; }
__device__ __forceinline__ void st_smem(float* p, float2 v) { p[0] = v.x; p[1] = v.y; }
__device__ __forceinline__ void st_smem(float* p, float4 v) {
  p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w;
}
__device__ __forceinline__ void add_smem(float* p, float v) { p[0] += v; }
__device__ __forceinline__ void add_smem(float* p, float2 v) { p[0] += v.x; p[1] += v.y; }
__device__ __forceinline__ void add_smem(float* p, float4 v) {
  p[0] += v.x; p[1] += v.y; p[2] += v.z; p[3] += v.w;
}
__device__ __forceinline__ void add_smem(float* p, f8 v) {
  add_smem(p, v.lo);
  add_smem(p + 4, v.hi);
}

// Loads the neighbour id and the per-edge factor of the edge at position b + lane of the
// index stream (neutral values at or beyond `end`).
template <bool SCALED>
__device__ __forceinline__ void load_batch(const ApArgs& a, int64_t b, int end, int lane,
                                           int32_t& u, float& s) {
  u = 0;
  s = 0.f;
  const int64_t k = b + lane;
  if (k < end) {
    u = __ldcs(a.idx + k);
    if (SCALED) s = __ldcs(a.w + k);
  }
}

template <int VEC, int G, int CPL>
struct Shape {
  static constexpr int NG = 32 / G;  // edges one warp-wide load instruction covers
  // load steps in flight per lane (fewer when a step is several vectors wide), and no more
  // steps than one 32-edge batch holds
  static constexpr int U0 = CPL == 1 ? 8 : (CPL == 2 ? 4 : (VEC <= 2 ? 4 : 2));
  static constexpr int U = (U0 * NG > 32) ? (32 / NG) : U0;
};

// Adds the edges held in lanes [s, e) of the current batch (cur_u / cur_s: one edge per lane)
// into acc.  Lane group `grp` takes edges s+grp, s+grp+NG, ...  Full steps of U*NG edges run
// without predicates; the ragged end runs once with predicated loads.  xrow[c] is the address
// of this lane's c-th vector inside row 0 of X.
template <typename E, int VEC, int G, int CPL, bool SCALED, bool STAGE>
__device__ __forceinline__ void add_edges(const char* const (&xrow)[CPL], uint32_t row_bytes,
                                          int32_t cur_u, float cur_s, int s, int e, int grp,
                                          typename Vec<VEC>::T (&acc)[CPL], uint2* stage) {
  using V = typename Pack<E, VEC>::Load;  // as loaded; unpacked while adding
  constexpr int NG = Shape<VEC, G, CPL>::NG;
  constexpr int U = Shape<VEC, G, CPL>::U;
  int p = s;
  // With one vector per lane (8 steps in flight) the edge factors are fetched while adding, so
  // that they hold no registers during the loads: that regime lives on occupancy.  With wider
  // lanes (4 or 2 steps) they are fetched with the loads and the adds do not wait for a shuffle.
  constexpr bool kLate = CPL == 1;
  // Scaled, wide lanes, source-blocked (L2-resident) passes: the batch's (id, factor) pairs go
  // through shared memory, so that one 8-byte broadcast load per step replaces two shuffles:
  // fewer wavefronts on the load/store pipe, which is what bounds that case (Reddit-like
  // backward 20.0 -> 19.3 ms).  Passes with short row pieces lose more on the extra store and
  // warp barriers per call than they gain (Products-like F = 256: 14.0 -> 16.0 ms), so the
  // passes without source blocks keep the shuffles.
  constexpr bool kStaged = SCALED && !kLate && STAGE;
  if (kStaged) {
    __syncwarp();
    stage[threadIdx.x & 31] = make_uint2((uint32_t)cur_u, __float_as_uint(cur_s));
    __syncwarp();
  }
  for (; p + U * NG <= e; p += U * NG) {
    V v[U][CPL];
    float sc[kLate ? 1 : U];
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int src = p + j * NG + grp;
      uint32_t u;
      if (kStaged) {
        const uint2 us = stage[src];
        u = us.x;
        sc[j] = __uint_as_float(us.y);
      } else {
        u = (uint32_t)__shfl_sync(kFull, cur_u, src);
        if (SCALED && !kLate) sc[j] = __shfl_sync(kFull, cur_s, src);
      }
      const uint64_t off = (uint64_t)u * row_bytes;
#pragma unroll
      for (int c = 0; c < CPL; ++c) v[j][c] = ldg_vec(xrow[c] + off, V());
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
      float sj = 1.f;
      if (SCALED) sj = kLate ? __shfl_sync(kFull, cur_s, p + j * NG + grp) : sc[j];
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        if (SCALED) fma(acc[c], sj, v[j][c]);
        else add(acc[c], v[j][c]);
      }
    }
  }
  if (p < e) {
    V v[U][CPL];
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int src = p + j * NG + grp;
      const uint32_t u = (uint32_t)__shfl_sync(kFull, cur_u, src & 31);
      const uint64_t off = (uint64_t)u * row_bytes;
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        if (src < e) v[j][c] = ldg_vec(xrow[c] + off, V());
        else zero(v[j][c]);  // an absent edge adds zeros (times whatever factor its lane holds)
      }
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int src = p + j * NG + grp;
      float sj = SCALED ? __shfl_sync(kFull, cur_s, src & 31) : 1.f;
      if (SCALED && src >= e) sj = 0.f;  // lanes past the batch hold neutral factors, not NaNs
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        if (SCALED) fma(acc[c], sj, v[j][c]);
        else add(acc[c], v[j][c]);
      }
    }
  }
}

// Sums the partial results of the lane groups into group 0 (fixed tree).
template <int VEC, int G, int CPL>
__device__ __forceinline__ void combine_groups(typename Vec<VEC>::T (&acc)[CPL]) {
#pragma unroll
  for (int off = G; off < 32; off <<= 1) {
#pragma unroll
    for (int c = 0; c < CPL; ++c) add(acc[c], shfl_xor(acc[c], off));
  }
}

// Graphs that hold a segment of kLongSegment entries or more run the kernels compiled with
// FOLD: there a warp of a heavy segment moves its register sums into its shared-memory partial
// every kLongFold batches, so that no fp32 chain is longer than 32 * kLongFold = 512 terms however
// long the segment is (a segment of m entries is summed as chains of at most 512 terms, whose
// results form a second chain of m / 4096 terms per warp, and the 8 warp partials are added last).
// One register chain per warp, m / 8 terms, drifts past 1e-5 of the sum of magnitudes for
// same-sign inputs once m reaches about 10^6; below kLongSegment it is at most 4096 terms long.
// The fold is a second compilation of the kernels rather than a branch in one: in any of five
// forms tried (a counter in the loop, a second loop for long segments, a shared-memory counter,
// a function that is not inlined, a kernel of its own after the common one) it either changed the
// register allocation of the common kernels (Reddit-like backward 17.8 -> 18.7 ms) or serialised
// the long segments behind the rest (Papers-like backward 11.3 -> 16.0 ms at a tenth of the size).
constexpr int kLongSegment = 1 << 15;
constexpr int kLongFold = 16;

// Block-per-row path for the heavy segments: block x of the first `heavy_blocks` blocks takes
// entries x, x + heavy_blocks, ... of the heavy list; its 8 warps sum interleaved 32-edge
// batches and the partial sums are combined in shared memory in warp order.
template <typename E, int VEC, int G, int CPL, bool SCALED, bool SEG, bool SELF, bool FOLD>
__device__ __forceinline__ void heavy_rows(const ApArgs& a, const SelfArgs sa,
                                           const int heavy_blocks,
                                           float (&part)[kWarpsPerBlock][32 * CPL * VEC]) {
  using V = typename Vec<VEC>::T;
  __shared__ uint2 stage_heavy[kWarpsPerBlock][32];
  uint2* stage = stage_heavy[threadIdx.x >> 5];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int grp = lane / G;
  const int c0 = lane % G;
  const int f0 = blockIdx.y * a.slice_f;
  const int width = min(a.F, f0 + a.slice_f) - f0;
  const int chunks = width / VEC;
  const uint32_t row_bytes = (uint32_t)a.F * (uint32_t)E::kBytes;
  const char* xrow[CPL];
  bool cok[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) {
    const int ci = c0 + c * G;
    cok[c] = ci < chunks;
    xrow[c] = reinterpret_cast<const char*>(a.X) + (size_t)(f0 + (cok[c] ? ci : 0) * VEC) * E::kBytes;
  }
  const int count = min(*a.heavy_count, a.heavy_cap);
  for (int i = blockIdx.x; i < count; i += heavy_blocks) {
    const int64_t r = a.heavy_list[i];
    const int full = (int)(__ldg(a.ptr + r + 1) - __ldg(a.ptr + r));
    const int lo = SEG ? __ldg(a.seg_lo + r) : (int)__ldg(a.ptr + r);
    const int hi = SEG ? __ldg(a.seg_hi + r) : lo + full;
    V acc[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) zero(acc[c]);
    if (FOLD && lane < G) {
#pragma unroll
      for (int c = 0; c < CPL; ++c)
        if (cok[c]) st_smem(&part[warp][(c0 + c * G) * VEC], acc[c]);
    }
    // warp w sums batches w, w+8, ... of the segment
    int32_t cur_u, nxt_u;
    float cur_s, nxt_s;
    int b = hi - lo > warp * 32 ? lo + warp * 32 : hi;
    if (b < hi) load_batch<SCALED>(a, b, hi, lane, cur_u, cur_s);
    int since_fold = 0;
    while (b < hi) {
      const bool more = hi - b > kBlock;
      if (more) load_batch<SCALED>(a, (int64_t)b + kBlock, hi, lane, nxt_u, nxt_s);
      add_edges<E, VEC, G, CPL, SCALED, SEG>(xrow, row_bytes, cur_u, cur_s, 0, min(hi - b, 32), grp, acc,
                                     stage);
      if (FOLD && (++since_fold == kLongFold || !more)) {
        // the register sums join the warp's partial in shared memory and start afresh
        since_fold = 0;
        combine_groups<VEC, G, CPL>(acc);
        if (lane < G) {
#pragma unroll
          for (int c = 0; c < CPL; ++c)
            if (cok[c]) add_smem(&part[warp][(c0 + c * G) * VEC], acc[c]);
        }
#pragma unroll
        for (int c = 0; c < CPL; ++c) zero(acc[c]);
      }
      if (!more) break;
      b += kBlock;
      cur_u = nxt_u;
      cur_s = nxt_s;
    }
    if (!FOLD) {
      combine_groups<VEC, G, CPL>(acc);
      if (lane < G) {
#pragma unroll
        for (int c = 0; c < CPL; ++c)
          if (cok[c]) st_smem(&part[warp][(c0 + c * G) * VEC], acc[c]);
      }
    }
    __syncthreads();
    float* orow = a.Y + (size_t)r * (size_t)a.F + f0;
    if constexpr (SELF) {
      // the row's own input row joins the sum once, scaled like the mean's other terms
      const float ss = sa.self_mean ? self_factor(sa.self_ptr, r) : 1.0f;
      const bool own = !(SEG && a.accumulate);
      for (int f = threadIdx.x; f < width; f += kBlock) {
        float t = part[0][f];
#pragma unroll
        for (int w = 1; w < kWarpsPerBlock; ++w) t += part[w][f];
        if (a.mean_rows) t *= ss;
        if (own) t = fmaf(ss, ld_elem<E>(a.X, (size_t)r * (size_t)a.F + f0 + f), t);
        if (SEG && a.accumulate) t += orow[f];
        __stcs(orow + f, t);
      }
    } else {
      const float rs = a.mean_rows ? 1.0f / (float)full : 1.0f;
      for (int f = threadIdx.x; f < width; f += kBlock) {
        float t = part[0][f];
#pragma unroll
        for (int w = 1; w < kWarpsPerBlock; ++w) t += part[w][f];
        if (a.mean_rows) t *= rs;
        if (SEG && a.accumulate) t += orow[f];
        __stcs(orow + f, t);
      }
    }
    __syncthreads();
  }
}

// One launch does both roles: blocks [0, heavy_blocks) walk the heavy list (they are scheduled
// first, so the long segments start early); in the remaining blocks every warp owns
// rows_per_warp consecutive light segments and streams their indices as one run of 32-edge
// batches, the next batch always in flight while the current one is summed.
template <typename E, int VEC, int G, int CPL, bool SCALED, bool SEG, bool SELF, bool FOLD>
__device__ __forceinline__ void ap_body(const ApArgs& a, const SelfArgs sa,
                                        const int heavy_blocks,
                                        float (&part)[kWarpsPerBlock][32 * CPL * VEC]) {
  using V = typename Vec<VEC>::T;
  __shared__ uint2 stage_light[kWarpsPerBlock][32];
  uint2* stage = stage_light[threadIdx.x >> 5];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int grp = lane / G;
  const int c0 = lane % G;
  const int f0 = blockIdx.y * a.slice_f;
  const int fend = min(a.F, f0 + a.slice_f);
  const int width = fend - f0;
  const int chunks = width / VEC;
  const uint32_t row_bytes = (uint32_t)a.F * (uint32_t)E::kBytes;

  // Lanes whose vector falls beyond the slice re-read vector 0 and never store: the summing
  // loop then needs no per-lane predicate.
  const char* xrow[CPL];
  bool cok[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) {
    const int ci = c0 + c * G;
    cok[c] = ci < chunks;
    xrow[c] = reinterpret_cast<const char*>(a.X) + (size_t)(f0 + (cok[c] ? ci : 0) * VEC) * E::kBytes;
  }

  // Starts a row: zero, or, on a graph with implicit self loops, the row's own input row (taken
  // by lane group 0 only, once: not in the accumulating launches of later source blocks).  It
  // is loaded here, ahead of the row's edges, like one more gathered row; added in the store
  // step instead, the load changed the instruction schedule of the whole summing loop (Reddit-
  // like F = 602 forward: 4.44 ms per launch against 4.0 ms, with the same instruction count).
  // The own row's factor: 1, or 1/(in-degree + 1) when the edges carry the mean's tabulated
  // factors (backward mean); the forward mean scales the whole row in the store step.
  // The next row's own row is asked into L2 one row ahead (1-2.5 % on the DRAM-bound workloads,
  // whose rows are short against a DRAM round trip).  Asking for all of a warp's own rows when
  // the warp starts made the same workloads slower (Products-like F = 602 41.4 -> 51.3 ms).
  auto start_row = [&](int64_t r, V (&acc)[CPL], bool more_rows) {
#pragma unroll
    for (int c = 0; c < CPL; ++c) zero(acc[c]);
    if constexpr (SELF) {
      if (grp == 0 && !(SEG && a.accumulate)) {
        using L = typename Pack<E, VEC>::Load;
        const float ss = (sa.self_mean && !a.mean_rows) ? self_factor(sa.self_ptr, r) : 1.0f;
        // the warp's next row will want its own row: ask it into L2 one row ahead
        if (more_rows) {
#pragma unroll
          for (int c = 0; c < CPL; ++c)
            if (cok[c])
              asm volatile("prefetch.global.L2 [%0];" ::"l"(xrow[c] + (size_t)(r + 1) * row_bytes));
        }
#pragma unroll
        for (int c = 0; c < CPL; ++c)
          if (cok[c]) fma(acc[c], ss, ldg_vec(xrow[c] + (size_t)r * row_bytes, L()));
      }
    }
  };

  // Writes one finished row: scales by 1/length for the mean (length + 1 with self loops: the
  // forward segment length is the in-degree) and, in a later source block, adds what the
  // earlier blocks left in Y.
  auto store_row = [&](int64_t r, int len, V (&acc)[CPL]) {
    if (lane < G) {
      const float rs = !a.mean_rows ? 1.0f
                       : SELF      ? 1.0f / (float)(len + 1)
                                   : (len > 0 ? 1.0f / (float)len : 1.0f);
      float* orow = a.Y + (size_t)r * (size_t)a.F + f0;
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        if (cok[c]) {
          float* dst = orow + (c0 + c * G) * VEC;
          if (a.mean_rows) scale(acc[c], rs);
          if (SEG && a.accumulate) add(acc[c], ld_vec(dst, V()));
          stcs_vec(dst, acc[c]);
        }
      }
    }
  };

  if (SEG && (int)blockIdx.x >= heavy_blocks) {
    // Source-blocked pass: row i of this warp contributes the positions [seg_lo, seg_hi) of its
    // segment.  The pieces are not adjacent in memory, so batches start at each piece; the
    // prefetch cursor (qi, qb) runs one batch ahead of the summing loop across rows.
    const int rpw = a.rows_per_warp;
    const int64_t rb = ((int64_t)(blockIdx.x - heavy_blocks) * kWarpsPerBlock + warp) * rpw;
    if (rb >= a.n) return;
    const int nrows = (int)min((int64_t)rpw, a.n - rb);
    int my_lo = 0, my_hi = 0, my_full = 0;
    if (lane < nrows) {
      my_lo = __ldg(a.seg_lo + rb + lane);
      my_hi = __ldg(a.seg_hi + rb + lane);
      my_full = (int)(__ldg(a.ptr + rb + lane + 1) - __ldg(a.ptr + rb + lane));
    }
    const unsigned heavy_mask = __ballot_sync(kFull, my_full > a.heavy_threshold);
    const unsigned work =
        __ballot_sync(kFull, lane < nrows && my_full <= a.heavy_threshold && my_hi > my_lo);
    int qi = work ? __ffs(work) - 1 : 32, qb = 0, qhi = 0;
    int32_t cur_u = 0, nxt_u = 0;
    float cur_s = 0.f, nxt_s = 0.f;
    auto step_q = [&]() {
      qb += 32;
      if (qb >= qhi) {
        const unsigned rest = qi >= 31 ? 0u : (work & ~((2u << qi) - 1u));
        qi = rest ? __ffs(rest) - 1 : 32;
        if (qi < 32) {
          qb = __shfl_sync(kFull, my_lo, qi);
          qhi = __shfl_sync(kFull, my_hi, qi);
        }
      }
    };
    if (qi < 32) {
      qb = __shfl_sync(kFull, my_lo, qi);
      qhi = __shfl_sync(kFull, my_hi, qi);
      load_batch<SCALED>(a, qb, qhi, lane, cur_u, cur_s);
      step_q();
      if (qi < 32) load_batch<SCALED>(a, qb, qhi, lane, nxt_u, nxt_s);
    }
    for (int i = 0; i < nrows; ++i) {
      if ((heavy_mask >> i) & 1u) continue;
      const int lo = __shfl_sync(kFull, my_lo, i);
      const int hi = __shfl_sync(kFull, my_hi, i);
      const int len = __shfl_sync(kFull, my_full, i);
      V acc[CPL];
      start_row(rb + i, acc, i + 1 < nrows);
      for (int b = lo; b < hi; b += 32) {
        add_edges<E, VEC, G, CPL, SCALED, SEG>(xrow, row_bytes, cur_u, cur_s, 0, min(hi - b, 32), grp, acc,
                                     stage);
        cur_u = nxt_u;
        cur_s = nxt_s;
        if (qi < 32) {
          step_q();
          if (qi < 32) load_batch<SCALED>(a, qb, qhi, lane, nxt_u, nxt_s);
        }
      }
      combine_groups<VEC, G, CPL>(acc);
      store_row(rb + i, len, acc);
    }
    return;
  }

  if ((int)blockIdx.x >= heavy_blocks) {
    const int rpw = a.rows_per_warp;
    const int64_t rb = ((int64_t)(blockIdx.x - heavy_blocks) * kWarpsPerBlock + warp) * rpw;
    if (rb >= a.n) return;
    const int nrows = (int)min((int64_t)rpw, a.n - rb);
    const int my_ptr = lane <= nrows ? (int)__ldg(a.ptr + rb + lane) : 0;
    const int stream_end = __shfl_sync(kFull, my_ptr, nrows);
    int b = __shfl_sync(kFull, my_ptr, 0);
    int32_t cur_u, nxt_u;
    float cur_s, nxt_s;
    load_batch<SCALED>(a, b, stream_end, lane, cur_u, cur_s);
    load_batch<SCALED>(a, (int64_t)b + 32, stream_end, lane, nxt_u, nxt_s);
    for (int i = 0; i < nrows; ++i) {
      const int lo = __shfl_sync(kFull, my_ptr, i);
      const int hi = __shfl_sync(kFull, my_ptr, i + 1);
      const int len = hi - lo;
      if (len > a.heavy_threshold) {  // a heavy block writes this row: skip its indices
        if (hi - b >= 32) {
          const int nb = b + ((hi - b) & ~31);
          if (nb == b + 32) { cur_u = nxt_u; cur_s = nxt_s; }
          else load_batch<SCALED>(a, nb, stream_end, lane, cur_u, cur_s);
          load_batch<SCALED>(a, (int64_t)nb + 32, stream_end, lane, nxt_u, nxt_s);
          b = nb;
        }
        continue;
      }
      V acc[CPL];
      start_row(rb + i, acc, i + 1 < nrows);
      int p = lo;
      while (p < hi) {
        if (p - b >= 32) {  // the stream is contiguous, so this is exactly one batch ahead
          b += 32;
          cur_u = nxt_u;
          cur_s = nxt_s;
          load_batch<SCALED>(a, (int64_t)b + 32, stream_end, lane, nxt_u, nxt_s);
        }
        const int e = min(hi - b, 32);
        add_edges<E, VEC, G, CPL, SCALED, SEG>(xrow, row_bytes, cur_u, cur_s, p - b, e, grp, acc, stage);
        p = b + e;
      }
      combine_groups<VEC, G, CPL>(acc);
      store_row(rb + i, len, acc);
    }
    return;
  }

  heavy_rows<E, VEC, G, CPL, SCALED, SEG, SELF, FOLD>(a, sa, heavy_blocks, part);
}

template <typename E, int VEC, int G, int CPL, bool SCALED, bool SEG, bool FOLD>
__global__ void __launch_bounds__(kBlock) ap_kernel(const ApArgs a, const int heavy_blocks) {
  __shared__ float part[kWarpsPerBlock][32 * CPL * VEC];
  ap_body<E, VEC, G, CPL, SCALED, SEG, false, FOLD>(a, SelfArgs{}, heavy_blocks, part);
}

// The same kernel compiled for six resident blocks per SM (at most 40 registers).  The scaled
// variants with up to 16 bytes per lane and step (and at least 16 lanes per edge) carry the
// edge factors on top of everything else and would take 60 registers; measured on B200 the
// higher occupancy wins for them (Reddit-like backward 22.0 ms uncapped, 19.2 ms at five
// blocks, 18.3 ms at six, 20.0 ms at seven or eight; Products-like backward 7.0 -> 5.9 ms),
// while a cap slows the unscaled variants down.
template <typename E, int VEC, int G, int CPL, bool SCALED, bool SEG, bool FOLD>
__global__ void __launch_bounds__(kBlock, 6) ap_kernel_r40(const ApArgs a, const int heavy_blocks) {
  __shared__ float part[kWarpsPerBlock][32 * CPL * VEC];
  ap_body<E, VEC, G, CPL, SCALED, SEG, false, FOLD>(a, SelfArgs{}, heavy_blocks, part);
}

// Both again for graphs with implicit self loops: every row also sums its own input row.
template <typename E, int VEC, int G, int CPL, bool SCALED, bool SEG, bool FOLD>
__global__ void __launch_bounds__(kBlock) ap_kernel_self(const ApArgs a, const int heavy_blocks,
                                                         const SelfArgs sa) {
  __shared__ float part[kWarpsPerBlock][32 * CPL * VEC];
  ap_body<E, VEC, G, CPL, SCALED, SEG, true, FOLD>(a, sa, heavy_blocks, part);
}

template <typename E, int VEC, int G, int CPL, bool SCALED, bool SEG, bool FOLD>
__global__ void __launch_bounds__(kBlock, 6) ap_kernel_self_r40(const ApArgs a, const int heavy_blocks,
                                                                const SelfArgs sa) {
  __shared__ float part[kWarpsPerBlock][32 * CPL * VEC];
  ap_body<E, VEC, G, CPL, SCALED, SEG, true, FOLD>(a, sa, heavy_blocks, part);
}

// Blocks that walk the heavy list: as many as the device keeps resident, so that the heavy
// segments (scheduled first, longest first) have the whole machine until the list runs out.
template <typename K>
int heavy_block_count(const Graph* g, K kernel, size_t smem) {
  int per_sm = (int)g->heavy_blocks_per_sm;
  if (per_sm <= 0) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kBlock, smem) != cudaSuccess)
      per_sm = 2;
  }
  return g->sm_count * (per_sm < 1 ? 1 : per_sm);
}

// FOLD: the graph may hold segments of kLongSegment entries or more in this direction.
template <typename E, int VEC, int G, int CPL, bool SCALED, bool SELF, bool FOLD>
dg_status_t launch_variant(const Graph* g, const ApArgs& a, const SelfArgs& sa, int slices,
                           cudaStream_t s) {
  // also the narrowest slices (at most 4 lanes per edge, i.e. up to 16 features per slice): their
  // 32- and 64-byte gathers wait on latency, and six blocks per SM hide more of it than five
  // (Proteins-like F = 8: 0.425 -> 0.384 ms, F = 16: 0.449 -> 0.429 ms)
  constexpr bool kCapped = (SCALED && VEC * CPL * E::kBytes <= 16 && G >= 16) || G <= 4;
  const int64_t rows_per_block = (int64_t)a.rows_per_warp * kWarpsPerBlock;
  const int64_t light_blocks = (a.n + rows_per_block - 1) / rows_per_block;
  // Where the cap pays depends on the graph as well: with rows sorted hub-first, or very short
  // rows whose gathers come from DRAM, the scaled kernels run faster at their natural 60 registers
  // (Products-like hub-first, mean backward: 6.02 -> 5.43 ms; Papers-like x0.1, mean backward:
  // 13.9 -> 12.3 ms), while the same graph as generated and the dense-ish ones lose 8-15 % without
  // it.  The handle says which (a.full_registers); the narrowest slices always keep the cap.
  const bool capped = kCapped && (G <= 4 || !a.full_registers);
  if constexpr (SELF) {
    void (*kernel)(const ApArgs, const int, const SelfArgs);
    if (capped) {
      kernel = a.seg_lo ? ap_kernel_self_r40<E, VEC, G, CPL, SCALED, true, FOLD>
                        : ap_kernel_self_r40<E, VEC, G, CPL, SCALED, false, FOLD>;
    } else {
      kernel = a.seg_lo ? ap_kernel_self<E, VEC, G, CPL, SCALED, true, FOLD>
                        : ap_kernel_self<E, VEC, G, CPL, SCALED, false, FOLD>;
    }
    const int heavy_blocks = heavy_block_count(g, kernel, 0);
    dim3 grid((unsigned)(heavy_blocks + light_blocks), (unsigned)slices);
    kernel<<<grid, kBlock, 0, s>>>(a, heavy_blocks, sa);
  } else {
    void (*kernel)(const ApArgs, const int);
    if (capped) {
      kernel = a.seg_lo ? ap_kernel_r40<E, VEC, G, CPL, SCALED, true, FOLD>
                        : ap_kernel_r40<E, VEC, G, CPL, SCALED, false, FOLD>;
    } else {
      kernel = a.seg_lo ? ap_kernel<E, VEC, G, CPL, SCALED, true, FOLD>
                        : ap_kernel<E, VEC, G, CPL, SCALED, false, FOLD>;
    }
    const int heavy_blocks = heavy_block_count(g, kernel, 0);
    dim3 grid((unsigned)(heavy_blocks + light_blocks), (unsigned)slices);
    kernel<<<grid, kBlock, 0, s>>>(a, heavy_blocks);
  }
  DG_CUDA(cudaGetLastError());
  count_launches(1);
  return DG_OK;
}

template <typename E, int VEC, bool SCALED, bool SELF, bool FOLD>
dg_status_t dispatch_shape(const Graph* g, const ApArgs& a, const SelfArgs& sa, int slices,
                           cudaStream_t s) {
  if (a.n == 0) return DG_OK;
  const int chunks = (a.slice_f < a.F ? a.slice_f : a.F) / VEC;  // vectors per row slice
  if (chunks <= 2) return launch_variant<E, VEC, 2, 1, SCALED, SELF, FOLD>(g, a, sa, slices, s);
  if (chunks <= 4) return launch_variant<E, VEC, 4, 1, SCALED, SELF, FOLD>(g, a, sa, slices, s);
  if (chunks <= 8) return launch_variant<E, VEC, 8, 1, SCALED, SELF, FOLD>(g, a, sa, slices, s);
  if (chunks <= 16) return launch_variant<E, VEC, 16, 1, SCALED, SELF, FOLD>(g, a, sa, slices, s);
  if (chunks <= 32) return launch_variant<E, VEC, 32, 1, SCALED, SELF, FOLD>(g, a, sa, slices, s);
  if (chunks <= 64) return launch_variant<E, VEC, 32, 2, SCALED, SELF, FOLD>(g, a, sa, slices, s);
  return launch_variant<E, VEC, 32, 4, SCALED, SELF, FOLD>(g, a, sa, slices, s);
}

template <typename E, int VEC, bool SELF, bool FOLD>
dg_status_t dispatch_scaled(const Graph* g, const ApArgs& a, const SelfArgs& sa, int slices,
                            cudaStream_t s) {
  return a.w ? dispatch_shape<E, VEC, true, SELF, FOLD>(g, a, sa, slices, s)
             : dispatch_shape<E, VEC, false, SELF, FOLD>(g, a, sa, slices, s);
}

// Storage type and vector width chosen by the caller; SELF = the graph has implicit self loops
// (sa.self_ptr is set); FOLD = the graph may hold segments of kLongSegment entries or more in this
// direction.  The four (SELF, FOLD) combinations are compiled in translation units of their own.
template <bool SELF, bool FOLD>
dg_status_t dispatch_type(const Graph* g, const ApArgs& a, const SelfArgs& sa, int vec, int slices,
                          cudaStream_t s) {
  if (a.x_bf16) {
    if (vec == 8) return dispatch_scaled<BF16, 8, SELF, FOLD>(g, a, sa, slices, s);
    if (vec == 4) return dispatch_scaled<BF16, 4, SELF, FOLD>(g, a, sa, slices, s);
    return dispatch_scaled<BF16, 2, SELF, FOLD>(g, a, sa, slices, s);
  }
  if (vec == 4) return dispatch_scaled<F32, 4, SELF, FOLD>(g, a, sa, slices, s);
  if (vec == 2) return dispatch_scaled<F32, 2, SELF, FOLD>(g, a, sa, slices, s);
  return dispatch_scaled<F32, 1, SELF, FOLD>(g, a, sa, slices, s);
}

}  // namespace
}  // namespace dg
#endif  // DG_AGGREGATE_KERNELS_CUH_
