// The general aggregation primitive: every operator pair of Table 1 of the paper,
//   f_O[v] = (+)_{edges e_uv into v} ( f_V[u] (x) f_E[e_uv] )          (Eq. 1, Eq. 2, Algorithm 1)
// with (x) in {copylhs, copyrhs, add, sub, mul, div}, (+) in {sum, max, min} and f_E a full
// |E| x F matrix (or |E| x 1, broadcast), its gradients with respect to f_V and f_E, and the
// gradient of the weighted sum / mean with respect to scalar edge weights (message passing onto
// edges, Section 2.2).
//
// These kernels are kept apart from the sum / mean kernels of dg_aggregate_kernels.cuh, which
// stay as they are: here a warp owns one row (one column in the pass over the CSC; the 8 warps of
// a block share a row of the handle's heavy list), its lanes are spread along the features in
// groups of G lanes, and the groups take different edges.  With
// a full edge-feature matrix the edge stream is as large as the gathered rows (nnz x F x 4
// bytes, read once, coalesced), so these passes are bound by HBM streaming rather than by the
// gather.
//
// Determinism: every output element is produced by one warp (one block) in a fixed order; the
// extremum of max / min is chosen on (message, edge position) pairs, equal messages going to the
// lowest position, so the order in which lane groups are combined does not matter.  No atomics.
#include "dg_internal.cuh"

namespace dg {
namespace {

constexpr int kGenBlock = 256;
constexpr int kGenWarps = kGenBlock / 32;
constexpr unsigned kAll = 0xffffffffu;
constexpr int kChain = 256;  // a register sum is moved to a second-level sum after this many terms

enum { kCopyLhs = DG_BIN_COPY_LHS, kCopyRhs = DG_BIN_COPY_RHS, kAdd = DG_BIN_ADD,
       kSub = DG_BIN_SUB, kMul = DG_BIN_MUL, kDiv = DG_BIN_DIV };
enum { kSum = DG_RED_SUM, kMax = DG_RED_MAX, kMin = DG_RED_MIN };

struct GenArgs {
  const int64_t* ptr;    // n+1 segment pointers: rowptr, or colptr in the pass over the CSC
  const int32_t* idx;    // colidx, or rowidx_T
  const int32_t* perm;   // CSC pass: CSR position of every CSC entry
  const int64_t* rowptr; // CSR row pointer (the divisor of the mean in the edge-weight gradient)
  const float* X;        // n x F vertex features (fV), or dO in the gradient passes
  const float* V;        // gradient passes: fV
  const float* Y;        // nnz x cols edge features in CSR position order
  const int32_t* arg;    // n x F edge positions of the extrema (max / min)
  float* out;            // n x F, or nnz x cols in the edge-gradient pass
  int32_t* arg_out;
  int64_t n;
  int32_t F, cols;
  int32_t log_g;         // lanes per edge = 1 << log_g
  int32_t row_scale;     // edge-weight gradient: 0 none, 1 = 1/deg(v), 2 = 1/(deg(v)+1)
  int32_t vec;           // floats per load, 4 or 2 when F and the operands' alignment allow
  // the handle's list of rows (columns, in the pass over the CSC) longer than heavy_threshold,
  // longest first; nullptr: every row is walked by one warp
  const int32_t* heavy_list;
  const int32_t* heavy_count;
  int32_t heavy_cap, heavy_threshold;
  int32_t heavy_blocks;  // leading blocks of the grid that walk the heavy list
  // one pass of a sliced / source-blocked call (forward and gradient with respect to fV):
  // features [f_lo, f_lo + f_cnt), the piece [seg_lo[v], seg_hi[v]) of every row (nullptr: whole
  // rows), and whether out (and arg_out) already hold the result of the earlier pieces
  int32_t f_lo, f_cnt;
  const int32_t* seg_lo;
  const int32_t* seg_hi;
  int32_t accumulate;
};

// one fp32 IEEE operation, never contracted into a neighbouring add
template <int BIN>
__device__ __forceinline__ float message(float x, float y) {
  if (BIN == kCopyLhs) return x;
  if (BIN == kCopyRhs) return y;
  if (BIN == kAdd) return __fadd_rn(x, y);
  if (BIN == kSub) return __fsub_rn(x, y);
  if (BIN == kMul) return __fmul_rn(x, y);
  return __fdiv_rn(x, y);
}
template <int BIN>
__device__ __forceinline__ float d_dx(float y) {
  if (BIN == kCopyRhs) return 0.f;
  if (BIN == kMul) return y;
  if (BIN == kDiv) return __fdiv_rn(1.f, y);
  return 1.f;
}
template <int BIN>
__device__ __forceinline__ float d_dy(float x, float y) {
  if (BIN == kCopyLhs) return 0.f;
  if (BIN == kSub) return -1.f;
  if (BIN == kMul) return x;
  if (BIN == kDiv) return -__fdiv_rn(x, __fmul_rn(y, y));
  return 1.f;
}

// (value, position) of the better of two candidates; position < 0 means "none"
template <int RED>
__device__ __forceinline__ void take_better(float& best, int32_t& best_k, float m, int32_t k) {
  if (k < 0) return;
  const bool better = RED == kMax ? m > best : m < best;
  if (best_k < 0 || better || (m == best && k < best_k)) {
    best = m;
    best_k = k;
  }
}

constexpr int kTiles = 4;  // feature tiles of G lanes a warp carries through one walk of a row
// edges in flight per lane group and step: four where only one operand is loaded per message
template <int BIN> struct EdgesInFlight {
  static constexpr int value = 4;
};

// ---- rows on the handle's heavy list: a block per row ----
//
// The first heavy_blocks blocks of a launch walk the list (longest first); they start before the
// blocks of the light rows, so a hub row runs beside the light ones instead of holding one warp
// long after the rest of the grid has drained.  The 8 warps of a block take interleaved 32-edge
// batches of one row, leave their partial results in shared memory, and warp 0 merges them in warp
// order (sums) or by (message, position) (max / min), so the result does not depend on timing.
// The walk below is the one of the light kernels with a batch stride; the light kernels keep it
// written out in their bodies, which compiles to faster code than the call (Products-like max:
// 13.0 against 21.0 ms).

// where a lane's four values per edge lie: kTiles / VEC vectors of VEC floats, G * VEC apart
template <int VEC>
struct LaneTiles {
  static constexpr int kT = kTiles / VEC;
  bool ok[kT], tile_on[kT];
  int base[kT];  // first feature of the lane's vector t (0 when it lies beyond F)
  __device__ __forceinline__ void place(int f0, int F, int G, int c) {
#pragma unroll
    for (int t = 0; t < kT; ++t) {
      tile_on[t] = f0 + t * G * VEC < F;  // the same for the whole warp
      ok[t] = f0 + (t * G + c) * VEC < F;
      base[t] = ok[t] ? f0 + (t * G + c) * VEC : 0;
    }
  }
};

// loads VEC consecutive floats (ints) into dst[0..VEC)
template <int VEC>
__device__ __forceinline__ void load_vec(float* dst, const float* src) {
  if (VEC == 4) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(src));
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  } else if (VEC == 2) {
    const float2 v = __ldg(reinterpret_cast<const float2*>(src));
    dst[0] = v.x; dst[1] = v.y;
  } else {
    dst[0] = __ldg(src);
  }
}
template <int VEC>
__device__ __forceinline__ void load_vec(int32_t* dst, const int32_t* src) {
  if (VEC == 4) {
    const int4 v = __ldg(reinterpret_cast<const int4*>(src));
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  } else if (VEC == 2) {
    const int2 v = __ldg(reinterpret_cast<const int2*>(src));
    dst[0] = v.x; dst[1] = v.y;
  } else {
    dst[0] = __ldg(src);
  }
}

// A warp's share of row [lo, hi): the 32-edge batches first_batch, first_batch + batch_stride, ...
// Leaves the per-lane sums (total) or extrema (best, best_k; best_k < 0: none), not yet combined
// across the lane groups.
template <int BIN, int RED, int VEC>
__device__ __forceinline__ void fwd_walk(const GenArgs& a, int64_t lo, int64_t hi, int first_batch,
                                         int batch_stride, const LaneTiles<VEC>& L, int grp, int NG,
                                         float (&total)[4], float (&best)[4], int32_t (&best_k)[4]) {
  constexpr int kT = kTiles / VEC;
  constexpr int kEdges = (VEC > 1 && EdgesInFlight<BIN>::value == 4) ? 4 : 2;
  const int lane = threadIdx.x & 31;
  const int F = a.F, cols = a.cols;
  const int64_t step = (int64_t)batch_stride * 32;
  float acc[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc[q] = total[q] = best[q] = 0.f;
    best_k[q] = -1;
  }
  int chain = 0;
  for (int64_t b = lo + (int64_t)first_batch * 32; b < hi; b += step) {
    const int32_t my_u = (BIN != kCopyRhs && b + lane < hi) ? __ldcs(a.idx + b + lane) : 0;
    const int cnt = (int)(hi - b < 32 ? hi - b : 32);
    for (int e0 = 0; e0 < cnt; e0 += NG * kEdges) {
      float x[kEdges][4], y[kEdges][4];
#pragma unroll
      for (int i = 0; i < kEdges; ++i) {
        const int e = e0 + i * NG + grp;
        const int32_t u = __shfl_sync(kAll, my_u, e & 31);
        const float* xrow = BIN != kCopyRhs ? a.X + (size_t)u * F : nullptr;
        const float* yrow = BIN != kCopyLhs ? a.Y + (size_t)(e < cnt ? b + e : b) * cols : nullptr;
        float y1 = 1.f;
        if (BIN != kCopyLhs && cols == 1) y1 = __ldg(yrow);
#pragma unroll
        for (int q = 0; q < 4; ++q) { x[i][q] = 0.f; y[i][q] = y1; }
#pragma unroll
        for (int t = 0; t < kT; ++t) {
          if (!L.tile_on[t]) continue;
          if (BIN != kCopyRhs) load_vec<VEC>(&x[i][t * VEC], xrow + L.base[t]);
          if (BIN != kCopyLhs && cols != 1) load_vec<VEC>(&y[i][t * VEC], yrow + L.base[t]);
        }
      }
#pragma unroll
      for (int i = 0; i < kEdges; ++i) {
        const int e = e0 + i * NG + grp;
        const bool valid = e < cnt;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (!L.tile_on[q / VEC]) continue;
          const float m = message<BIN>(x[i][q], y[i][q]);
          if (RED == kSum) {
            acc[q] += valid ? m : 0.f;
          } else {
            // ascending positions within a lane: "strictly better" keeps the lowest among equals
            const bool take =
                valid && (best_k[q] < 0 || (RED == kMax ? m > best[q] : m < best[q]));
            best[q] = take ? m : best[q];
            best_k[q] = take ? (int32_t)(b + e) : best_k[q];
          }
        }
      }
      chain += kEdges;
      if (RED == kSum && chain >= kChain) {
        chain = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) { total[q] += acc[q]; acc[q] = 0.f; }
      }
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) total[q] += acc[q];
}

template <int BIN, int RED, int VEC>
__device__ __forceinline__ void fwd_heavy_rows(const GenArgs& a, int first, int stride) {
  __shared__ float part_v[kGenWarps][4][32];
  __shared__ int32_t part_k[kGenWarps][4][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int count = min(*a.heavy_count, a.heavy_cap);
  for (int i = first; i < count; i += stride) {
    const int64_t row = a.heavy_list[i];
    const int64_t lo = a.seg_lo ? __ldg(a.seg_lo + row) : __ldg(a.ptr + row);
    const int64_t hi = a.seg_hi ? __ldg(a.seg_hi + row) : __ldg(a.ptr + row + 1);
    const int f_end = a.f_lo + a.f_cnt;
    for (int f0 = a.f_lo; f0 < f_end; f0 += kTiles * G) {
      LaneTiles<VEC> L;
      L.place(f0, f_end, G, c);
      float total[4], best[4];
      int32_t best_k[4];
      fwd_walk<BIN, RED, VEC>(a, lo, hi, warp, kGenWarps, L, grp, NG, total, best, best_k);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        part_v[warp][q][lane] = RED == kSum ? total[q] : best[q];
        part_k[warp][q][lane] = best_k[q];
      }
      __syncthreads();
      if (warp == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (!L.tile_on[q / VEC]) continue;
          for (int w = 1; w < kGenWarps; ++w) {
            if (RED == kSum) total[q] += part_v[w][q][lane];
            else take_better<RED>(best[q], best_k[q], part_v[w][q][lane], part_k[w][q][lane]);
          }
          for (int off = G; off < 32; off <<= 1) {
            if (RED == kSum) {
              total[q] += __shfl_xor_sync(kAll, total[q], off);
            } else {
              const float ob = __shfl_xor_sync(kAll, best[q], off);
              const int32_t ok2 = __shfl_xor_sync(kAll, best_k[q], off);
              take_better<RED>(best[q], best_k[q], ob, ok2);
            }
          }
          if (grp == 0 && L.ok[q / VEC]) {
            const size_t o = (size_t)row * a.F + L.base[q / VEC] + q % VEC;
            if (RED == kSum) {
              a.out[o] = a.accumulate ? a.out[o] + total[q] : total[q];
            } else {
              if (a.accumulate) take_better<RED>(best[q], best_k[q], a.out[o], a.arg_out[o]);
              a.out[o] = best_k[q] >= 0 ? best[q] : 0.f;
              if (a.arg_out) a.arg_out[o] = best_k[q];
            }
          }
        }
      }
      __syncthreads();
    }
  }
}

// the same for a column of the CSC in the gradient with respect to fV
template <int BIN, int RED, int VEC>
__device__ __forceinline__ void bwd_walk(const GenArgs& a, int64_t lo, int64_t hi, int first_batch,
                                         int batch_stride, const LaneTiles<VEC>& L, int grp, int NG,
                                         float (&total)[4]) {
  constexpr int kT = kTiles / VEC;
  constexpr int kEdges = 2;
  constexpr bool kNeedsY = BIN == kMul || BIN == kDiv;
  constexpr bool kNeedsK = kNeedsY || RED != kSum;
  const int lane = threadIdx.x & 31;
  const int F = a.F, cols = a.cols;
  const int64_t step = (int64_t)batch_stride * 32;
  float acc[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) acc[q] = total[q] = 0.f;
  int chain = 0;
  for (int64_t b = lo + (int64_t)first_batch * 32; b < hi; b += step) {
    const bool mine = b + lane < hi;
    const int32_t my_v = mine ? __ldcs(a.idx + b + lane) : 0;
    const int32_t my_k = (kNeedsK && mine) ? __ldcs(a.perm + b + lane) : 0;
    const int cnt = (int)(hi - b < 32 ? hi - b : 32);
    for (int e0 = 0; e0 < cnt; e0 += NG * kEdges) {
      float g[kEdges][4], y[kEdges][4];
      int32_t sel[kEdges][4], k[kEdges];
#pragma unroll
      for (int i = 0; i < kEdges; ++i) {
        const int e = e0 + i * NG + grp;
        const size_t vrow = (size_t)__shfl_sync(kAll, my_v, e & 31) * F;
        k[i] = __shfl_sync(kAll, my_k, e & 31);
        const float* yrow = kNeedsY ? a.Y + (size_t)k[i] * cols : nullptr;
        float y1 = 1.f;
        if (kNeedsY && cols == 1) y1 = __ldg(yrow);
#pragma unroll
        for (int q = 0; q < 4; ++q) { g[i][q] = 0.f; y[i][q] = y1; sel[i][q] = 0; }
#pragma unroll
        for (int t = 0; t < kT; ++t) {
          if (!L.tile_on[t]) continue;
          load_vec<VEC>(&g[i][t * VEC], a.X + vrow + L.base[t]);
          if (kNeedsY && cols != 1) load_vec<VEC>(&y[i][t * VEC], yrow + L.base[t]);
          if (RED != kSum) load_vec<VEC>(&sel[i][t * VEC], a.arg + vrow + L.base[t]);
        }
      }
#pragma unroll
      for (int i = 0; i < kEdges; ++i) {
        const bool valid = e0 + i * NG + grp < cnt;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (!L.tile_on[q / VEC]) continue;
          float v = g[i][q];
          if (kNeedsY) v *= d_dx<BIN>(y[i][q]);
          if (!valid || (RED != kSum && sel[i][q] != k[i])) v = 0.f;
          acc[q] += v;
        }
      }
      chain += kEdges;
      if (chain >= kChain) {
        chain = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) { total[q] += acc[q]; acc[q] = 0.f; }
      }
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) total[q] += acc[q];
}

template <int BIN, int RED, int VEC>
__device__ __forceinline__ void bwd_heavy_cols(const GenArgs& a, int first, int stride) {
  __shared__ float part_v[kGenWarps][4][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int count = min(*a.heavy_count, a.heavy_cap);
  for (int i = first; i < count; i += stride) {
    const int64_t u = a.heavy_list[i];
    const int64_t lo = a.seg_lo ? __ldg(a.seg_lo + u) : __ldg(a.ptr + u);
    const int64_t hi = a.seg_hi ? __ldg(a.seg_hi + u) : __ldg(a.ptr + u + 1);
    const int f_end = a.f_lo + a.f_cnt;
    for (int f0 = a.f_lo; f0 < f_end; f0 += kTiles * G) {
      LaneTiles<VEC> L;
      L.place(f0, f_end, G, c);
      float total[4];
      bwd_walk<BIN, RED, VEC>(a, lo, hi, warp, kGenWarps, L, grp, NG, total);
#pragma unroll
      for (int q = 0; q < 4; ++q) part_v[warp][q][lane] = total[q];
      __syncthreads();
      if (warp == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (!L.tile_on[q / VEC]) continue;
          for (int w = 1; w < kGenWarps; ++w) total[q] += part_v[w][q][lane];
          for (int off = G; off < 32; off <<= 1) total[q] += __shfl_xor_sync(kAll, total[q], off);
          if (grp == 0 && L.ok[q / VEC]) {
            float* o = a.out + (size_t)u * a.F + L.base[q / VEC] + q % VEC;
            *o = a.accumulate ? *o + total[q] : total[q];
          }
        }
      }
      __syncthreads();
    }
  }
}

// Forward: warp per destination row.  The indices of a row are read as coalesced batches of 32
// (one per lane, the next batch in flight while the current one is used) and broadcast by
// shuffles.  A lane holds four values of a message per edge: with VEC = 4 one 16-byte vector of
// consecutive features (F a multiple of 4, 16-byte aligned matrices), with VEC = 2 two 8-byte
// vectors G apart, with VEC = 1 four features G apart; G lanes cover 4 G features per pass, and
// vectors that lie beyond F are skipped for the whole warp.  Two or four edges per lane group are
// in flight per step.  No load is predicated per lane: lanes without an edge or a feature read a
// valid address and their values are dropped.  Rows longer than heavy_threshold are left to the
// leading blocks of the launch (see fwd_heavy_rows) when a.heavy_list is set.
template <int BIN, int RED, int VEC>
__global__ void __launch_bounds__(kGenBlock) general_fwd_kernel(const GenArgs a) {
  constexpr int kT = kTiles / VEC;  // vectors per lane and edge (4, 2 or 1)
  constexpr int NV = kT * VEC;      // values per lane and edge: always 4
  // edges in flight per lane group and step: four where a message needs one vector load only
  constexpr int kEdges = (VEC > 1 && EdgesInFlight<BIN>::value == 4) ? 4 : 2;
  const int lane = threadIdx.x & 31;
  const int hb = a.heavy_list ? a.heavy_blocks : 0;
  if ((int)blockIdx.x < hb) {
    fwd_heavy_rows<BIN, RED, VEC>(a, blockIdx.x, hb);
    return;
  }
  const int64_t row = (int64_t)(blockIdx.x - hb) * kGenWarps + (threadIdx.x >> 5);
  if (row >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  int64_t lo = __ldg(a.ptr + row), hi = __ldg(a.ptr + row + 1);
  if (a.heavy_list && hi - lo > a.heavy_threshold) return;  // a block of the list walk has it
  if (a.seg_lo) {  // this launch's piece of the row (one range of source ids)
    lo = __ldg(a.seg_lo + row);
    hi = __ldg(a.seg_hi + row);
  }
  const int F = a.F, cols = a.cols;
  const int f_end = a.f_lo + a.f_cnt;
  for (int f0 = a.f_lo; f0 < f_end; f0 += kT * G * VEC) {
    bool ok[kT], tile_on[kT];
    int base[kT];  // first feature of the lane's vector t (0 when it lies beyond F)
    float acc[NV], total[NV], best[NV];
    int32_t best_k[NV];
#pragma unroll
    for (int t = 0; t < kT; ++t) {
      tile_on[t] = f0 + t * G * VEC < f_end;         // the same for the whole warp
      ok[t] = f0 + (t * G + c) * VEC < f_end;
      base[t] = ok[t] ? f0 + (t * G + c) * VEC : 0;
    }
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      acc[q] = total[q] = best[q] = 0.f;
      best_k[q] = -1;
    }
    int chain = 0;
    int32_t next_u = (BIN != kCopyRhs && lo + lane < hi) ? __ldcs(a.idx + lo + lane) : 0;
    for (int64_t b = lo; b < hi; b += 32) {
      const int32_t my_u = next_u;
      next_u = (BIN != kCopyRhs && b + 32 + lane < hi) ? __ldcs(a.idx + b + 32 + lane) : 0;
      const int cnt = (int)(hi - b < 32 ? hi - b : 32);
      for (int e0 = 0; e0 < cnt; e0 += NG * kEdges) {
        float x[kEdges][NV], y[kEdges][NV];
#pragma unroll
        for (int i = 0; i < kEdges; ++i) {
          const int e = e0 + i * NG + grp;
          const int32_t u = __shfl_sync(kAll, my_u, e & 31);
          const float* xrow = BIN != kCopyRhs ? a.X + (size_t)u * F : nullptr;
          const float* yrow = BIN != kCopyLhs ? a.Y + (size_t)(e < cnt ? b + e : b) * cols : nullptr;
          float y1 = 1.f;
          if (BIN != kCopyLhs && cols == 1) y1 = __ldg(yrow);
#pragma unroll
          for (int t = 0; t < kT; ++t) {
            if (!tile_on[t]) continue;
            if (VEC == 2) {
              float2 xv = make_float2(0.f, 0.f), yv = make_float2(y1, y1);
              if (BIN != kCopyRhs) xv = __ldg(reinterpret_cast<const float2*>(xrow + base[t]));
              if (BIN != kCopyLhs && cols != 1)
                yv = __ldcs(reinterpret_cast<const float2*>(yrow + base[t]));
              x[i][t * 2 + 0] = xv.x; x[i][t * 2 + 1] = xv.y;
              y[i][t * 2 + 0] = yv.x; y[i][t * 2 + 1] = yv.y;
            } else if (VEC == 4) {
              float4 xv = make_float4(0.f, 0.f, 0.f, 0.f), yv = make_float4(y1, y1, y1, y1);
              if (BIN != kCopyRhs) xv = __ldg(reinterpret_cast<const float4*>(xrow + base[t]));
              if (BIN != kCopyLhs && cols != 1)
                yv = __ldcs(reinterpret_cast<const float4*>(yrow + base[t]));
              x[i][t * 4 + 0] = xv.x; x[i][t * 4 + 1] = xv.y;
              x[i][t * 4 + 2] = xv.z; x[i][t * 4 + 3] = xv.w;
              y[i][t * 4 + 0] = yv.x; y[i][t * 4 + 1] = yv.y;
              y[i][t * 4 + 2] = yv.z; y[i][t * 4 + 3] = yv.w;
            } else {
              x[i][t] = BIN != kCopyRhs ? __ldg(xrow + base[t]) : 0.f;
              y[i][t] = (BIN != kCopyLhs && cols != 1) ? __ldcs(yrow + base[t]) : y1;
            }
          }
        }
#pragma unroll
        for (int i = 0; i < kEdges; ++i) {
          const int e = e0 + i * NG + grp;
          const bool valid = e < cnt;
#pragma unroll
          for (int q = 0; q < NV; ++q) {
            if (!tile_on[q / VEC]) continue;
            const float m = message<BIN>(x[i][q], y[i][q]);
            if (RED == kSum) {
              acc[q] += valid ? m : 0.f;
            } else {
              // a lane meets its edges in ascending position, so "strictly better" keeps the
              // lowest position among equal messages; lane groups are merged by take_better
              const bool take =
                  valid && (best_k[q] < 0 || (RED == kMax ? m > best[q] : m < best[q]));
              best[q] = take ? m : best[q];
              best_k[q] = take ? (int32_t)(b + e) : best_k[q];
            }
          }
        }
        chain += kEdges;
        if (RED == kSum && chain >= kChain) {
          chain = 0;
#pragma unroll
          for (int q = 0; q < NV; ++q) { total[q] += acc[q]; acc[q] = 0.f; }
        }
      }
    }
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      if (!tile_on[q / VEC]) continue;
      total[q] += acc[q];
      for (int off = G; off < 32; off <<= 1) {
        if (RED == kSum) {
          total[q] += __shfl_xor_sync(kAll, total[q], off);
        } else {
          const float ob = __shfl_xor_sync(kAll, best[q], off);
          const int32_t ok2 = __shfl_xor_sync(kAll, best_k[q], off);
          take_better<RED>(best[q], best_k[q], ob, ok2);
        }
      }
      if (grp == 0 && ok[q / VEC]) {
        const size_t o = (size_t)row * F + base[q / VEC] + q % VEC;
        if (RED == kSum) {
          a.out[o] = a.accumulate ? a.out[o] + total[q] : total[q];
        } else {
          if (a.accumulate) take_better<RED>(best[q], best_k[q], a.out[o], a.arg_out[o]);
          a.out[o] = best_k[q] >= 0 ? best[q] : 0.f;
          if (a.arg_out) a.arg_out[o] = best_k[q];
        }
      }
    }
  }
}

// Gradient with respect to fV: warp per source vertex u over its CSC segment,
//   dV[u][j] = sum_q sel * dO[v_q][j] * d(x (x) y)/dx,   sel = [arg[v_q][j] == perm[q]] (max/min)
// The derivative depends on y only (and not at all for copylhs / add / sub).  Same walk as the
// forward kernel: batched indices (destination and CSR position), four values per lane and edge
// in vectors of VEC floats, unpredicated loads; the handle's heavy columns go to the leading blocks
// (bwd_heavy_cols).
template <int BIN, int RED, int VEC>
__global__ void __launch_bounds__(kGenBlock) general_bwd_vertex_kernel(const GenArgs a) {
  constexpr int kT = kTiles / VEC;
  constexpr int NV = kT * VEC;
  constexpr int kEdges = 2;
  const int lane = threadIdx.x & 31;
  const int hb = a.heavy_list ? a.heavy_blocks : 0;
  if ((int)blockIdx.x < hb) {
    bwd_heavy_cols<BIN, RED, VEC>(a, blockIdx.x, hb);
    return;
  }
  const int64_t u = (int64_t)(blockIdx.x - hb) * kGenWarps + (threadIdx.x >> 5);
  if (u >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  int64_t lo = __ldg(a.ptr + u), hi = __ldg(a.ptr + u + 1);
  if (a.heavy_list && hi - lo > a.heavy_threshold) return;  // a block of the list walk has it
  if (a.seg_lo) {  // this launch's piece of the column (one range of destination ids)
    lo = __ldg(a.seg_lo + u);
    hi = __ldg(a.seg_hi + u);
  }
  const int F = a.F, cols = a.cols;
  const int f_end = a.f_lo + a.f_cnt;
  constexpr bool kNeedsY = BIN == kMul || BIN == kDiv;
  constexpr bool kNeedsK = kNeedsY || RED != kSum;
  for (int f0 = a.f_lo; f0 < f_end; f0 += kT * G * VEC) {
    bool ok[kT], tile_on[kT];
    int base[kT];
    float acc[NV], total[NV];
#pragma unroll
    for (int t = 0; t < kT; ++t) {
      tile_on[t] = f0 + t * G * VEC < f_end;
      ok[t] = f0 + (t * G + c) * VEC < f_end;
      base[t] = ok[t] ? f0 + (t * G + c) * VEC : 0;
    }
#pragma unroll
    for (int q = 0; q < NV; ++q) acc[q] = total[q] = 0.f;
    int chain = 0;
    for (int64_t b = lo; b < hi; b += 32) {
      const bool mine = b + lane < hi;
      const int32_t my_v = mine ? __ldcs(a.idx + b + lane) : 0;
      const int32_t my_k = (kNeedsK && mine) ? __ldcs(a.perm + b + lane) : 0;
      const int cnt = (int)(hi - b < 32 ? hi - b : 32);
      for (int e0 = 0; e0 < cnt; e0 += NG * kEdges) {
        float g[kEdges][NV], y[kEdges][NV];
        int32_t sel[kEdges][NV], k[kEdges];
#pragma unroll
        for (int i = 0; i < kEdges; ++i) {
          const int e = e0 + i * NG + grp;
          const size_t vrow = (size_t)__shfl_sync(kAll, my_v, e & 31) * F;
          k[i] = __shfl_sync(kAll, my_k, e & 31);
          const float* yrow = kNeedsY ? a.Y + (size_t)k[i] * cols : nullptr;
          float y1 = 1.f;
          if (kNeedsY && cols == 1) y1 = __ldg(yrow);
#pragma unroll
          for (int t = 0; t < kT; ++t) {
            if (!tile_on[t]) continue;
            if (VEC == 4) {
              const float4 gv = __ldg(reinterpret_cast<const float4*>(a.X + vrow + base[t]));
              float4 yv = make_float4(y1, y1, y1, y1);
              int4 sv = make_int4(0, 0, 0, 0);
              if (kNeedsY && cols != 1) yv = __ldg(reinterpret_cast<const float4*>(yrow + base[t]));
              if (RED != kSum) sv = __ldg(reinterpret_cast<const int4*>(a.arg + vrow + base[t]));
              g[i][t * 4 + 0] = gv.x; g[i][t * 4 + 1] = gv.y; g[i][t * 4 + 2] = gv.z; g[i][t * 4 + 3] = gv.w;
              y[i][t * 4 + 0] = yv.x; y[i][t * 4 + 1] = yv.y; y[i][t * 4 + 2] = yv.z; y[i][t * 4 + 3] = yv.w;
              sel[i][t * 4 + 0] = sv.x; sel[i][t * 4 + 1] = sv.y; sel[i][t * 4 + 2] = sv.z; sel[i][t * 4 + 3] = sv.w;
            } else if (VEC == 2) {
              const float2 gv = __ldg(reinterpret_cast<const float2*>(a.X + vrow + base[t]));
              float2 yv = make_float2(y1, y1);
              int2 sv = make_int2(0, 0);
              if (kNeedsY && cols != 1) yv = __ldg(reinterpret_cast<const float2*>(yrow + base[t]));
              if (RED != kSum) sv = __ldg(reinterpret_cast<const int2*>(a.arg + vrow + base[t]));
              g[i][t * 2 + 0] = gv.x; g[i][t * 2 + 1] = gv.y;
              y[i][t * 2 + 0] = yv.x; y[i][t * 2 + 1] = yv.y;
              sel[i][t * 2 + 0] = sv.x; sel[i][t * 2 + 1] = sv.y;
            } else {
              g[i][t] = __ldg(a.X + vrow + base[t]);
              y[i][t] = (kNeedsY && cols != 1) ? __ldg(yrow + base[t]) : y1;
              sel[i][t] = RED != kSum ? __ldg(a.arg + vrow + base[t]) : 0;
            }
          }
        }
#pragma unroll
        for (int i = 0; i < kEdges; ++i) {
          const bool valid = e0 + i * NG + grp < cnt;
#pragma unroll
          for (int q = 0; q < NV; ++q) {
            if (!tile_on[q / VEC]) continue;
            float v = g[i][q];
            if (kNeedsY) v *= d_dx<BIN>(y[i][q]);
            if (!valid || (RED != kSum && sel[i][q] != k[i])) v = 0.f;
            acc[q] += v;
          }
        }
        chain += kEdges;
        if (chain >= kChain) {
          chain = 0;
#pragma unroll
          for (int q = 0; q < NV; ++q) { total[q] += acc[q]; acc[q] = 0.f; }
        }
      }
    }
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      if (!tile_on[q / VEC]) continue;
      total[q] += acc[q];
      for (int off = G; off < 32; off <<= 1) total[q] += __shfl_xor_sync(kAll, total[q], off);
      if (grp == 0 && ok[q / VEC]) {
        float* o = a.out + (size_t)u * F + base[q / VEC] + q % VEC;
        *o = a.accumulate ? *o + total[q] : total[q];
      }
    }
  }
}

// Gradient with respect to fE: the output is per edge, so a row splits freely.  As in the
// edge-weight gradient below, the first heavy_blocks blocks of a launch walk the handle's heavy
// rows, the 8 warps of a block taking interleaved steps of one row (first = warp, stride = 8); in
// the other blocks a warp owns one light row (first = 0, stride = 1).
template <class Row>
__device__ __forceinline__ void edge_rows(const GenArgs& a, Row row) {
  const int warp = threadIdx.x >> 5;
  const int hb = a.heavy_list ? a.heavy_blocks : 0;
  if ((int)blockIdx.x < hb) {
    const int count = min(*a.heavy_count, a.heavy_cap);
    for (int i = blockIdx.x; i < count; i += hb) row(a.heavy_list[i], warp, kGenWarps);
    return;
  }
  const int64_t v = (int64_t)(blockIdx.x - hb) * kGenWarps + warp;
  if (v >= a.n) return;
  if (a.heavy_list && __ldg(a.ptr + v + 1) - __ldg(a.ptr + v) > a.heavy_threshold) return;
  row(v, 0, 1);
}

// Full edge features (cols == F): one value per (edge, feature),
//   dE[k][j] = sel * dO[v][j] * d(x (x) y)/dy
// G lanes per edge, VEC consecutive features per lane (16-byte loads and stores when F is a
// multiple of 4 and the matrices are 16-byte aligned): the written rows are the traffic.
template <int BIN, int RED, int VEC>
__global__ void __launch_bounds__(kGenBlock) general_bwd_edge_full_kernel(const GenArgs a) {
  edge_rows(a, [&](int64_t v, int first, int stride) {
    const int lane = threadIdx.x & 31;
    const int G = 1 << a.log_g, NG = 32 >> a.log_g;
    const int grp = lane >> a.log_g, c = lane & (G - 1);
    const int64_t lo = __ldg(a.ptr + v), hi = __ldg(a.ptr + v + 1);
    const int F = a.F;
    constexpr bool kNeedsX = BIN == kMul || BIN == kDiv;
    for (int f0 = 0; f0 < F; f0 += G * VEC) {
      const int j = f0 + c * VEC;
      if (j >= F) continue;
      float g[VEC], x[VEC], y[VEC], t[VEC];
      int32_t sel[VEC];
      load_vec<VEC>(g, a.X + (size_t)v * F + j);
#pragma unroll
      for (int q = 0; q < VEC; ++q) { sel[q] = 0; x[q] = y[q] = 0.f; }
      if (RED != kSum) load_vec<VEC>(sel, a.arg + (size_t)v * F + j);
      for (int64_t e = lo + (int64_t)first * NG + grp; e < hi; e += (int64_t)stride * NG) {
        if (kNeedsX) load_vec<VEC>(x, a.V + (size_t)__ldg(a.idx + e) * F + j);
        if (BIN == kDiv) load_vec<VEC>(y, a.Y + (size_t)e * F + j);
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
          t[q] = g[q] * d_dy<BIN>(x[q], y[q]);
          if (RED != kSum && sel[q] != (int32_t)e) t[q] = 0.f;
        }
        float* o = a.out + (size_t)e * F + j;
        // written once, never read here: streaming stores leave L2 to the gathered rows
        if (VEC == 4) __stcs(reinterpret_cast<float4*>(o), make_float4(t[0], t[1], t[2], t[3]));
        else __stcs(o, t[0]);
      }
    }
  });
}

// Gradient with respect to fE with one column (the broadcast scalar): the feature sum of the
// above, one dot product per edge reduced inside the lane group:
//   dE[k] = s_v * sum_j sel * dO[v][j] * d(x (x) y)/dy
// With (x) = mul and (+) = sum this is the sampled dense-dense product <fV[u_k], dO[v_k]>, the
// gradient with respect to a scalar edge weight; row_scale gives the mean's s_v.
template <int BIN, int RED>
__global__ void __launch_bounds__(kGenBlock) general_bwd_edge_scalar_kernel(const GenArgs a) {
  edge_rows(a, [&](int64_t v, int first, int stride) {
    const int lane = threadIdx.x & 31;
    const int G = 1 << a.log_g, NG = 32 >> a.log_g;
    const int grp = lane >> a.log_g, c = lane & (G - 1);
    const int64_t lo = __ldg(a.ptr + v), hi = __ldg(a.ptr + v + 1);
    const int F = a.F;
    constexpr bool kNeedsX = BIN == kMul || BIN == kDiv;
    float s = 1.f;
    if (a.row_scale) s = 1.0f / (float)(hi - lo + (a.row_scale == 2 ? 1 : 0));
    // uniform trip count per warp: the shuffles need all lanes
    for (int64_t e0 = lo + (int64_t)first * NG; e0 < hi; e0 += (int64_t)stride * NG) {
      const int64_t e = e0 + grp;
      const bool eok = e < hi;
      float dot = 0.f;
      if (eok) {
        const float* xrow = kNeedsX ? a.V + (size_t)__ldg(a.idx + e) * F : nullptr;
        const float y = BIN == kDiv ? __ldg(a.Y + e) : 0.f;
        for (int j = c; j < F; j += G) {
          float t = __ldg(a.X + (size_t)v * F + j) * d_dy<BIN>(kNeedsX ? __ldg(xrow + j) : 0.f, y);
          if (RED != kSum && __ldg(a.arg + (size_t)v * F + j) != (int32_t)e) t = 0.f;
          dot += t;
        }
      }
      for (int off = 1; off < G; off <<= 1) dot += __shfl_xor_sync(kAll, dot, off);
      if (eok && c == 0) a.out[e] = dot * s;
    }
  });
}

// ---- dg_aggregate_edge_grad: dW[k] = s_v * <H[u_k], dOut[v_k]>, one dot product per edge ----
//
// The output is one value per edge, so a row of any length splits freely: the first blocks of the
// launch walk the handle's list of heavy rows (longest first), the 8 warps of a block taking
// interleaved 32-edge batches of one row; in the other blocks a warp owns one light row.  Lanes
// are spread along the features (G lanes per edge, VEC floats per load), U edges are in flight
// per lane group before the first multiply, and with G = 32 the eight partial dot products of a
// step are reduced together by a transposing butterfly (9 shuffles for 8 edges instead of 40).
// dOut[v] is the same row for every edge of v: a slab of it is read (from L1) once per U edges.
struct EdgeGradArgs {
  const int64_t* rowptr;
  const int32_t* colidx;
  const float* H;
  const float* dOut;
  float* dW;
  const int32_t* heavy_list;
  const int32_t* heavy_count;
  int32_t heavy_cap;
  int32_t heavy_threshold;
  int64_t n;
  int32_t F;
  int32_t row_scale;  // 0 none, 1 = 1/deg(v), 2 = 1/(deg(v)+1)
  // one pass of a sliced / source-blocked call: features [f_lo, f_lo + f_cnt), the piece
  // [seg_lo[v], seg_hi[v]) of every row (nullptr: whole rows), and whether dW already holds the
  // dot products of the earlier feature slices
  int32_t f_lo, f_cnt;
  const int32_t* seg_lo;
  const int32_t* seg_hi;
  int32_t accumulate;
};

template <int VEC> struct LoadVec;
template <> struct LoadVec<1> { using T = float; };
template <> struct LoadVec<2> { using T = float2; };
template <> struct LoadVec<4> { using T = float4; };
__device__ __forceinline__ float dotv(float x, float g) { return x * g; }
__device__ __forceinline__ float dotv(float2 x, float2 g) { return x.x * g.x + x.y * g.y; }
__device__ __forceinline__ float dotv(float4 x, float4 g) {
  return x.x * g.x + x.y * g.y + x.z * g.z + x.w * g.w;
}

template <int VEC, int G>
__device__ __forceinline__ void edge_grad_row(const EdgeGradArgs& a, int64_t v, int64_t lo,
                                              int64_t hi, int64_t degree, int first_batch,
                                              int batch_stride) {
  using V = typename LoadVec<VEC>::T;
  constexpr int NG = 32 / G;
  constexpr int U = G == 32 ? 8 : 4;  // edges in flight per lane group
  const int lane = threadIdx.x & 31;
  const int grp = lane / G, c = lane % G;
  const int nvec = a.f_cnt / VEC;
  float s = 1.f;
  if (a.row_scale) s = 1.0f / (float)(degree + (a.row_scale == 2 ? 1 : 0));
  const V* grow = reinterpret_cast<const V*>(a.dOut + (size_t)v * a.F + a.f_lo);
  for (int64_t b = lo + (int64_t)first_batch * 32; b < hi; b += (int64_t)batch_stride * 32) {
    // lanes past the end of the row name vertex 0: their loads are harmless and never written
    const int32_t my_u = b + lane < hi ? __ldcs(a.colidx + b + lane) : 0;
    const int cnt = (int)(hi - b < 32 ? hi - b : 32);
    for (int e0 = 0; e0 < cnt; e0 += NG * U) {
      // No predicate on the loads: a slab of dOut[v] (one vector per lane) is read once and
      // multiplied with the matching slab of the U gathered rows, U independent loads in flight.
      const V* xrow[U];
      float p[U];
#pragma unroll
      for (int j = 0; j < U; ++j) {
        const int32_t u = __shfl_sync(kAll, my_u, (e0 + j * NG + grp) & 31);
        xrow[j] = reinterpret_cast<const V*>(a.H + (size_t)u * a.F + a.f_lo);
        p[j] = 0.f;
      }
      for (int t = c; t < nvec; t += G) {
        const V gt = __ldg(grow + t);
        V x[U];
#pragma unroll
        for (int j = 0; j < U; ++j) x[j] = __ldg(xrow[j] + t);
#pragma unroll
        for (int j = 0; j < U; ++j) p[j] += dotv(x[j], gt);
      }
      if constexpr (G == 32) {
        // transposing butterfly: after the three exchange steps lane L holds, summed over eight
        // lanes, the dot product of edge j(L) = 4*bit4 + 2*bit3 + bit2; two more steps finish it
        float q[4], r[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const bool up = lane & 16;
          const float got = __shfl_xor_sync(kAll, up ? p[i] : p[i + 4], 16);
          q[i] = (up ? p[i + 4] : p[i]) + got;
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const bool up = lane & 8;
          const float got = __shfl_xor_sync(kAll, up ? q[i] : q[i + 2], 8);
          r[i] = (up ? q[i + 2] : q[i]) + got;
        }
        const bool up = lane & 4;
        float t = (up ? r[1] : r[0]) + __shfl_xor_sync(kAll, up ? r[0] : r[1], 4);
        t += __shfl_xor_sync(kAll, t, 2);
        t += __shfl_xor_sync(kAll, t, 1);
        const int j = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
        if ((lane & 3) == 0 && e0 + j < cnt) {
          float* w = a.dW + b + e0 + j;
          *w = a.accumulate ? *w + t * s : t * s;
        }
      } else {
#pragma unroll
        for (int j = 0; j < U; ++j) {
          float t = p[j];
#pragma unroll
          for (int off = 1; off < G; off <<= 1) t += __shfl_xor_sync(kAll, t, off);
          const int e = e0 + j * NG + grp;
          if (c == 0 && e < cnt) {
            float* w = a.dW + b + e;
            *w = a.accumulate ? *w + t * s : t * s;
          }
        }
      }
    }
  }
}

template <int VEC, int G>
// four blocks per SM (64 registers): Products-like F = 100 10.9 -> 9.2 ms against the compiler's 74
__global__ void __launch_bounds__(kGenBlock, 4) edge_grad_kernel(const EdgeGradArgs a,
                                                              const int heavy_blocks) {
  const int warp = threadIdx.x >> 5;
  if ((int)blockIdx.x < heavy_blocks) {
    const int count = min(*a.heavy_count, a.heavy_cap);
    for (int i = blockIdx.x; i < count; i += heavy_blocks) {
      const int64_t v = a.heavy_list[i];
      const int64_t lo = __ldg(a.rowptr + v), hi = __ldg(a.rowptr + v + 1);
      edge_grad_row<VEC, G>(a, v, a.seg_lo ? __ldg(a.seg_lo + v) : lo,
                            a.seg_hi ? __ldg(a.seg_hi + v) : hi, hi - lo, warp, kGenWarps);
    }
    return;
  }
  const int64_t v = (int64_t)(blockIdx.x - heavy_blocks) * kGenWarps + warp;
  if (v >= a.n) return;
  const int64_t lo = __ldg(a.rowptr + v), hi = __ldg(a.rowptr + v + 1);
  if (hi - lo > a.heavy_threshold) return;  // a block of the list walk writes this row's edges
  edge_grad_row<VEC, G>(a, v, a.seg_lo ? __ldg(a.seg_lo + v) : lo,
                        a.seg_hi ? __ldg(a.seg_hi + v) : hi, hi - lo, 0, 1);
}

template <int VEC>
dg_status_t launch_edge_grad(const dg_graph* g, const EdgeGradArgs& a, cudaStream_t s) {
  const int nvec = a.f_cnt / VEC;
  const int heavy_blocks = g->sm_count * 4;
  const unsigned grid = (unsigned)(heavy_blocks + (a.n + kGenWarps - 1) / kGenWarps);
#define DG_EG_CASE(GG)                                                              \
  if (nvec <= GG || GG == 32) {                                                     \
    edge_grad_kernel<VEC, GG><<<grid, kGenBlock, 0, s>>>(a, heavy_blocks);          \
    DG_CUDA(cudaGetLastError());                                                    \
    count_launches(1);                                                              \
    return DG_OK;                                                                   \
  }
  DG_EG_CASE(1) DG_EG_CASE(2) DG_EG_CASE(4) DG_EG_CASE(8) DG_EG_CASE(16) DG_EG_CASE(32)
#undef DG_EG_CASE
  return DG_OK;
}

int log_group(int32_t width) {  // lanes per edge: the power of two covering `width`, at most 32
  int lg = 0;
  while (lg < 5 && (1 << lg) < width) ++lg;
  return lg;
}

// Feature slices and source blocks of one general call, like the sum / mean kernels' (Algorithm 2
// with L2 as the cache): when the gathered matrices (`gathered` of them, n x F floats each) do not
// fit the handle's L2 budget, the call runs as one launch per (range of neighbour ids, slice of 128
// features: one walk of a row with 32 lanes x 4 values); the ranges partition the edges and each
// launch folds its piece into the output of the earlier ones (can_merge: max / min need the arg
// matrix for that).  Without split pointers, or where the pieces of a row would fall under 32
// edges, slices alone are used if one slice of all rows fits; otherwise the call stays one launch.
// The handle's "source_blocks" attribute forces the number of ranges.
void plan_pieces(const dg_graph* g, int32_t F, int gathered, const int32_t* split, bool can_merge,
                 int64_t* slice, int* nb) {
  *slice = F;
  *nb = 1;
  const double budget = (double)g->l2_budget_bytes;
  const int64_t w = F < 128 ? F : 128;
  const double row_bytes = (double)(w * 4 + 128) * gathered;  // a slice rarely starts on a line
  if (split && can_merge && g->source_blocks > 1) {
    *slice = w;
    *nb = (int)g->source_blocks;
    return;
  }
  if (g->source_blocks == 1 || (double)g->n * F * 4.0 * gathered <= budget) return;
  if (split && can_merge) {
    int cand = 1;
    while (cand < kFineBlocks && (double)g->n / cand * row_bytes > budget) cand *= 2;
    if ((double)g->nnz / (double)g->n / cand >= 32.0) {
      *slice = w;
      *nb = cand;
      return;
    }
  }
  if ((double)g->n * row_bytes <= budget) *slice = w;
}

inline unsigned warp_blocks(int64_t n) { return (unsigned)((n + kGenWarps - 1) / kGenWarps); }

template <template <int, int> class L>
dg_status_t dispatch_ops(int bin, int red, const GenArgs& a, cudaStream_t s) {
#define DG_GEN_CASE(B)                                                   \
  case B:                                                                \
    if (red == kSum) return L<B, kSum>::run(a, s);                       \
    if (red == kMax) return L<B, kMax>::run(a, s);                       \
    return L<B, kMin>::run(a, s);
  switch (bin) {
    DG_GEN_CASE(kCopyLhs)
    DG_GEN_CASE(kCopyRhs)
    DG_GEN_CASE(kAdd)
    DG_GEN_CASE(kSub)
    DG_GEN_CASE(kMul)
    default:
      DG_GEN_CASE(kDiv)
  }
#undef DG_GEN_CASE
}

#define DG_GEN_LAUNCHER(NAME, KERNEL)                                         \
  template <int BIN, int RED>                                                 \
  struct NAME {                                                               \
    static dg_status_t run(const GenArgs& a, cudaStream_t s) {                \
      const unsigned heavy = a.heavy_list ? (unsigned)a.heavy_blocks : 0u;    \
      KERNEL<BIN, RED><<<heavy + warp_blocks(a.n), kGenBlock, 0, s>>>(a);     \
      DG_CUDA(cudaGetLastError());                                            \
      count_launches(1);                                                      \
      return DG_OK;                                                           \
    }                                                                         \
  };
template <int BIN, int RED>
struct FwdLauncher {
  static dg_status_t run(const GenArgs& a, cudaStream_t s) {
    if constexpr (BIN == kCopyLhs && RED == kSum) {  // dg_ap_fwd hands this pair to aggregate_sum
      (void)a; (void)s;
      return DG_ERR_UNSUPPORTED;
    } else {
      const unsigned grid = (a.heavy_list ? (unsigned)a.heavy_blocks : 0u) + warp_blocks(a.n);
      if (a.vec == 4) general_fwd_kernel<BIN, RED, 4><<<grid, kGenBlock, 0, s>>>(a);
      else if (a.vec == 2) general_fwd_kernel<BIN, RED, 2><<<grid, kGenBlock, 0, s>>>(a);
      else general_fwd_kernel<BIN, RED, 1><<<grid, kGenBlock, 0, s>>>(a);
      DG_CUDA(cudaGetLastError());
      count_launches(1);
      return DG_OK;
    }
  }
};
template <int BIN, int RED>
struct BwdVertexLauncher {
  static dg_status_t run(const GenArgs& a, cudaStream_t s) {
    // dg_ap_bwd hands the pairs whose derivative is 1 to aggregate_sum
    if constexpr (RED == kSum && (BIN == kCopyLhs || BIN == kAdd || BIN == kSub)) {
      (void)a; (void)s;
      return DG_ERR_UNSUPPORTED;
    } else {
      const unsigned grid = (a.heavy_list ? (unsigned)a.heavy_blocks : 0u) + warp_blocks(a.n);
      if (a.vec == 4) general_bwd_vertex_kernel<BIN, RED, 4><<<grid, kGenBlock, 0, s>>>(a);
      else if (a.vec == 2) general_bwd_vertex_kernel<BIN, RED, 2><<<grid, kGenBlock, 0, s>>>(a);
      else general_bwd_vertex_kernel<BIN, RED, 1><<<grid, kGenBlock, 0, s>>>(a);
      DG_CUDA(cudaGetLastError());
      count_launches(1);
      return DG_OK;
    }
  }
};
// one launch per piece; L::run launches the kernel of the operator pair
template <template <int, int> class L>
dg_status_t run_pieces(const dg_graph* g, GenArgs a, int bin, int red, const int32_t* split,
                       int64_t slice, int nb, cudaStream_t s) {
  const int per = kFineBlocks / nb;
  for (int j = 0; j < nb; ++j) {
    if (nb > 1) {
      a.seg_lo = split + (size_t)(j * per) * (size_t)g->n;
      a.seg_hi = split + (size_t)((j + 1) * per) * (size_t)g->n;
    }
    a.accumulate = j > 0;
    for (int64_t f0 = 0; f0 < a.F; f0 += slice) {
      a.f_lo = (int32_t)f0;
      a.f_cnt = (int32_t)(a.F - f0 < slice ? a.F - f0 : slice);
      if (dg_status_t st = dispatch_ops<L>(bin, red, a, s)) return st;
    }
  }
  return DG_OK;
}
template <int BIN, int RED>
struct BwdEdgeFullLauncher {
  static dg_status_t run(const GenArgs& a, cudaStream_t s) {
    const unsigned grid = (a.heavy_list ? (unsigned)a.heavy_blocks : 0u) + warp_blocks(a.n);
    if (a.vec == 4) general_bwd_edge_full_kernel<BIN, RED, 4><<<grid, kGenBlock, 0, s>>>(a);
    else general_bwd_edge_full_kernel<BIN, RED, 1><<<grid, kGenBlock, 0, s>>>(a);
    DG_CUDA(cudaGetLastError());
    count_launches(1);
    return DG_OK;
  }
};
DG_GEN_LAUNCHER(BwdEdgeScalarLauncher, general_bwd_edge_scalar_kernel)
#undef DG_GEN_LAUNCHER

dg_status_t bad(const char* msg) {
  set_error("%s", msg);
  return DG_ERR_INVALID_ARG;
}

dg_status_t check_operands(const dg_graph* g, const float* fV, const float* fE, int32_t fE_cols,
                           int32_t F, int bin, int red) {
  if (!g) return bad("graph handle is NULL");
  if (F < 1) return bad("F must be >= 1");
  if (F > (1 << 20)) {
    set_error("F must be at most 2^20");
    return DG_ERR_UNSUPPORTED;
  }
  if (bin < kCopyLhs || bin > kDiv) return bad("binary must be one of the dg_binary_t values");
  if (red < kSum || red > kMin) return bad("reduce must be one of the dg_reduce_t values");
  if (bin != kCopyRhs && !fV && g->n > 0) return bad("fV is NULL (only copyrhs works without it)");
  if (bin != kCopyLhs) {
    if (!fE && g->nnz > 0) return bad("fE is NULL (only copylhs works without it)");
    if (fE_cols != 1 && fE_cols != F) return bad("fE_cols must be 1 or F");
  }
  return DG_OK;
}

}  // namespace
}  // namespace dg

using namespace dg;

extern "C" {

dg_status_t dg_ap_fwd(dg_graph_t g, const float* fV, const float* fE, int32_t fE_cols, int32_t F,
                      dg_binary_t binary, dg_reduce_t reduce, float* fO, int32_t* arg,
                      void* stream) {
  if (dg_status_t st = check_operands(g, fV, fE, fE_cols, F, (int)binary, (int)reduce)) return st;
  if (g->n == 0) return DG_OK;
  if (!fO) return bad("fO is NULL");
  // copylhs / sum is the plain sum, mul / sum with one column the weighted sum with fE as the
  // weights: the sum / mean kernels do these two (about 2.5x faster on the dense graphs)
  if (reduce == DG_RED_SUM &&
      (binary == DG_BIN_COPY_LHS || (binary == DG_BIN_MUL && fE_cols == 1)))
    return aggregate_sum(g, false, binary == DG_BIN_MUL ? fE : nullptr, fV, F, fO,
                         (cudaStream_t)stream);
  GenArgs a{};
  a.ptr = g->rowptr;
  a.idx = g->colidx;
  a.X = fV;
  a.Y = fE;
  a.out = fO;
  a.arg_out = reduce == DG_RED_SUM ? nullptr : arg;
  a.n = g->n;
  a.F = F;
  a.cols = binary == DG_BIN_COPY_LHS ? 1 : fE_cols;
  uintptr_t both = 0;
  if (binary != DG_BIN_COPY_RHS) both |= (uintptr_t)fV;
  if (binary != DG_BIN_COPY_LHS && a.cols != 1) both |= (uintptr_t)fE;
  a.vec = (F % 4 == 0 && (both & 15) == 0) ? 4 : (F % 2 == 0 && (both & 7) == 0) ? 2 : 1;
  a.log_g = log_group(F / a.vec);
  if (g->nnz > g->heavy_threshold) {  // only then can a row be on the heavy list
    a.heavy_list = g->heavy_rows;
    a.heavy_count = g->counters + 0;
    a.heavy_cap = (int32_t)g->heavy_cap;
    a.heavy_threshold = (int32_t)g->heavy_threshold;
    a.heavy_blocks = g->sm_count * 4;
  }
  int64_t slice;
  int nb;
  // copyrhs gathers nothing: its edge rows are a stream
  plan_pieces(g, F, binary == DG_BIN_COPY_RHS ? 0 : 1, g->split_csr,
              reduce == DG_RED_SUM || arg != nullptr, &slice, &nb);
  return run_pieces<FwdLauncher>(g, a, (int)binary, (int)reduce, g->split_csr, slice, nb,
                                 (cudaStream_t)stream);
}

dg_status_t dg_ap_bwd(dg_graph_t g, const float* dO, const float* fV, const float* fE,
                      int32_t fE_cols, int32_t F, dg_binary_t binary, dg_reduce_t reduce,
                      const int32_t* arg, float* dV, float* dE, void* stream) {
  if (dg_status_t st = check_operands(g, fV, fE, fE_cols, F, (int)binary, (int)reduce)) return st;
  if (g->n == 0) return DG_OK;
  if (!dO) return bad("dO is NULL");
  if (reduce != DG_RED_SUM && !arg) return bad("max / min need the arg output of dg_ap_fwd");
  if (dE && binary == DG_BIN_COPY_LHS) return bad("copylhs has no edge operand: dE must be NULL");
  cudaStream_t s = (cudaStream_t)stream;
  const int32_t cols = binary == DG_BIN_COPY_LHS ? 1 : fE_cols;
  if (dV) {
    if (binary == DG_BIN_COPY_RHS) {  // the result does not depend on fV
      DG_CUDA(cudaMemsetAsync(dV, 0, (size_t)g->n * (size_t)F * sizeof(float), s));
    } else {
      if (!g->transposed) {
        set_error("the gradient with respect to fV gathers over the CSC: call dg_graph_transpose first");
        return DG_ERR_NOT_TRANSPOSED;
      }
      // sum with copylhs / add / sub: dV[u] is the plain sum of dO over the out-edges of u
      if (reduce == DG_RED_SUM && (binary == DG_BIN_COPY_LHS || binary == DG_BIN_ADD ||
                                   binary == DG_BIN_SUB)) {
        if (dg_status_t st = aggregate_sum(g, true, nullptr, dO, F, dV, s)) return st;
      } else {
        GenArgs a{};
        a.ptr = g->colptr;
        a.idx = g->rowidx_T;
        a.perm = g->perm;
        a.X = dO;
        a.Y = fE;
        a.arg = arg;
        a.out = dV;
        a.n = g->n;
        a.F = F;
        a.cols = cols;
        uintptr_t both = (uintptr_t)dO;
        if ((binary == DG_BIN_MUL || binary == DG_BIN_DIV) && cols != 1) both |= (uintptr_t)fE;
        if (reduce != DG_RED_SUM) both |= (uintptr_t)arg;
        a.vec = (F % 4 == 0 && (both & 15) == 0) ? 4 : (F % 2 == 0 && (both & 7) == 0) ? 2 : 1;
        a.log_g = log_group(F / a.vec);
        if (g->nnz > g->heavy_threshold) {  // the heavy columns of the CSC
          a.heavy_list = g->heavy_cols;
          a.heavy_count = g->counters + 1;
          a.heavy_cap = (int32_t)g->heavy_cap;
          a.heavy_threshold = (int32_t)g->heavy_threshold;
          a.heavy_blocks = g->sm_count * 4;
        }
        int64_t slice;
        int nb;
        plan_pieces(g, F, reduce == DG_RED_SUM ? 1 : 2, g->split_csc, true, &slice, &nb);  // dO, arg
        if (dg_status_t st = run_pieces<BwdVertexLauncher>(g, a, (int)binary, (int)reduce,
                                                           g->split_csc, slice, nb, s))
          return st;
      }
    }
  }
  if (dE && g->nnz > 0) {
    // mul / sum with one edge column: dE[k] = <fV[u_k], dO[v_k]>, the edge-weight gradient of the sum
    if (binary == DG_BIN_MUL && reduce == DG_RED_SUM && cols == 1)
      return dg_aggregate_edge_grad(g, fV, dO, F, DG_OP_SUM, dE, stream);
    GenArgs a{};
    a.ptr = g->rowptr;
    a.idx = g->colidx;
    a.X = dO;
    a.V = fV;
    a.Y = fE;
    a.arg = arg;
    a.out = dE;
    a.n = g->n;
    a.F = F;
    a.cols = cols;
    a.vec = 1;
    if (cols != 1) {  // 16-byte rows of every matrix the full-width kernel touches
      uintptr_t all = (uintptr_t)dO | (uintptr_t)dE;
      if (binary == DG_BIN_MUL || binary == DG_BIN_DIV) all |= (uintptr_t)fV;
      if (binary == DG_BIN_DIV) all |= (uintptr_t)fE;
      if (reduce != DG_RED_SUM) all |= (uintptr_t)arg;
      if (F % 4 == 0 && (all & 15) == 0) a.vec = 4;
    }
    a.log_g = log_group(F / a.vec);
    if (g->nnz > g->heavy_threshold) {
      a.heavy_list = g->heavy_rows;
      a.heavy_count = g->counters + 0;
      a.heavy_cap = (int32_t)g->heavy_cap;
      a.heavy_threshold = (int32_t)g->heavy_threshold;
      a.heavy_blocks = g->sm_count * 4;
    }
    if (cols == 1)
      return dispatch_ops<BwdEdgeScalarLauncher>((int)binary, (int)reduce, a, s);
    return dispatch_ops<BwdEdgeFullLauncher>((int)binary, (int)reduce, a, s);
  }
  return DG_OK;
}

dg_status_t dg_aggregate_edge_grad(dg_graph_t g, const float* H, const float* dOut, int32_t F,
                                   dg_op_t op, float* dW, void* stream) {
  if (!g) return bad("graph handle is NULL");
  if (F < 1) return bad("F must be >= 1");
  if (F > (1 << 20)) {
    set_error("F must be at most 2^20");
    return DG_ERR_UNSUPPORTED;
  }
  if (op != DG_OP_SUM && op != DG_OP_MEAN) return bad("op must be DG_OP_SUM or DG_OP_MEAN");
  if (g->nnz == 0) return DG_OK;
  if (!H || !dOut || !dW) return bad("H, dOut or dW is NULL");
  EdgeGradArgs a{};
  a.rowptr = g->rowptr;
  a.colidx = g->colidx;
  a.H = H;
  a.dOut = dOut;
  a.dW = dW;
  a.heavy_list = g->heavy_rows;
  a.heavy_count = g->counters + 0;
  a.heavy_cap = (int32_t)g->heavy_cap;
  a.heavy_threshold = (int32_t)g->heavy_threshold;
  a.n = g->n;
  a.F = F;
  a.row_scale = op == DG_OP_MEAN ? (g->self_loops ? 2 : 1) : 0;
  cudaStream_t s = (cudaStream_t)stream;
  const uintptr_t both = (uintptr_t)H | (uintptr_t)dOut;
  const int vec = (F % 4 == 0 && (both & 15) == 0) ? 4 : (F % 2 == 0 && (both & 7) == 0) ? 2 : 1;
  // Like the aggregation itself (Algorithm 2 with L2 as the cache): when the gathered matrix
  // does not stay L2-resident and the rows carry split pointers, the call is cut into feature
  // slices of 128 vectors and source-vertex blocks sized to the L2 budget, one launch each; the
  // blocks partition the edges, the slices add up in dW.
  int64_t slice = F;
  int nb = 1;
  if (g->split_csr && (double)g->n * F * 4.0 > (double)g->l2_budget_bytes) {
    slice = 128LL * vec < F ? 128LL * vec : F;
    while (nb < kFineBlocks && (double)g->n / nb * (double)(slice * 4 + 128) > (double)g->l2_budget_bytes)
      nb *= 2;
    if ((double)g->nnz / (double)g->n / nb < 32.0) { nb = 1; slice = F; }  // pieces too short to pay
  }
  const int per = kFineBlocks / nb;
  for (int j = 0; j < nb; ++j) {
    if (nb > 1) {
      a.seg_lo = g->split_csr + (size_t)(j * per) * (size_t)g->n;
      a.seg_hi = g->split_csr + (size_t)((j + 1) * per) * (size_t)g->n;
    }
    for (int64_t f0 = 0; f0 < F; f0 += slice) {
      a.f_lo = (int32_t)f0;
      a.f_cnt = (int32_t)(F - f0 < slice ? F - f0 : slice);
      a.accumulate = f0 > 0;
      const dg_status_t st = vec == 4 ? launch_edge_grad<4>(g, a, s)
                           : vec == 2 ? launch_edge_grad<2>(g, a, s) : launch_edge_grad<1>(g, a, s);
      if (st != DG_OK) return st;
    }
  }
  return DG_OK;
}

}  // extern "C"
