// CSR -> CSC on the GPU as a stable least-significant-digit radix sort of (key = colidx[k],
// value = k).  The paper keeps the graph in CSR only (Section 3.1) and leaves the reverse graph
// of the backward pass implicit; the result here is defined as the stable counting sort of the
// edge positions by source vertex, which has exactly one correct answer.
//
// The digits are 8 bits wide, or 9 where that pays (see sort_plan).  One pass over a digit is
// three kernels and never makes one block wait for another:
//   1. digit_histogram : per tile of kTile keys, the number of keys per digit -> hist[digit][tile]
//   2. exclusive scan of hist (digit-major, so the scan yields global output offsets):
//      scan_reduce -> scan_spine (one block) -> scan_apply
//   3. digit_scatter   : ranks every key inside its tile in input order (ballots over the digit
//      bits inside a warp, per-warp counters across rounds, a fixed pass across the warps), stages
//      the tile sorted by digit in shared memory and writes each digit run to its global offset.
// Stability of every step makes the final order (key, k) ascending.  After the last pass the
// sorted keys give colptr by boundary detection, and perm gives rowidx_T and w_T by gathers.
#include "dg_internal.cuh"

namespace dg {
namespace {

constexpr int kMaxRadixBits = 9;
constexpr int kSortBlock = 256;
constexpr int kSortWarps = kSortBlock / 32;
constexpr int kItems = 16;                       // keys per thread
constexpr int kTile = kSortBlock * kItems;       // 4096 keys per block
constexpr int kScanBlock = 256;
constexpr int kScanItems = 16;
constexpr int kScanChunk = kScanBlock * kScanItems;
constexpr unsigned kFull = 0xffffffffu;

template <int BITS>
__device__ __forceinline__ uint32_t digit_of(uint32_t key, int shift) {
  return (key >> shift) & ((1u << BITS) - 1u);
}

// A thread reads its keys as 16-byte vectors when the array allows it (four loads in flight
// then cover the whole tile; with 4-byte loads the kernel waited on memory at a third of the
// copy bandwidth).  The caller's colidx, the keys of the first pass, is only 4-byte aligned in
// general: `vector_ok` says whether keys is 16-byte aligned.
template <int BITS>
__global__ void __launch_bounds__(kSortBlock)
digit_histogram(const uint32_t* __restrict__ keys, int64_t count, int shift, int64_t tiles,
                int vector_ok, uint32_t* __restrict__ hist) {
  constexpr int R = 1 << BITS;
  __shared__ uint32_t h[R];
  for (int d = threadIdx.x; d < R; d += kSortBlock) h[d] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kTile;
  if (vector_ok && base + kTile <= count) {
    const uint4* v = reinterpret_cast<const uint4*>(keys + base);
    uint4 k[kItems / 4];
#pragma unroll
    for (int i = 0; i < kItems / 4; ++i) k[i] = v[i * kSortBlock + threadIdx.x];
#pragma unroll
    for (int i = 0; i < kItems / 4; ++i) {
      atomicAdd(&h[digit_of<BITS>(k[i].x, shift)], 1u);
      atomicAdd(&h[digit_of<BITS>(k[i].y, shift)], 1u);
      atomicAdd(&h[digit_of<BITS>(k[i].z, shift)], 1u);
      atomicAdd(&h[digit_of<BITS>(k[i].w, shift)], 1u);
    }
  } else {
#pragma unroll 4
    for (int i = 0; i < kItems; ++i) {
      const int64_t k = base + i * kSortBlock + threadIdx.x;
      if (k < count) atomicAdd(&h[digit_of<BITS>(keys[k], shift)], 1u);
    }
  }
  __syncthreads();
  for (int d = threadIdx.x; d < R; d += kSortBlock) hist[(int64_t)d * tiles + blockIdx.x] = h[d];
}

// ---- exclusive scan of a uint32 array of length m (in place), three kernels ----
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* total) {
  __shared__ uint32_t warp_sums[kScanBlock / 32];
  __shared__ uint32_t block_total;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t t = __shfl_up_sync(kFull, inc, d);
    if (lane >= d) inc += t;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = lane < kScanBlock / 32 ? warp_sums[lane] : 0;
    uint32_t winc = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t t = __shfl_up_sync(kFull, winc, d);
      if (lane >= d) winc += t;
    }
    if (lane < kScanBlock / 32) warp_sums[lane] = winc - w;
    if (lane == kScanBlock / 32 - 1) block_total = winc;
  }
  __syncthreads();
  const uint32_t r = inc - v + warp_sums[warp];
  *total = block_total;
  __syncthreads();  // the shared arrays may be reused by the next call
  return r;
}

__global__ void __launch_bounds__(kScanBlock)
scan_reduce(const uint32_t* __restrict__ data, int64_t m, uint32_t* __restrict__ chunk_sums) {
  const int64_t base = (int64_t)blockIdx.x * kScanChunk + (int64_t)threadIdx.x * kScanItems;
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i)
    if (base + i < m) s += data[base + i];
  uint32_t total;
  block_exclusive_scan(s, &total);
  if (threadIdx.x == 0) chunk_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kScanBlock)
scan_spine(uint32_t* __restrict__ chunk_sums, int64_t chunks) {
  uint32_t carry = 0;
  for (int64_t base = 0; base < chunks; base += kScanBlock) {
    const int64_t i = base + threadIdx.x;
    const uint32_t v = i < chunks ? chunk_sums[i] : 0;
    uint32_t total;
    const uint32_t ex = block_exclusive_scan(v, &total);
    if (i < chunks) chunk_sums[i] = carry + ex;
    carry += total;
  }
}

__global__ void __launch_bounds__(kScanBlock)
scan_apply(uint32_t* __restrict__ data, int64_t m, const uint32_t* __restrict__ chunk_sums) {
  const int64_t base = (int64_t)blockIdx.x * kScanChunk + (int64_t)threadIdx.x * kScanItems;
  uint32_t v[kScanItems];
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    v[i] = base + i < m ? data[base + i] : 0;
    s += v[i];
  }
  uint32_t total;
  uint32_t run = block_exclusive_scan(s, &total) + chunk_sums[blockIdx.x];
#pragma unroll
  for (int i = 0; i < kScanItems; ++i) {
    if (base + i < m) data[base + i] = run;
    run += v[i];
  }
}

// Lanes of the warp that hold the same digit as this lane (lanes without a key only match one
// another): one ballot per digit bit, each keeping the lanes that agree with this lane on that
// bit.  Unlike match.any, whose cost grows with the number of distinct values in the warp (about
// 30 for the random low digits of vertex ids), this costs the same for every digit mix.
template <int BITS>
__device__ __forceinline__ unsigned digit_peers(uint32_t d, bool valid) {
  const unsigned have = __ballot_sync(kFull, valid);
  unsigned peers = valid ? have : ~have;
#pragma unroll
  for (int b = 0; b < BITS; ++b) {
    const bool bit = (d >> b) & 1u;
    const unsigned m = __ballot_sync(kFull, bit);
    peers &= bit ? m : ~m;
  }
  return peers;
}

// ---- stable scatter of one tile ----
// vals_in == nullptr means "the value of key k is k" (first pass).  keys_out may be nullptr when
// the sorted keys are not needed (never the case for the last pass, which feeds colptr).
// Four blocks per SM (64 registers a thread): the ranking is a chain of shared-memory and
// ballot latencies, and the fourth block hides more of it than the few spilled words cost
// (three blocks at 80 registers were 10 % slower, five with the values read late 3 % slower).
template <int BITS>
__global__ void __launch_bounds__(kSortBlock, 4)
digit_scatter(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
              int64_t count, int shift, int64_t tiles, const uint32_t* __restrict__ offsets,
              uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out) {
  constexpr int R = 1 << BITS;
  constexpr int DPT = R / kSortBlock;  // digits a thread owns (consecutive ones): 1 or 2
  // A warp ranks its 512 keys as two streams of 256 (rounds 0..7 and 8..15), each with its own
  // counters, so that two independent chains of counter updates are in flight at a time.
  // Dynamic shared memory (52 KB with 9-bit digits): cnt_a, cnt_b, digit_base, global_base,
  // skeys, svals.
  extern __shared__ __align__(16) unsigned char scatter_smem[];
  uint16_t (*cnt_a)[R] = reinterpret_cast<uint16_t (*)[R]>(scatter_smem);
  uint16_t (*cnt_b)[R] = cnt_a + kSortWarps;
  uint32_t* digit_base = reinterpret_cast<uint32_t*>(cnt_b + kSortWarps);
  uint32_t* global_base = digit_base + R;
  uint32_t* skeys = global_base + R;
  uint32_t* svals = skeys + kTile;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned lt_mask = (1u << lane) - 1u;
  const int64_t tile_base = (int64_t)blockIdx.x * kTile;
  const int64_t remaining = count - tile_base;
  const int tile_count = remaining < kTile ? (int)remaining : kTile;

  // this tile's global offsets of the thread's digits: fetched now, needed after the ranking
  uint32_t my_global_base[DPT];
#pragma unroll
  for (int i = 0; i < DPT; ++i)
    my_global_base[i] = offsets[(int64_t)(threadIdx.x * DPT + i) * tiles + blockIdx.x];
  for (int w = 0; w < kSortWarps; ++w) {
#pragma unroll
    for (int i = 0; i < DPT; ++i) {
      cnt_a[w][threadIdx.x * DPT + i] = 0;
      cnt_b[w][threadIdx.x * DPT + i] = 0;
    }
  }
  __syncthreads();

  // Warp `warp` owns keys [warp*512, warp*512+512) of the tile, 32 consecutive keys per round,
  // so (warp, round, lane) order is input order.
  uint32_t key[kItems];
  uint32_t val[kItems];
  uint16_t rank[kItems];
#pragma unroll
  for (int r = 0; r < kItems; ++r) {
    const int local = warp * (32 * kItems) + r * 32 + lane;
    const bool valid = local < tile_count;
    key[r] = valid ? keys_in[tile_base + local] : 0u;
    val[r] = valid ? (vals_in ? vals_in[tile_base + local] : (uint32_t)(tile_base + local)) : 0u;
  }
  constexpr int kHalf = kItems / 2;
#pragma unroll
  for (int r = 0; r < kHalf; ++r) {
#pragma unroll
    for (int stream = 0; stream < 2; ++stream) {
      const int rr = r + stream * kHalf;
      uint16_t* cnt = stream ? cnt_b[warp] : cnt_a[warp];
      const bool valid = warp * (32 * kItems) + rr * 32 + lane < tile_count;
      const uint32_t d = valid ? digit_of<BITS>(key[rr], shift) : 0u;
      const unsigned peers = digit_peers<BITS>(d, valid);
      const int leader = __ffs(peers) - 1;
      uint32_t before = 0;
      if (valid && lane == leader) {
        before = cnt[d];
        cnt[d] = (uint16_t)(before + __popc(peers));
      }
      before = __shfl_sync(kFull, before, leader);
      rank[rr] = (uint16_t)(before + __popc(peers & lt_mask));
    }
    __syncwarp();
  }
  __syncthreads();

  // a thread owns DPT consecutive digits: exclusive prefix over (warp, stream) inside each, then
  // over the digits
  {
    uint32_t in_digit[DPT];
    uint32_t mine = 0;
#pragma unroll
    for (int i = 0; i < DPT; ++i) {
      const int d = threadIdx.x * DPT + i;
      uint32_t run = 0;
#pragma unroll
      for (int w = 0; w < kSortWarps; ++w) {
        const uint32_t ca = cnt_a[w][d];
        cnt_a[w][d] = (uint16_t)run;
        run += ca;
        const uint32_t cb = cnt_b[w][d];
        cnt_b[w][d] = (uint16_t)run;
        run += cb;
      }
      in_digit[i] = run;
      mine += run;
    }
    uint32_t total;
    uint32_t start = block_exclusive_scan(mine, &total);
#pragma unroll
    for (int i = 0; i < DPT; ++i) {
      digit_base[threadIdx.x * DPT + i] = start;
      global_base[threadIdx.x * DPT + i] = my_global_base[i];
      start += in_digit[i];
    }
  }
  __syncthreads();

#pragma unroll
  for (int r = 0; r < kItems; ++r) {
    const int local = warp * (32 * kItems) + r * 32 + lane;
    if (local < tile_count) {
      const uint32_t d = digit_of<BITS>(key[r], shift);
      const uint32_t in_digit = r < kHalf ? cnt_a[warp][d] : cnt_b[warp][d];
      const uint32_t pos = digit_base[d] + in_digit + rank[r];
      skeys[pos] = key[r];
      svals[pos] = val[r];
    }
  }
  __syncthreads();

  for (int i = threadIdx.x; i < tile_count; i += kSortBlock) {
    const uint32_t k = skeys[i];
    const uint32_t d = digit_of<BITS>(k, shift);
    const uint32_t dst = global_base[d] + ((uint32_t)i - digit_base[d]);
    if (keys_out) keys_out[dst] = k;
    vals_out[dst] = svals[i];
  }
}

template <int BITS>
constexpr size_t scatter_smem_bytes() {
  return (size_t)2 * kSortWarps * (1 << BITS) * sizeof(uint16_t) + (size_t)2 * (1 << BITS) * sizeof(uint32_t) +
         (size_t)2 * kTile * sizeof(uint32_t);
}

// colptr[u] = first position q whose sorted key is >= u.  Position q fills the ids between the
// key before it and its own key; position nnz closes the array up to n.  A thread takes
// kColptrItems consecutive positions (one 16-byte load when `vector_ok`: sorted 16-byte aligned)
// and fills at most the last kMaxFill ids of a gap itself: a long run of ids without a key (a
// hub-first numbering puts every vertex without out-edges at the end, millions of them) would
// otherwise be one thread's loop (Papers-like x0.1, hub-first: 17 ms).  The ids it leaves keep
// the -1 the array was filled with, and fill_long_gaps finds each by a binary search.
constexpr int kColptrItems = 4;
constexpr int kMaxFill = 32;
__global__ void colptr_from_sorted_keys(const uint32_t* __restrict__ sorted, int64_t nnz,
                                        int64_t n, int vector_ok, int64_t* __restrict__ colptr) {
  const int64_t q0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kColptrItems;
  if (q0 > nnz) return;
  uint32_t k[kColptrItems];
  if (vector_ok && q0 + kColptrItems <= nnz) {
    const uint4 v = *reinterpret_cast<const uint4*>(sorted + q0);
    k[0] = v.x; k[1] = v.y; k[2] = v.z; k[3] = v.w;
  } else {
#pragma unroll
    for (int i = 0; i < kColptrItems; ++i) k[i] = q0 + i < nnz ? sorted[q0 + i] : 0u;
  }
  int64_t prev = q0 > 0 ? (int64_t)sorted[q0 - 1] : -1;
#pragma unroll
  for (int i = 0; i < kColptrItems; ++i) {
    const int64_t q = q0 + i;
    if (q > nnz) break;
    int64_t cur = q < nnz ? (int64_t)k[i] : n;
    const int64_t next_prev = cur;
    if (cur > n) cur = n;  // an id outside [0, n) must not turn into a write outside colptr
    int64_t u = prev + 1;
    if (cur - u >= kMaxFill) u = cur - kMaxFill + 1;
    for (; u <= cur; ++u) colptr[u] = q;
    prev = next_prev;
  }
}

// the ids colptr_from_sorted_keys left at -1: the first position whose key is >= u, by search
__global__ void fill_long_gaps(const uint32_t* __restrict__ sorted, int64_t nnz, int64_t n,
                               int64_t* __restrict__ colptr) {
  const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (u > n || colptr[u] >= 0) return;
  int64_t lo = 0, hi = nnz;  // invariant: keys before lo are < u, keys from hi on are >= u
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(sorted + mid) < u) lo = mid + 1;
    else hi = mid;
  }
  colptr[u] = lo;
}

// row_info[k] = (row r with rowptr[r] <= k < rowptr[r+1], bits of 1/(deg(r) + self)) for every
// CSR position k; self = 1 when the graph has implicit self loops, else 0.  A thread takes kRowItems consecutive positions: one binary search for the first, then a
// galloping search forward from the previous row for each of the others (rows are usually a few
// positions long, empty rows are skipped in doubling strides).  Searching once per perm[q] in
// CSC order instead, with random access to rowptr, took 218 ms of the 296 ms transpose of the
// 1.6 G-edge graph.
constexpr int kRowItems = 8;
__global__ void row_info_kernel(const int64_t* __restrict__ rowptr, int self, int64_t n,
                                int64_t nnz, uint2* __restrict__ row_info) {
  const int64_t k0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kRowItems;
  if (k0 >= nnz) return;
  int64_t lo = 0, hi = n;  // invariant: rowptr[lo] <= k0 < rowptr[hi]
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if (__ldg(rowptr + mid) <= k0) lo = mid; else hi = mid;
  }
  int64_t r = lo;
  int64_t r_end = __ldg(rowptr + r + 1);  // first position after row r
#pragma unroll 1
  for (int i = 0; i < kRowItems; ++i) {
    const int64_t k = k0 + i;
    if (k >= nnz) break;
    if (k >= r_end) {
      // gallop: find a row `hi2` with rowptr[hi2] > k, then bisect (r, hi2]
      int64_t step = 1, lo2 = r, hi2 = r + 1;
      while (hi2 < n && __ldg(rowptr + hi2) <= k) {
        lo2 = hi2;
        step <<= 1;
        hi2 = hi2 + step < n ? hi2 + step : n;
      }
      while (hi2 - lo2 > 1) {
        const int64_t mid = (lo2 + hi2) >> 1;
        if (__ldg(rowptr + mid) <= k) lo2 = mid; else hi2 = mid;
      }
      r = lo2;
      r_end = __ldg(rowptr + r + 1);
    }
    // k lies in row r, so deg(r) >= 1
    const float inv = 1.0f / (float)(r_end - __ldg(rowptr + r) + self);
    row_info[k] = make_uint2((uint32_t)r, __float_as_uint(inv));
  }
}

// The same walk with another payload: out[k] = map[r] (or r) for the row r that holds position k.
__global__ void expand_rows_kernel(const int64_t* __restrict__ rowptr, int64_t n, int64_t nnz,
                                   const int32_t* __restrict__ map, uint32_t* __restrict__ out) {
  const int64_t k0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kRowItems;
  if (k0 >= nnz) return;
  int64_t lo = 0, hi = n;  // invariant: rowptr[lo] <= k0 < rowptr[hi]
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if (__ldg(rowptr + mid) <= k0) lo = mid; else hi = mid;
  }
  int64_t r = lo;
  int64_t r_end = __ldg(rowptr + r + 1);
  uint32_t payload = map ? (uint32_t)__ldg(map + r) : (uint32_t)r;
#pragma unroll 1
  for (int i = 0; i < kRowItems; ++i) {
    const int64_t k = k0 + i;
    if (k >= nnz) break;
    if (k >= r_end) {
      int64_t step = 1, lo2 = r, hi2 = r + 1;
      while (hi2 < n && __ldg(rowptr + hi2) <= k) {
        lo2 = hi2;
        step <<= 1;
        hi2 = hi2 + step < n ? hi2 + step : n;
      }
      while (hi2 - lo2 > 1) {
        const int64_t mid = (lo2 + hi2) >> 1;
        if (__ldg(rowptr + mid) <= k) lo2 = mid; else hi2 = mid;
      }
      r = lo2;
      r_end = __ldg(rowptr + r + 1);
      payload = map ? (uint32_t)__ldg(map + r) : (uint32_t)r;
    }
    out[k] = payload;
  }
}

// rowidx_T[q] = row of perm[q];  w_T[q] = edge_w[perm[q]];  mean_scale_T[q] = w_T[q] (1 if
// unweighted) / (deg(row) + self), the factor of edge q in the backward pass of the mean, so that
// the backward kernel streams it instead of gathering 1/deg.  One 8-byte gather per edge.
__global__ void gather_rows_and_weights(const uint32_t* __restrict__ perm, int64_t nnz,
                                        const uint2* __restrict__ row_info,
                                        const float* __restrict__ edge_w,
                                        int32_t* __restrict__ rowidx_T, float* __restrict__ w_T,
                                        float* __restrict__ mean_scale_T) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= nnz) return;
  const int64_t k = perm[q];
  const uint2 info = __ldg(row_info + k);
  rowidx_T[q] = (int32_t)info.x;
  float w = 1.f;
  if (edge_w) {
    w = edge_w[k];
    w_T[q] = w;
  }
  mean_scale_T[q] = w * __uint_as_float(info.y);
}

// After the caller changed edge_w in place (learnable edge weights): the two weight arrays of the
// CSC again, from perm.  The in-degree comes from the CSR row pointer.
__global__ void regather_weights_kernel(const uint32_t* __restrict__ perm, int64_t nnz,
                                        const float* __restrict__ edge_w,
                                        const int32_t* __restrict__ rowidx_T,
                                        const int64_t* __restrict__ rowptr, int self,
                                        float* __restrict__ w_T, float* __restrict__ mean_scale_T) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= nnz) return;
  const float w = edge_w[perm[q]];
  const int64_t v = rowidx_T[q];
  w_T[q] = w;
  mean_scale_T[q] = w * (1.0f / (float)(__ldg(rowptr + v + 1) - __ldg(rowptr + v) + self));
}

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
inline int aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

struct Layout {
  // csc storage
  size_t colptr_off, rowidx_off, perm_off, w_off, mscale_off, split_off, csc_bytes;
  // scratch
  size_t keys_a_off, keys_b_off, vals_off, hist_off, sums_off, scratch_bytes;
  int64_t tiles, hist_len, chunks;
  int passes;
};

Layout make_layout(int64_t n, int64_t nnz, bool weighted) {
  Layout L{};
  size_t o = 0;
  L.colptr_off = o; o += align256((size_t)(n + 1) * 8);
  L.rowidx_off = o; o += align256((size_t)nnz * 4);
  L.perm_off = o;   o += align256((size_t)nnz * 4);
  L.w_off = o;      o += weighted ? align256((size_t)nnz * 4) : 0;
  L.mscale_off = o; o += align256((size_t)nnz * 4);
  L.split_off = o;  o += wants_split(n, nnz) ? align256((size_t)(kFineBlocks + 1) * n * 4) : 0;
  L.csc_bytes = o > 0 ? o : 256;
  L.passes = sort_plan(n).passes;
  L.tiles = (nnz + kTile - 1) / kTile;
  L.hist_len = L.tiles * (1 << kMaxRadixBits);
  L.chunks = (L.hist_len + kScanChunk - 1) / kScanChunk;
  o = 0;
  L.keys_a_off = o; o += align256((size_t)nnz * 4);
  L.keys_b_off = o; o += align256((size_t)nnz * 4);
  L.vals_off = o;   o += align256((size_t)nnz * 4);
  L.hist_off = o;   o += align256((size_t)L.hist_len * 4);
  L.sums_off = o;   o += align256((size_t)(L.chunks > 0 ? L.chunks : 1) * 4);
  L.scratch_bytes = o > 0 ? o : 256;
  return L;
}

}  // namespace

// Digit width and number of passes for keys in [0, key_range).  A 9-bit pass costs about a third
// more than an 8-bit one (nine ballots per ranking round, twice the counters and histogram, more
// spilled registers: measured on the 1.6 G-edge graph, 27 key bits, 3 x 9 bits took 100.3 ms
// against 98.1 ms for 4 x 8), so the wider digit is taken only where it turns three passes into
// two or two into one (key ranges of 9, 17 and 18 bits: the Reddit- and Proteins-like graphs,
// whose transposition gains 5 %).
SortPlan sort_plan(int64_t key_range) {
  int bits = 1;
  while (bits < 31 && ((int64_t)1 << bits) < key_range) ++bits;
  const int p8 = (bits + 7) / 8, p9 = (bits + 8) / 9;
  SortPlan plan;
  const bool wide = 4 * p9 < 3 * p8;
  plan.digit_bits = wide ? 9 : 8;
  plan.passes = wide ? p9 : p8;
  return plan;
}

// Sized for the wider digit, so that one workspace query serves every key range.
void sort_scratch_sizes(int64_t count, size_t* hist_bytes, size_t* sums_bytes) {
  const int64_t tiles = (count + kTile - 1) / kTile;
  const int64_t hist_len = tiles * (1 << kMaxRadixBits);
  const int64_t chunks = (hist_len + kScanChunk - 1) / kScanChunk;
  *hist_bytes = align256((size_t)(hist_len > 0 ? hist_len : 1) * 4);
  *sums_bytes = align256((size_t)(chunks > 0 ? chunks : 1) * 4);
}

template <int BITS>
static dg_status_t sort_passes_run(const uint32_t* keys_in, const uint32_t* vals_in, int64_t count,
                                   int passes, uint32_t* const keys_buf[2], uint32_t* vals_final,
                                   uint32_t* vals_tmp, uint32_t* hist, uint32_t* sums,
                                   const uint32_t** sorted_keys, cudaStream_t s) {
  const int64_t tiles = (count + kTile - 1) / kTile;
  const int64_t hist_len = tiles * (1 << BITS);
  const int64_t chunks = (hist_len + kScanChunk - 1) / kScanChunk;
  constexpr size_t smem = scatter_smem_bytes<BITS>();
  DG_CUDA(cudaFuncSetAttribute(digit_scatter<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem));
  for (int p = 0; p < passes; ++p) {
    const int shift = p * BITS;
    // value buffers alternate so that the last pass lands in vals_final
    uint32_t* vals_out = ((passes - 1 - p) % 2 == 0) ? vals_final : vals_tmp;
    uint32_t* keys_out = keys_buf[p % 2];
    digit_histogram<BITS><<<(unsigned)tiles, kSortBlock, 0, s>>>(keys_in, count, shift, tiles,
                                                                 aligned16(keys_in), hist);
    DG_CUDA(cudaGetLastError());
    scan_reduce<<<(unsigned)chunks, kScanBlock, 0, s>>>(hist, hist_len, sums);
    DG_CUDA(cudaGetLastError());
    scan_spine<<<1, kScanBlock, 0, s>>>(sums, chunks);
    DG_CUDA(cudaGetLastError());
    scan_apply<<<(unsigned)chunks, kScanBlock, 0, s>>>(hist, hist_len, sums);
    DG_CUDA(cudaGetLastError());
    digit_scatter<BITS><<<(unsigned)tiles, kSortBlock, smem, s>>>(keys_in, vals_in, count, shift,
                                                                  tiles, hist, keys_out, vals_out);
    DG_CUDA(cudaGetLastError());
    count_launches(5);
    keys_in = keys_out;
    vals_in = vals_out;
  }
  *sorted_keys = keys_in;
  return DG_OK;
}

// Stable LSD radix sort of `count` (key, value) pairs.  vals_in == nullptr means "the value of key
// i is i".  keys_in is only read; the sorted keys end in one of keys_buf (reported through
// *sorted_keys; keys_in may be keys_buf[1], which is first written by the second pass), the
// sorted values in vals_final (vals_tmp is the other buffer of the ping-pong).
dg_status_t sort_pairs(const uint32_t* keys_in, const uint32_t* vals_in, int64_t count,
                       SortPlan plan, uint32_t* const keys_buf[2], uint32_t* vals_final,
                       uint32_t* vals_tmp, uint32_t* hist, uint32_t* sums,
                       const uint32_t** sorted_keys, cudaStream_t s) {
  if (plan.digit_bits == 9)
    return sort_passes_run<9>(keys_in, vals_in, count, plan.passes, keys_buf, vals_final, vals_tmp,
                              hist, sums, sorted_keys, s);
  return sort_passes_run<8>(keys_in, vals_in, count, plan.passes, keys_buf, vals_final, vals_tmp,
                            hist, sums, sorted_keys, s);
}

// ptr[u] = first position whose sorted key is >= u, for u = 0..n (ptr[n] = count)
dg_status_t pointers_from_sorted_keys(const uint32_t* sorted, int64_t count, int64_t n,
                                      int64_t* ptr, cudaStream_t s) {
  DG_CUDA(cudaMemsetAsync(ptr, 0xFF, (size_t)(n + 1) * sizeof(int64_t), s));  // -1 everywhere
  const unsigned blocks = (unsigned)(((count + kColptrItems) / kColptrItems + 255) / 256);
  colptr_from_sorted_keys<<<blocks, 256, 0, s>>>(sorted, count, n, aligned16(sorted), ptr);
  DG_CUDA(cudaGetLastError());
  fill_long_gaps<<<(unsigned)((n + 1 + 255) / 256), 256, 0, s>>>(sorted, count, n, ptr);
  DG_CUDA(cudaGetLastError());
  count_launches(2);
  return DG_OK;
}

// out[k] = map[r] (r itself when map is nullptr) for the CSR row r that contains position k
dg_status_t expand_rows(const int64_t* rowptr, int64_t n, int64_t nnz, const int32_t* map,
                        uint32_t* out, cudaStream_t s) {
  if (nnz == 0) return DG_OK;
  const unsigned blocks = (unsigned)(((nnz + kRowItems - 1) / kRowItems + 255) / 256);
  expand_rows_kernel<<<blocks, 256, 0, s>>>(rowptr, n, nnz, map, out);
  DG_CUDA(cudaGetLastError());
  count_launches(1);
  return DG_OK;
}

void transpose_sizes(int64_t n, int64_t nnz, bool weighted, size_t* csc_bytes,
                     size_t* scratch_bytes) {
  const Layout L = make_layout(n, nnz, weighted);
  *csc_bytes = L.csc_bytes;
  *scratch_bytes = L.scratch_bytes;
}

dg_status_t refresh_csc_weights(Graph* g, cudaStream_t s) {
  if (g->nnz == 0 || !g->edge_w) return DG_OK;
  regather_weights_kernel<<<(unsigned)((g->nnz + 255) / 256), 256, 0, s>>>(
      reinterpret_cast<const uint32_t*>(g->perm), g->nnz, g->edge_w, g->rowidx_T, g->rowptr,
      g->self_loops_in_csc ? 1 : 0, const_cast<float*>(g->w_T), const_cast<float*>(g->mean_scale_T));
  DG_CUDA(cudaGetLastError());
  count_launches(1);
  return DG_OK;
}

dg_status_t transpose_run(Graph* g, void* csc, void* scratch, cudaStream_t s) {
  const int64_t n = g->n, nnz = g->nnz;
  const bool weighted = g->edge_w != nullptr;
  const Layout L = make_layout(n, nnz, weighted);
  char* cb = static_cast<char*>(csc);
  char* sb = static_cast<char*>(scratch);
  int64_t* colptr = reinterpret_cast<int64_t*>(cb + L.colptr_off);
  int32_t* rowidx_T = reinterpret_cast<int32_t*>(cb + L.rowidx_off);
  uint32_t* perm = reinterpret_cast<uint32_t*>(cb + L.perm_off);
  float* w_T = weighted ? reinterpret_cast<float*>(cb + L.w_off) : nullptr;
  float* mean_scale_T = reinterpret_cast<float*>(cb + L.mscale_off);
  uint32_t* keys_buf[2] = {reinterpret_cast<uint32_t*>(sb + L.keys_a_off),
                           reinterpret_cast<uint32_t*>(sb + L.keys_b_off)};
  uint32_t* vals_tmp = reinterpret_cast<uint32_t*>(sb + L.vals_off);
  uint32_t* hist = reinterpret_cast<uint32_t*>(sb + L.hist_off);
  uint32_t* sums = reinterpret_cast<uint32_t*>(sb + L.sums_off);

  if (nnz == 0) {
    DG_CUDA(cudaMemsetAsync(colptr, 0, (size_t)(n + 1) * 8, s));
  } else {
    const uint32_t* keys_in = nullptr;
    if (dg_status_t st = sort_pairs(reinterpret_cast<const uint32_t*>(g->colidx), nullptr, nnz,
                                    sort_plan(n), keys_buf, perm, vals_tmp, hist, sums, &keys_in, s))
      return st;
    if (dg_status_t st = pointers_from_sorted_keys(keys_in, nnz, n, colptr, s)) return st;
    const unsigned b2 = (unsigned)((nnz + 255) / 256);
    // colptr has been derived from the sorted keys (stream order), so both key buffers, which
    // are adjacent in the scratch, are free: they hold the nnz (row, 1/deg) pairs
    uint2* row_info = reinterpret_cast<uint2*>(sb + L.keys_a_off);
    const unsigned b3 = (unsigned)(((nnz + kRowItems - 1) / kRowItems + 255) / 256);
    row_info_kernel<<<b3, 256, 0, s>>>(g->rowptr, g->self_loops ? 1 : 0, n, nnz, row_info);
    DG_CUDA(cudaGetLastError());
    gather_rows_and_weights<<<b2, 256, 0, s>>>(perm, nnz, row_info, g->edge_w, rowidx_T, w_T,
                                               mean_scale_T);
    DG_CUDA(cudaGetLastError());
    count_launches(2);
  }
  g->colptr = colptr;
  g->rowidx_T = rowidx_T;
  g->perm = reinterpret_cast<const int32_t*>(perm);
  g->w_T = w_T;
  g->mean_scale_T = mean_scale_T;
  g->self_loops_in_csc = g->self_loops;
  g->split_csc = nullptr;
  if (wants_split(n, nnz)) {
    // the columns come out of the stable sort ordered by row, so the check never fires here
    int32_t* split = reinterpret_cast<int32_t*>(cb + L.split_off);
    if (dg_status_t st = build_split(colptr, rowidx_T, n, g->fine_rows, split, g->counters + 3, s))
      return st;
    g->split_csc = split;
  }
  return DG_OK;
}

}  // namespace dg
