// Graph ingest kernels: the lists of heavy segments, split pointers, CSR validation.
// All integer work; nothing here waits on another block.
#include "dg_internal.cuh"

namespace dg {
namespace {

constexpr int kBlock = 256;

// The heavy list holds every segment longer than `threshold`, longest first (in 64 length
// classes, two per power of two): the blocks that walk it take entries x, x + B, x + 2B, ...,
// so starting with the long ones evens out their finishing times.  The order of the list does
// not influence any result: each heavy segment is summed by one block on its own.  The 64
// class counters sit behind the list's `cap` entries.
__device__ __forceinline__ int length_class(int64_t len) {
  const int lg = 63 - __clzll(len);                     // len >= 1
  const int half = lg > 0 ? (int)((len >> (lg - 1)) & 1) : 0;
  const int c = 2 * lg + half;
  return c > 63 ? 63 : c;
}

__global__ void heavy_count_kernel(const int64_t* __restrict__ ptr, int64_t n, int64_t threshold,
                                   int32_t* __restrict__ classes, int32_t* __restrict__ count) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n) return;
  const int64_t len = ptr[v + 1] - ptr[v];
  if (len > threshold) {
    atomicAdd(&classes[length_class(len)], 1);
    atomicAdd(count, 1);
  }
}

// One warp: classes[c] becomes the list position where class c starts (longest class first).
__global__ void heavy_offsets_kernel(int32_t* __restrict__ classes) {
  if (threadIdx.x != 0) return;
  int32_t run = 0;
  for (int c = 63; c >= 0; --c) {
    const int32_t k = classes[c];
    classes[c] = run;
    run += k;
  }
}

__global__ void heavy_fill_kernel(const int64_t* __restrict__ ptr, int64_t n, int64_t threshold,
                                  int32_t* __restrict__ list, int64_t cap,
                                  int32_t* __restrict__ classes) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n) return;
  const int64_t len = ptr[v + 1] - ptr[v];
  if (len > threshold) {
    const int32_t slot = atomicAdd(&classes[length_class(len)], 1);
    if (slot < cap) list[slot] = (int32_t)v;
  }
}

// flags: bit 0 rowptr[0] != 0, bit 1 rowptr decreasing, bit 2 rowptr[n] != nnz,
//        bit 3 colidx out of range
__global__ void validate_rowptr_kernel(const int64_t* __restrict__ rowptr, int64_t n,
                                       int64_t nnz, int32_t* __restrict__ flags) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v > n) return;
  int f = 0;
  if (v == 0 && rowptr[0] != 0) f |= 1;
  if (v < n && rowptr[v + 1] < rowptr[v]) f |= 2;
  if (v == n && rowptr[n] != nnz) f |= 4;
  if (f) atomicOr(flags, f);
}

__global__ void validate_colidx_kernel(const int32_t* __restrict__ colidx, int64_t nnz,
                                       int64_t n, int32_t* __restrict__ flags) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int bad = 0;
  for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < nnz; k += stride) {
    const int32_t u = colidx[k];
    if (u < 0 || u >= n) bad = 1;
  }
  if (bad) atomicOr(flags, 8);
}

// split[b * n + v] for b = 0..kFineBlocks: the first position of segment v whose id is
// >= b * fine_rows, by binary search (the segment must be sorted ascending).
__global__ void split_kernel(const int64_t* __restrict__ ptr, const int32_t* __restrict__ idx,
                             int64_t n, int64_t fine_rows, int32_t* __restrict__ split) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (int64_t)(kFineBlocks + 1) * n) return;
  const int64_t b = t / n, v = t - b * n;
  int64_t lo = ptr[v], hi = ptr[v + 1];
  if (b == 0) { split[t] = (int32_t)lo; return; }
  if (b == kFineBlocks) { split[t] = (int32_t)hi; return; }
  const int64_t bound = b * fine_rows;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(idx + mid) < bound) lo = mid + 1; else hi = mid;
  }
  split[t] = (int32_t)lo;
}

// One warp per segment: sets *flag when two adjacent ids of a segment are out of order.
__global__ void sorted_check_kernel(const int64_t* __restrict__ ptr,
                                    const int32_t* __restrict__ idx, int64_t n,
                                    int32_t* __restrict__ flag) {
  const int64_t v = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (v >= n) return;
  const int lane = threadIdx.x & 31;
  const int64_t lo = ptr[v], hi = ptr[v + 1];
  int bad = 0;
  for (int64_t k = lo + 1 + lane; k < hi; k += 32)
    if (__ldg(idx + k - 1) > __ldg(idx + k)) bad = 1;
  if (bad) atomicOr(flag, 1);
}

inline unsigned blocks_for(int64_t items) { return (unsigned)((items + kBlock - 1) / kBlock); }

}  // namespace

dg_status_t build_heavy_list(const int64_t* ptr, int64_t n, int64_t threshold, int32_t* list,
                             int64_t cap, int32_t* count, cudaStream_t s) {
  int32_t* classes = list + cap;  // 64 counters behind the list (see kHeavyListExtra)
  DG_CUDA(cudaMemsetAsync(count, 0, sizeof(int32_t), s));
  DG_CUDA(cudaMemsetAsync(classes, 0, kHeavyListExtra * sizeof(int32_t), s));
  if (n == 0) return DG_OK;
  heavy_count_kernel<<<blocks_for(n), kBlock, 0, s>>>(ptr, n, threshold, classes, count);
  DG_CUDA(cudaGetLastError());
  heavy_offsets_kernel<<<1, 32, 0, s>>>(classes);
  DG_CUDA(cudaGetLastError());
  heavy_fill_kernel<<<blocks_for(n), kBlock, 0, s>>>(ptr, n, threshold, list, cap, classes);
  DG_CUDA(cudaGetLastError());
  count_launches(3);
  return DG_OK;
}

bool wants_split(int64_t n, int64_t nnz) {
  return n >= 4096 && nnz >= kBlockingMinAvgLen * n &&
         (int64_t)(kFineBlocks + 1) * n < ((int64_t)1 << 40);
}

// Fills the split pointers of one direction and raises *unsorted_flag (device) when a segment
// is not sorted ascending, in which case the pointers must not be used.
dg_status_t build_split(const int64_t* ptr, const int32_t* idx, int64_t n, int64_t fine_rows,
                        int32_t* split, int32_t* unsorted_flag, cudaStream_t s) {
  DG_CUDA(cudaMemsetAsync(unsorted_flag, 0, sizeof(int32_t), s));
  sorted_check_kernel<<<blocks_for(n * 32), kBlock, 0, s>>>(ptr, idx, n, unsorted_flag);
  DG_CUDA(cudaGetLastError());
  split_kernel<<<blocks_for((int64_t)(kFineBlocks + 1) * n), kBlock, 0, s>>>(ptr, idx, n,
                                                                            fine_rows, split);
  DG_CUDA(cudaGetLastError());
  count_launches(2);
  return DG_OK;
}

dg_status_t validate_csr(Graph* g, cudaStream_t s, int* flags_host) {
  int32_t* flags = g->counters + 2;
  DG_CUDA(cudaMemsetAsync(flags, 0, sizeof(int32_t), s));
  validate_rowptr_kernel<<<blocks_for(g->n + 1), kBlock, 0, s>>>(g->rowptr, g->n, g->nnz, flags);
  DG_CUDA(cudaGetLastError());
  count_launches(1);
  // rowptr must be sane before colidx is walked up to nnz: stop here if it is not
  int32_t h = 0;
  DG_CUDA(cudaMemcpyAsync(&h, flags, sizeof(h), cudaMemcpyDeviceToHost, s));
  DG_CUDA(cudaStreamSynchronize(s));
  if (h == 0 && g->nnz > 0) {
    const unsigned grid = (unsigned)(g->sm_count * 8);
    validate_colidx_kernel<<<grid, kBlock, 0, s>>>(g->colidx, g->nnz, g->n, flags);
    DG_CUDA(cudaGetLastError());
    count_launches(1);
    DG_CUDA(cudaMemcpyAsync(&h, flags, sizeof(h), cudaMemcpyDeviceToHost, s));
    DG_CUDA(cudaStreamSynchronize(s));
  }
  *flags_host = h;
  return DG_OK;
}

}  // namespace dg
