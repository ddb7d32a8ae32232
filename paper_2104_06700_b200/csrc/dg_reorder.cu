// Vertex reordering as a pre-processing step: the same graph with its vertices renamed so that
// the rows the aggregation gathers most often sit next to each other.  The paper makes its
// cache blocks effective by building one CSR per block of source vertices before training
// (Section 3.2, Cache blocking) and shows in Table 3 how much cache reuse a graph offers; on a GPU
// the counterpart is an order of the vertices under which the hot rows of the feature matrix
// form one contiguous, L2-sized range.
//
// The relabelled CSR is defined exactly (it is integer work with one correct result): old vertex
// v becomes new_of_old[v]; new row new_of_old[v] holds the entries of old row v with every source
// u replaced by new_of_old[u], sorted by new source id, duplicates in the order of their old
// positions.  It is computed as two stable radix sorts of the edge positions, by new source id
// and then by new destination id, with the sort of the CSR -> CSC build.
#include <stdlib.h>

#include "dg_internal.cuh"

namespace dg {
namespace {

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
inline unsigned blocks_of(int64_t items) { return (unsigned)((items + 255) / 256); }

struct ReorderLayout {
  // storage (kept by the reordered handle)
  size_t order_off, rowptr_off, colidx_off, pos_off, w_off, storage_bytes;
  // scratch
  size_t k1_off, ka_off, kb_off, va_off, vb_off, hist_off, sums_off, scratch_bytes;
  int64_t items;  // entries per scratch array: max(n, nnz)
};

ReorderLayout reorder_layout(int64_t n, int64_t nnz, bool weighted) {
  ReorderLayout L{};
  size_t o = 0;
  L.order_off = o;  o += align256((size_t)(n > 0 ? n : 1) * 4);
  L.rowptr_off = o; o += align256((size_t)(n + 1) * 8);
  L.colidx_off = o; o += align256((size_t)(nnz > 0 ? nnz : 1) * 4);
  L.pos_off = o;    o += align256((size_t)(nnz > 0 ? nnz : 1) * 4);
  L.w_off = o;      o += weighted ? align256((size_t)(nnz > 0 ? nnz : 1) * 4) : 0;
  L.storage_bytes = o;
  L.items = n > nnz ? n : nnz;
  if (L.items < 1) L.items = 1;
  size_t hist = 0, sums = 0;
  sort_scratch_sizes(L.items, &hist, &sums);
  o = 0;
  const size_t arr = align256((size_t)L.items * 4);
  L.k1_off = o; o += arr;
  L.ka_off = o; o += arr;
  L.kb_off = o; o += arr;
  L.va_off = o; o += arr;
  L.vb_off = o; o += arr;
  L.hist_off = o; o += hist;
  L.sums_off = o; o += sums;
  L.scratch_bytes = o;
  return L;
}

// degree[u] += 1 for every edge with source u (integer atomics: the result does not depend on
// their order)
__global__ void count_sources_kernel(const int32_t* __restrict__ colidx, int64_t nnz,
                                     uint32_t* __restrict__ degree) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < nnz; k += stride)
    atomicAdd(&degree[colidx[k]], 1u);
}

// key[v] = top - degree(v): ascending keys = descending degrees
__global__ void degree_keys_kernel(const int64_t* __restrict__ rowptr,
                                   const uint32_t* __restrict__ source_count, int64_t n,
                                   uint32_t top, uint32_t* __restrict__ key) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n) return;
  const uint32_t d = source_count ? source_count[v] : (uint32_t)(rowptr[v + 1] - rowptr[v]);
  key[v] = top - d;
}

// new_of_old[old_of_new[i]] = i
__global__ void invert_order_kernel(const uint32_t* __restrict__ old_of_new, int64_t n,
                                    int32_t* __restrict__ new_of_old) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) new_of_old[old_of_new[i]] = (int32_t)i;
}

// flags bit 0: an entry outside [0, n); bit 1: a value used twice
__global__ void check_permutation_kernel(const int32_t* __restrict__ order, int64_t n,
                                         uint32_t* __restrict__ seen, int32_t* __restrict__ flags) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n) return;
  const int32_t p = order[v];
  if (p < 0 || p >= n) { atomicOr(flags, 1); return; }
  if (atomicExch(&seen[p], 1u) != 0u) atomicOr(flags, 2);
}

// out[i] = table[index[i]] (index == nullptr: out[i] = table[src[i]] with src = colidx)
__global__ void gather_u32_kernel(const uint32_t* __restrict__ table,
                                  const uint32_t* __restrict__ index, int64_t count,
                                  uint32_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) out[i] = table[index[i]];
}

__global__ void permute_rows_kernel(const int32_t* __restrict__ new_of_old, int64_t n, int32_t F,
                                    const float* __restrict__ in, float* __restrict__ out,
                                    int to_old) {
  const int64_t v = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (v >= n) return;
  const int64_t p = new_of_old[v];
  const float* src = in + (size_t)(to_old ? p : v) * F;
  float* dst = out + (size_t)(to_old ? v : p) * F;
  for (int j = threadIdx.x & 31; j < F; j += 32) dst[j] = src[j];
}

dg_status_t bad(const char* msg) {
  set_error("%s", msg);
  return DG_ERR_INVALID_ARG;
}

}  // namespace
}  // namespace dg

using namespace dg;

extern "C" {

dg_status_t dg_graph_reorder_workspace(dg_graph_t g, size_t* storage_bytes, size_t* scratch_bytes) {
  if (!g) return bad("graph handle is NULL");
  if (!storage_bytes || !scratch_bytes) return bad("size output is NULL");
  const ReorderLayout L = reorder_layout(g->n, g->nnz, g->edge_w != nullptr);
  *storage_bytes = L.storage_bytes;
  *scratch_bytes = L.scratch_bytes;
  return DG_OK;
}

dg_status_t dg_graph_reorder(dg_graph_t g, dg_order_t order, const int32_t* given_new_of_old,
                             void* storage, size_t storage_bytes, void* scratch,
                             size_t scratch_bytes, void* stream, dg_graph_t* out_graph) {
  if (!out_graph) return bad("out_graph is NULL");
  *out_graph = nullptr;
  if (!g) return bad("graph handle is NULL");
  if (order != DG_ORDER_GIVEN && order != DG_ORDER_OUT_DEGREE && order != DG_ORDER_IN_DEGREE)
    return bad("order must be one of the dg_order_t values");
  if (order == DG_ORDER_GIVEN && !given_new_of_old && g->n > 0)
    return bad("DG_ORDER_GIVEN needs the permutation new_of_old");
  if (!storage || !scratch) return bad("storage or scratch is NULL");
  if (((uintptr_t)storage | (uintptr_t)scratch) & 255)
    return bad("storage and scratch must be 256-byte aligned");
  const int64_t n = g->n, nnz = g->nnz;
  const bool weighted = g->edge_w != nullptr;
  const ReorderLayout L = reorder_layout(n, nnz, weighted);
  if (storage_bytes < L.storage_bytes || scratch_bytes < L.scratch_bytes) {
    set_error("workspace smaller than dg_graph_reorder_workspace reports");
    return DG_ERR_WORKSPACE;
  }
  {
    const uintptr_t x = (uintptr_t)storage, y = (uintptr_t)scratch;
    if (x < y + L.scratch_bytes && y < x + L.storage_bytes) return bad("storage and scratch overlap");
  }
  cudaStream_t s = (cudaStream_t)stream;
  char* sb = static_cast<char*>(storage);
  char* wb = static_cast<char*>(scratch);
  int32_t* new_of_old = reinterpret_cast<int32_t*>(sb + L.order_off);
  int64_t* rowptr2 = reinterpret_cast<int64_t*>(sb + L.rowptr_off);
  int32_t* colidx2 = reinterpret_cast<int32_t*>(sb + L.colidx_off);
  uint32_t* pos2 = reinterpret_cast<uint32_t*>(sb + L.pos_off);
  float* w2 = weighted ? reinterpret_cast<float*>(sb + L.w_off) : nullptr;
  uint32_t* k1 = reinterpret_cast<uint32_t*>(wb + L.k1_off);
  uint32_t* keys_buf[2] = {reinterpret_cast<uint32_t*>(wb + L.ka_off),
                           reinterpret_cast<uint32_t*>(wb + L.kb_off)};
  uint32_t* va = reinterpret_cast<uint32_t*>(wb + L.va_off);
  uint32_t* vb = reinterpret_cast<uint32_t*>(wb + L.vb_off);
  uint32_t* hist = reinterpret_cast<uint32_t*>(wb + L.hist_off);
  uint32_t* sums = reinterpret_cast<uint32_t*>(wb + L.sums_off);

  // ---- 1. the order
  if (n > 0 && order == DG_ORDER_GIVEN) {
    int32_t* flags = g->counters + 2;
    DG_CUDA(cudaMemsetAsync(flags, 0, sizeof(int32_t), s));
    DG_CUDA(cudaMemsetAsync(va, 0, (size_t)n * 4, s));
    check_permutation_kernel<<<blocks_of(n), 256, 0, s>>>(given_new_of_old, n, va, flags);
    DG_CUDA(cudaGetLastError());
    count_launches(1);
    int32_t h = 0;
    DG_CUDA(cudaMemcpyAsync(&h, flags, sizeof(h), cudaMemcpyDeviceToHost, s));
    DG_CUDA(cudaStreamSynchronize(s));
    if (h) return bad("new_of_old is not a permutation of 0..n-1");
    DG_CUDA(cudaMemcpyAsync(new_of_old, given_new_of_old, (size_t)n * 4, cudaMemcpyDeviceToDevice, s));
  } else if (n > 0) {
    // stable sort of the vertices by (top - degree): largest degree first, equal degrees by id
    uint32_t* source_count = nullptr;
    if (order == DG_ORDER_OUT_DEGREE) {
      source_count = vb;
      DG_CUDA(cudaMemsetAsync(source_count, 0, (size_t)n * 4, s));
      if (nnz > 0) {
        count_sources_kernel<<<(unsigned)(g->sm_count * 8), 256, 0, s>>>(g->colidx, nnz, source_count);
        DG_CUDA(cudaGetLastError());
        count_launches(1);
      }
    }
    degree_keys_kernel<<<blocks_of(n), 256, 0, s>>>(g->rowptr, source_count, n, (uint32_t)nnz, k1);
    DG_CUDA(cudaGetLastError());
    count_launches(1);
    const uint32_t* sorted = nullptr;
    // values end in va (old_of_new); vb may be reused as the ping-pong buffer: the keys are made
    if (dg_status_t st = sort_pairs(k1, nullptr, n, sort_plan(nnz + 1), keys_buf, va, vb, hist,
                                    sums, &sorted, s))
      return st;
    invert_order_kernel<<<blocks_of(n), 256, 0, s>>>(va, n, new_of_old);
    DG_CUDA(cudaGetLastError());
    count_launches(1);
  }

  // ---- 2. the relabelled CSR
  if (nnz == 0) {
    DG_CUDA(cudaMemsetAsync(rowptr2, 0, (size_t)(n + 1) * 8, s));
  } else {
    const uint32_t* order_u = reinterpret_cast<const uint32_t*>(new_of_old);
    // k1[k] = new id of the source of edge k; positions sorted by it (stable) -> va
    gather_u32_kernel<<<blocks_of(nnz), 256, 0, s>>>(
        order_u, reinterpret_cast<const uint32_t*>(g->colidx), nnz, k1);
    DG_CUDA(cudaGetLastError());
    const uint32_t* sorted = nullptr;
    if (dg_status_t st = sort_pairs(k1, nullptr, nnz, sort_plan(n), keys_buf, va, vb, hist, sums,
                                    &sorted, s))
      return st;
    // keys of the second sort: new id of the destination of every position, in the first sort's order
    if (dg_status_t st = expand_rows(g->rowptr, n, nnz, new_of_old, keys_buf[0], s)) return st;
    gather_u32_kernel<<<blocks_of(nnz), 256, 0, s>>>(keys_buf[0], va, nnz, keys_buf[1]);
    DG_CUDA(cudaGetLastError());
    if (dg_status_t st = sort_pairs(keys_buf[1], va, nnz, sort_plan(n), keys_buf, pos2, vb, hist,
                                    sums, &sorted, s))
      return st;
    if (dg_status_t st = pointers_from_sorted_keys(sorted, nnz, n, rowptr2, s)) return st;
    gather_u32_kernel<<<blocks_of(nnz), 256, 0, s>>>(k1, pos2, nnz,
                                                     reinterpret_cast<uint32_t*>(colidx2));
    DG_CUDA(cudaGetLastError());
    count_launches(3);
    if (weighted) {
      gather_u32_kernel<<<blocks_of(nnz), 256, 0, s>>>(reinterpret_cast<const uint32_t*>(g->edge_w),
                                                       pos2, nnz, reinterpret_cast<uint32_t*>(w2));
      DG_CUDA(cudaGetLastError());
      count_launches(1);
    }
  }
  DG_CUDA(cudaStreamSynchronize(s));

  // ---- 3. a handle of its own over the new arrays
  dg_graph_t h = nullptr;
  if (dg_status_t st = dg_graph_create(n, nnz, rowptr2, colidx2, w2, &h)) return st;
  h->new_of_old = new_of_old;
  h->reorder_pos = reinterpret_cast<const int32_t*>(pos2);
  h->self_loops = g->self_loops;
  h->degree_ordered = order != DG_ORDER_GIVEN;
  *out_graph = h;
  return DG_OK;
}

dg_status_t dg_graph_get_order(dg_graph_t reordered, const int32_t** new_of_old,
                               const int64_t** rowptr, const int32_t** colidx,
                               const float** edge_w, const int32_t** pos) {
  if (!reordered) return bad("graph handle is NULL");
  if (!reordered->new_of_old) return bad("the handle was not made by dg_graph_reorder");
  if (new_of_old) *new_of_old = reordered->new_of_old;
  if (rowptr) *rowptr = reordered->rowptr;
  if (colidx) *colidx = reordered->colidx;
  if (edge_w) *edge_w = reordered->edge_w;
  if (pos) *pos = reordered->reorder_pos;
  return DG_OK;
}

dg_status_t dg_permute_rows(const int32_t* new_of_old, int64_t n, int32_t F, const float* in,
                            float* out, int to_old, void* stream) {
  if (n < 0 || F < 1) return bad("n must be >= 0 and F >= 1");
  if (n == 0) return DG_OK;
  if (!new_of_old || !in || !out) return bad("NULL pointer");
  if (in == out) return bad("dg_permute_rows does not work in place");
  permute_rows_kernel<<<(unsigned)((n + 7) / 8), 256, 0, (cudaStream_t)stream>>>(
      new_of_old, n, F, in, out, to_old);
  DG_CUDA(cudaGetLastError());
  count_launches(1);
  return DG_OK;
}

}  // extern "C"
