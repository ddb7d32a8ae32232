// Internal declarations shared by the translation units of libdgagg (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "dg.h"

// What a handle records.  CSR and CSC arrays are borrowed; the small arrays below are owned.
struct dg_graph {
  int64_t n = 0, nnz = 0;
  const int64_t* rowptr = nullptr;
  const int32_t* colidx = nullptr;
  const float* edge_w = nullptr;

  int32_t* heavy_rows = nullptr; // CSR rows longer than heavy_threshold (forward)
  int32_t* heavy_cols = nullptr; // CSC columns longer than heavy_threshold (backward)
  int32_t* counters = nullptr;   // [0] #heavy rows, [1] #heavy cols, [2] validation flags
  int64_t heavy_cap = 0;         // capacity of each heavy list (kHeavyListExtra more ints are allocated)

  // Source blocking: the neighbour ids are cut into kFineBlocks ranges of fine_rows ids;
  // split[b * n + v] is the first position of segment v whose neighbour id is >= b * fine_rows
  // (entry kFineBlocks is the segment end).  Built only for graphs whose rows are long and
  // sorted; nullptr otherwise.  split_csr is owned, split_csc lives in the caller's CSC storage.
  int32_t* split_csr = nullptr;
  int32_t* split_csc = nullptr;
  int64_t fine_rows = 0;

  // dg_aggregate_host: helper streams (upload, download) and events, created on first use
  bool aux_ready = false;
  cudaStream_t aux_stream[2] = {nullptr, nullptr};
  cudaEvent_t* aux_events = nullptr;  // malloc'ed pool, aux_event_count entries
  size_t aux_event_count = 0;

  // Whether a CSR row / CSC column of 2^15 entries or more exists (1), does not (0), or is not
  // known yet (-1: the count of the last transposition is still on its way to the host).  Such
  // graphs run the kernels compiled with the two-level sum of the block-per-row path.
  int long_rows = 1;
  int long_cols = -1;
  int32_t* long_cols_host = nullptr;     // pinned; written by a copy enqueued after a transposition
  cudaEvent_t long_cols_ready = nullptr; // recorded behind that copy

  bool transposed = false;
  const int64_t* colptr = nullptr;
  const int32_t* rowidx_T = nullptr;
  const float* w_T = nullptr;
  const int32_t* perm = nullptr;
  const float* mean_scale_T = nullptr;  // w_T[q] / (deg(rowidx_T[q]) + self_loops): edge factor of the mean's backward
  int64_t self_loops = 0;        // 1: every vertex is its own in-neighbour with weight 1
  int64_t self_loops_in_csc = 0; // value mean_scale_T was built with

  // set on a handle made by dg_graph_reorder: arrays inside the caller's reorder storage
  const int32_t* new_of_old = nullptr;   // n: new id of every old vertex
  const int32_t* reorder_pos = nullptr;  // nnz: old CSR position of every new position
  bool degree_ordered = false;           // made by dg_graph_reorder with a hub-first order

  int device = 0;
  int sm_count = 148;
  size_t l2_bytes = 0;
  int64_t heavy_threshold = 1024;
  int64_t heavy_built_for = 0;   // threshold the heavy lists were built with
  int64_t slice_features = 0;    // 0 = automatic
  int64_t rows_per_block = 0;    // 0 = from the average row length
  int64_t heavy_blocks_per_sm = 0;  // blocks per SM that walk the heavy list; 0 = all resident ones
  int64_t l2_budget_bytes = 0;   // bytes of the gathered matrix one launch may keep L2-resident
  int64_t source_blocks = 0;     // 0 = automatic, else 1, 2, 4, 8 or 16
};

namespace dg {

using Graph = ::dg_graph;

constexpr int kHeavyListExtra = 64;      // counters of the length classes, stored behind a heavy list
constexpr int kFineBlocks = 16;          // finest cut of the neighbour ids for source blocking
constexpr int64_t kBlockingMinAvgLen = 64;  // split pointers are built when nnz >= 64 n

// One direction of AP as the kernels see it: out[r] = rs_r * sum_k s_k * X[idx[k]],
// s_k = w[k] (1 when w is absent).
struct ApArgs {
  const int64_t* ptr;         // n+1 segment pointers (rowptr or colptr)
  const int32_t* idx;         // neighbour ids (colidx or rowidx_T)
  const float* w;             // per-edge weight or nullptr
  const void* X;              // n x F input: fp32, or bf16 when x_bf16 is set
  int32_t x_bf16;
  float* Y;                   // n x F output
  const int32_t* heavy_list;  // segments longer than heavy_threshold
  const int32_t* heavy_count; // device scalar
  int32_t heavy_cap;          // capacity of heavy_list (the count is clamped to it)
  int64_t n;
  int32_t F;
  int32_t slice_f;            // features per slice (multiple of the vector width)
  int32_t mean_rows;          // 1: multiply the finished row by 1/(segment length)
  int32_t heavy_threshold;
  int32_t rows_per_warp;     // consecutive light segments per warp (1..31)
  const int32_t* seg_lo;      // source-blocked pass: first and one-past-last position of every
  const int32_t* seg_hi;      //   segment's piece (n entries each); nullptr = whole segments
  int32_t accumulate;         // source-blocked pass after the first: add to what Y holds
  int32_t long_segments;      // host side only: a segment of 2^15 entries or more may exist
  int32_t full_registers;     // host side only: run the scaled kernels without the register cap
};

// Implicit self loops (every vertex its own neighbour with weight 1): row r also receives
// ss_r * X[r], once (not in accumulating passes).  self_ptr is the CSR row pointer, in both
// directions (the in-degree belongs to the vertex, not to the segment the kernel walks);
// nullptr = no self loops.  self_mean: ss_r = 1 / (in-degree(r) + 1) instead of 1, and
// mean_rows scales by the same factor instead of 1 / (segment length).  A parameter of its own,
// passed only to the kernels compiled for self loops.
struct SelfArgs {
  const int64_t* self_ptr;
  int32_t self_mean;
};

// One launch of the aggregation kernels in the shape aggregate_run chose (dg_aggregate.cu,
// dg_aggregate_self.cu).
dg_status_t launch_plain(const dg_graph* g, const ApArgs& a, int vec, int slices, cudaStream_t s);
dg_status_t launch_with_self_loops(const dg_graph* g, const ApArgs& a, const SelfArgs& sa, int vec,
                                   int slices, cudaStream_t s);
// the same with the two-level sum for long segments (dg_aggregate_fold.cu, dg_aggregate_self_fold.cu)
dg_status_t launch_plain_fold(const dg_graph* g, const ApArgs& a, int vec, int slices,
                              cudaStream_t s);
dg_status_t launch_with_self_loops_fold(const dg_graph* g, const ApArgs& a, const SelfArgs& sa,
                                        int vec, int slices, cudaStream_t s);

// Records the calling thread's last error message (printf-style, truncated to a fixed buffer:
// nothing on an error path allocates, so nothing can throw across the C boundary).
void set_error(const char* fmt, ...) __attribute__((format(printf, 1, 2)));
dg_status_t cuda_fail(cudaError_t e, const char* what);
void count_launches(int64_t k);

#define DG_CUDA(call)                                          \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return dg::cuda_fail(e__, #call);  \
  } while (0)

// dg_graph.cu
dg_status_t build_heavy_list(const int64_t* ptr, int64_t n, int64_t threshold, int32_t* list,
                             int64_t cap, int32_t* count, cudaStream_t s);
dg_status_t validate_csr(Graph* g, cudaStream_t s, int* flags_host);
bool wants_split(int64_t n, int64_t nnz);
dg_status_t build_split(const int64_t* ptr, const int32_t* idx, int64_t n, int64_t fine_rows,
                        int32_t* split, int32_t* unsorted_flag, cudaStream_t s);

// dg_transpose.cu
void transpose_sizes(int64_t n, int64_t nnz, bool weighted, size_t* csc_bytes,
                     size_t* scratch_bytes);
dg_status_t transpose_run(Graph* g, void* csc, void* scratch, cudaStream_t s);
dg_status_t refresh_csc_weights(Graph* g, cudaStream_t s);
// dg_api.cu: what follows every transposition (heavy columns, the long-column count on its way)
dg_status_t finish_transpose(Graph* g, cudaStream_t s);
// the stable radix sort behind it, for other pre-processing steps (see dg_transpose.cu)
struct SortPlan { int digit_bits; int passes; };
SortPlan sort_plan(int64_t key_range);
void sort_scratch_sizes(int64_t count, size_t* hist_bytes, size_t* sums_bytes);
dg_status_t sort_pairs(const uint32_t* keys_in, const uint32_t* vals_in, int64_t count, SortPlan plan,
                       uint32_t* const keys_buf[2], uint32_t* vals_final, uint32_t* vals_tmp,
                       uint32_t* hist, uint32_t* sums, const uint32_t** sorted_keys,
                       cudaStream_t s);
dg_status_t pointers_from_sorted_keys(const uint32_t* sorted, int64_t count, int64_t n,
                                      int64_t* ptr, cudaStream_t s);
dg_status_t expand_rows(const int64_t* rowptr, int64_t n, int64_t nnz, const int32_t* map,
                        uint32_t* out, cudaStream_t s);

// dg_aggregate.cu
dg_status_t aggregate_run(const Graph* g, const ApArgs& a, const SelfArgs& sa, const int32_t* split,
                          cudaStream_t s);
// sum_k w_k X[idx[k]] over the CSR rows or the CSC columns with those kernels (dg_api.cu); w in
// the order of that direction or nullptr, no self loops.
dg_status_t aggregate_sum(Graph* g, bool over_csc, const float* w, const float* X, int32_t F,
                          float* Y, cudaStream_t s);

}  // namespace dg
