// Internal declarations shared by the translation units of libdgagg (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <string>

#include "dg.h"

// What a handle records.  CSR and CSC arrays are borrowed; the small arrays below are owned.
struct dg_graph {
  int64_t n = 0, nnz = 0;
  const int64_t* rowptr = nullptr;
  const int32_t* colidx = nullptr;
  const float* edge_w = nullptr;

  float* inv_deg = nullptr;      // n: 1/deg(v), 0 for empty rows (mean backward gathers it)
  int32_t* heavy_rows = nullptr; // CSR rows longer than heavy_threshold (forward)
  int32_t* heavy_cols = nullptr; // CSC columns longer than heavy_threshold (backward)
  int32_t* counters = nullptr;   // [0] #heavy rows, [1] #heavy cols, [2] validation flags
  int64_t heavy_cap = 0;         // capacity of each heavy list

  bool transposed = false;
  const int64_t* colptr = nullptr;
  const int32_t* rowidx_T = nullptr;
  const float* w_T = nullptr;
  const int32_t* perm = nullptr;

  int device = 0;
  int sm_count = 148;
  size_t l2_bytes = 0;
  int64_t heavy_threshold = 1024;
  int64_t heavy_built_for = 0;   // threshold the heavy lists were built with
  int64_t slice_features = 0;    // 0 = automatic
  int64_t rows_per_block = 32;
};

namespace dg {

using Graph = ::dg_graph;

// One direction of AP as the kernels see it: out[r] = rs_r * sum_k s_k * X[idx[k]],
// s_k = w[k] * node_scale[idx[k]] (either factor may be absent).
struct ApArgs {
  const int64_t* ptr;         // n+1 segment pointers (rowptr or colptr)
  const int32_t* idx;         // neighbour ids (colidx or rowidx_T)
  const float* w;             // per-edge weight or nullptr
  const float* node_scale;    // per-neighbour factor (1/deg) or nullptr
  const float* X;             // n x F input
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
};

void set_error(const std::string& msg);
dg_status_t cuda_fail(cudaError_t e, const char* what);
void count_launches(int64_t k);

#define DG_CUDA(call)                                          \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return dg::cuda_fail(e__, #call);  \
  } while (0)

// dg_graph.cu
dg_status_t build_degree_info(Graph* g, cudaStream_t s);
dg_status_t build_heavy_list(const int64_t* ptr, int64_t n, int64_t threshold, int32_t* list,
                             int64_t cap, int32_t* count, cudaStream_t s);
dg_status_t validate_csr(Graph* g, cudaStream_t s, int* flags_host);

// dg_transpose.cu
void transpose_sizes(int64_t n, int64_t nnz, bool weighted, size_t* csc_bytes,
                     size_t* scratch_bytes);
dg_status_t transpose_run(Graph* g, void* csc, void* scratch, cudaStream_t s);

// dg_aggregate.cu
dg_status_t aggregate_run(const Graph* g, const ApArgs& a, cudaStream_t s);

}  // namespace dg
