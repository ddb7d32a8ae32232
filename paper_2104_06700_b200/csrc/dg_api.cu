// The C ABI of libdgagg: argument checks, handle bookkeeping and kernel dispatch.
// Declarations and the meaning of every argument are in include/dg.h.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "dg_internal.cuh"

namespace dg {

static thread_local char g_last_error[512] = "";
static std::atomic<int64_t> g_launches{0};

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
  va_end(ap);
}

dg_status_t cuda_fail(cudaError_t e, const char* what) {
  set_error("%s: %s", what, cudaGetErrorString(e));
  return DG_ERR_CUDA;
}

void count_launches(int64_t k) { g_launches.fetch_add(k, std::memory_order_relaxed); }

static dg_status_t invalid(const char* msg) {
  set_error("%s", msg);
  return DG_ERR_INVALID_ARG;
}

// [a, a + a_bytes) and [b, b + b_bytes) share a byte
static bool overlaps(const void* a, size_t a_bytes, const void* b, size_t b_bytes) {
  const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
  return x < y + b_bytes && y < x + a_bytes;
}

static dg_status_t free_owned(Graph* g) {
  if (g->heavy_rows) cudaFree(g->heavy_rows);
  if (g->heavy_cols) cudaFree(g->heavy_cols);
  if (g->counters) cudaFree(g->counters);
  if (g->split_csr) cudaFree(g->split_csr);
  g->split_csr = nullptr;
  if (g->long_cols_host) cudaFreeHost(g->long_cols_host);
  g->long_cols_host = nullptr;
  if (g->long_cols_ready) cudaEventDestroy(g->long_cols_ready);
  g->long_cols_ready = nullptr;

  for (size_t i = 0; i < g->aux_event_count; ++i) cudaEventDestroy(g->aux_events[i]);
  free(g->aux_events);
  g->aux_events = nullptr;
  g->aux_event_count = 0;
  if (g->aux_ready) {
    for (int i = 0; i < 2; ++i) cudaStreamDestroy(g->aux_stream[i]);
    g->aux_ready = false;
  }
  g->heavy_rows = g->heavy_cols = g->counters = nullptr;
  return DG_OK;
}

// (Re)builds the heavy lists for the current threshold; called at create, after a transpose
// and after the threshold changes.
static dg_status_t refresh_heavy(Graph* g, bool csr, bool csc, cudaStream_t s) {
  if (csr)
    if (dg_status_t st = build_heavy_list(g->rowptr, g->n, g->heavy_threshold, g->heavy_rows,
                                          g->heavy_cap, g->counters + 0, s))
      return st;
  if (csc && g->transposed)
    if (dg_status_t st = build_heavy_list(g->colptr, g->n, g->heavy_threshold, g->heavy_cols,
                                          g->heavy_cap, g->counters + 1, s))
      return st;
  return DG_OK;
}

// Index of the length class of the heavy-list builder at which segments of 2^15 entries start;
// after the list is filled, counter [class] holds the number of segments in that class or above.
constexpr int kLongClass = 30;

// Heavy columns of a fresh CSC, and the number of long ones sent to the host behind them (read
// by the first backward pass that finds the copy finished; until then the columns count as long).
dg_status_t finish_transpose(Graph* g, cudaStream_t s) {
  if (dg_status_t st = refresh_heavy(g, false, true, s)) return st;
  g->long_cols = -1;
  DG_CUDA(cudaMemcpyAsync(g->long_cols_host, g->heavy_cols + g->heavy_cap + kLongClass,
                          sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  DG_CUDA(cudaEventRecord(g->long_cols_ready, s));
  return DG_OK;
}

// Synchronous: the heavy rows have just been (re)built on the default stream.
static dg_status_t count_long_rows(Graph* g) {
  int32_t longs = 0;
  DG_CUDA(cudaMemcpy(&longs, g->heavy_rows + g->heavy_cap + kLongClass, sizeof(longs),
                     cudaMemcpyDeviceToHost));
  g->long_rows = longs > 0 ? 1 : 0;
  return DG_OK;
}

// Graphs on which the scaled kernels run better without their register cap: renamed hub-first,
// or fewer than 32 edges per vertex (see launch_variant).
static int full_registers(const Graph* g) {
  return g->degree_ordered || (g->n > 0 && g->nnz < 32 * g->n);
}

static int long_columns(Graph* g) {
  if (g->long_cols < 0) {
    if (cudaEventQuery(g->long_cols_ready) == cudaSuccess)
      g->long_cols = *g->long_cols_host > 0 ? 1 : 0;
    else
      (void)cudaGetLastError();  // "not ready" must not be mistaken for a failed launch later
  }
  return g->long_cols != 0;
}

// rows_per_block is rounded up to a whole number of rows per warp (8 warps per block).  0 picks
// about 1024 edges per warp, between 4 and 31 rows: short rows want long-lived blocks (less
// block turnover), long rows want many blocks.
static int32_t rows_per_warp(const Graph* g) {
  int64_t r;
  if (g->rows_per_block > 0) {
    r = (g->rows_per_block + 7) / 8;
  } else {
    const double avg = g->n > 0 ? (double)g->nnz / (double)g->n : 1.0;
    r = (int64_t)(1024.0 / (avg > 1.0 ? avg : 1.0));
    if (r < 4) r = 4;
    // small graphs: keep at least 64 warps' worth of row runs per SM
    const int64_t fill = g->n / ((int64_t)g->sm_count * 64);
    if (r > fill) r = fill;
  }
  return (int32_t)(r < 1 ? 1 : (r > 31 ? 31 : r));
}

static dg_status_t check_features(const Graph* g, const void* in, size_t in_elem_bytes, float* out,
                                  int32_t F, dg_op_t op) {
  if (!g) return invalid("graph handle is NULL");
  if (F < 1) return invalid("F must be >= 1");
  if (F > (1 << 20)) {
    set_error("F must be at most 2^20");
    return DG_ERR_UNSUPPORTED;
  }
  if (op != DG_OP_SUM && op != DG_OP_MEAN) return invalid("op must be DG_OP_SUM or DG_OP_MEAN");
  if (g->n > 0) {
    if (!in || !out) return invalid("feature matrix pointer is NULL");
    const size_t elems = (size_t)g->n * (size_t)F;
    const uintptr_t x = (uintptr_t)in, y = (uintptr_t)out;
    if (x < y + elems * sizeof(float) && y < x + elems * in_elem_bytes)
      return invalid("input and output feature matrices overlap");
  }
  return DG_OK;
}

// Forward / backward AP for either storage type of the gathered matrix.
static dg_status_t run_forward(Graph* g, const void* H, bool bf16, int32_t F, dg_op_t op,
                               float* out, void* stream) {
  if (dg_status_t st = check_features(g, H, bf16 ? 2 : 4, out, F, op)) return st;
  ApArgs a{};
  a.ptr = g->rowptr;
  a.idx = g->colidx;
  a.w = g->edge_w;
  a.X = H;
  a.x_bf16 = bf16;
  a.Y = out;
  a.heavy_list = g->heavy_rows;
  a.heavy_count = g->counters + 0;
  a.heavy_cap = (int32_t)g->heavy_cap;
  a.n = g->n;
  a.F = F;
  a.mean_rows = op == DG_OP_MEAN;
  a.heavy_threshold = (int32_t)g->heavy_threshold;
  a.rows_per_warp = rows_per_warp(g);
  a.long_segments = g->long_rows;
  a.full_registers = full_registers(g);
  const SelfArgs sa{g->self_loops ? g->rowptr : nullptr, op == DG_OP_MEAN};
  return aggregate_run(g, a, sa, g->split_csr, (cudaStream_t)stream);
}

static dg_status_t run_backward(Graph* g, const void* dOut, bool bf16, int32_t F, dg_op_t op,
                                float* dH, void* stream) {
  if (dg_status_t st = check_features(g, dOut, bf16 ? 2 : 4, dH, F, op)) return st;
  if (!g->transposed) {
    set_error("the backward pass needs dg_graph_transpose first");
    return DG_ERR_NOT_TRANSPOSED;
  }
  if (op == DG_OP_MEAN && g->self_loops != g->self_loops_in_csc) {
    set_error("self_loops was changed after dg_graph_transpose: transpose again");
    return DG_ERR_NOT_TRANSPOSED;
  }
  ApArgs a{};
  a.ptr = g->colptr;
  a.idx = g->rowidx_T;
  a.w = op == DG_OP_MEAN ? g->mean_scale_T : g->w_T;
  a.X = dOut;
  a.x_bf16 = bf16;
  a.Y = dH;
  a.heavy_list = g->heavy_cols;
  a.heavy_count = g->counters + 1;
  a.heavy_cap = (int32_t)g->heavy_cap;
  a.n = g->n;
  a.F = F;
  a.mean_rows = 0;
  a.heavy_threshold = (int32_t)g->heavy_threshold;
  a.rows_per_warp = rows_per_warp(g);
  a.long_segments = long_columns(g);
  a.full_registers = full_registers(g);
  const SelfArgs sa{g->self_loops ? g->rowptr : nullptr, op == DG_OP_MEAN};
  return aggregate_run(g, a, sa, g->split_csc, (cudaStream_t)stream);
}

// sum_k w_k X[idx[k]] over the CSR rows (or the CSC columns) with the sum / mean kernels, for
// the operator pairs of the general entry points that are exactly this.  w is in the order of
// the direction walked, or nullptr; the handle's own weights and its "self_loops" attribute play
// no part.
dg_status_t aggregate_sum(Graph* g, bool over_csc, const float* w, const float* X, int32_t F,
                          float* Y, cudaStream_t s) {
  ApArgs a{};
  a.ptr = over_csc ? g->colptr : g->rowptr;
  a.idx = over_csc ? g->rowidx_T : g->colidx;
  a.w = w;
  a.X = X;
  a.Y = Y;
  a.heavy_list = over_csc ? g->heavy_cols : g->heavy_rows;
  a.heavy_count = g->counters + (over_csc ? 1 : 0);
  a.heavy_cap = (int32_t)g->heavy_cap;
  a.n = g->n;
  a.F = F;
  a.heavy_threshold = (int32_t)g->heavy_threshold;
  a.rows_per_warp = rows_per_warp(g);
  a.long_segments = over_csc ? long_columns(g) : g->long_rows;
  a.full_registers = full_registers(g);
  return aggregate_run(g, a, SelfArgs{nullptr, 0}, over_csc ? g->split_csc : g->split_csr, s);
}

static dg_status_t malformed(int flags) {
  set_error("malformed CSR:%s%s%s%s", (flags & 1) ? " rowptr[0] != 0;" : "",
            (flags & 2) ? " rowptr decreases;" : "", (flags & 4) ? " rowptr[n] != nnz;" : "",
            (flags & 8) ? " colidx outside [0, n);" : "");
  return DG_ERR_INVALID_GRAPH;
}

}  // namespace dg

using namespace dg;

extern "C" {

dg_status_t dg_graph_create(int64_t n, int64_t nnz, const int64_t* rowptr,
                            const int32_t* colidx, const float* edge_w, dg_graph_t* out_graph) {
  if (!out_graph) return invalid("out_graph is NULL");
  *out_graph = nullptr;
  if (n < 0 || nnz < 0) return invalid("n and nnz must be >= 0");
  if (n >= ((int64_t)1 << 31) || nnz >= ((int64_t)1 << 31)) {
    set_error("n and nnz must be below 2^31");
    return DG_ERR_UNSUPPORTED;
  }
  if (!rowptr) return invalid("rowptr is NULL");
  if (nnz > 0 && !colidx) return invalid("colidx is NULL");
  if (nnz > 0 && n == 0) return invalid("edges without vertices");

  Graph* g = new (std::nothrow) Graph();
  if (!g) return invalid("out of host memory");
  g->n = n;
  g->nnz = nnz;
  g->rowptr = rowptr;
  g->colidx = colidx;
  g->edge_w = edge_w;
  cudaError_t e = cudaGetDevice(&g->device);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, g->device);
  if (e != cudaSuccess) { delete g; return cuda_fail(e, "cudaGetDeviceProperties"); }
  g->sm_count = prop.multiProcessorCount;
  g->l2_bytes = (size_t)prop.l2CacheSize;
  g->l2_budget_bytes = (int64_t)(g->l2_bytes * 19 / 40);  // 60 of 126 MB measured best on B200
  g->fine_rows = (n + kFineBlocks - 1) / kFineBlocks;
  if (g->fine_rows < 1) g->fine_rows = 1;
  g->heavy_cap = nnz / 64 + 1;  // enough for any threshold >= 64
  if (g->heavy_cap > n) g->heavy_cap = n > 0 ? n : 1;

  // The caller may have produced the arrays on any stream: wait for the device once, then
  // everything below runs on the default stream and is waited for before the call returns.
  e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMalloc(&g->heavy_rows, (size_t)(g->heavy_cap + kHeavyListExtra) * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&g->heavy_cols, (size_t)(g->heavy_cap + kHeavyListExtra) * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&g->counters, 4 * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaHostAlloc(&g->long_cols_host, sizeof(int32_t), cudaHostAllocDefault);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&g->long_cols_ready, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMemset(g->counters, 0, 4 * sizeof(int32_t));
  if (e == cudaSuccess && wants_split(n, nnz))
    e = cudaMalloc(&g->split_csr, (size_t)(kFineBlocks + 1) * (size_t)n * sizeof(int32_t));
  if (e != cudaSuccess) { free_owned(g); delete g; return cuda_fail(e, "cudaMalloc (graph metadata)"); }

  // The kernels gather X[colidx[k]] without a range check, so a malformed CSR must never reach
  // them: one streaming pass over rowptr and colidx here (about a millisecond per 10^9 edges).
  int flags = 0;
  dg_status_t st = validate_csr(g, 0, &flags);
  if (st == DG_OK && flags) st = malformed(flags);
  if (st == DG_OK) st = refresh_heavy(g, true, false, 0);
  if (st == DG_OK && g->split_csr)
    st = build_split(rowptr, colidx, n, g->fine_rows, g->split_csr, g->counters + 3, 0);
  if (st == DG_OK) st = count_long_rows(g);
  if (st == DG_OK) {
    int32_t unsorted = 0;
    e = cudaMemcpy(&unsorted, g->counters + 3, sizeof(unsorted), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) st = cuda_fail(e, "cudaDeviceSynchronize (graph create)");
    if (st == DG_OK && unsorted && g->split_csr) {  // rows not sorted: no source blocking
      cudaFree(g->split_csr);
      g->split_csr = nullptr;
    }
  }
  if (st != DG_OK) { free_owned(g); delete g; return st; }
  *out_graph = g;
  return DG_OK;
}

dg_status_t dg_graph_destroy(dg_graph_t g) {
  if (!g) return DG_OK;
  free_owned(g);
  delete g;
  return DG_OK;
}

dg_status_t dg_graph_validate(dg_graph_t g, void* stream) {
  if (!g) return invalid("graph handle is NULL");
  int flags = 0;
  if (dg_status_t st = validate_csr(g, (cudaStream_t)stream, &flags)) return st;
  return flags ? malformed(flags) : DG_OK;
}

dg_status_t dg_graph_transpose_workspace(dg_graph_t g, size_t* csc_bytes, size_t* scratch_bytes) {
  if (!g) return invalid("graph handle is NULL");
  if (!csc_bytes || !scratch_bytes) return invalid("size output is NULL");
  transpose_sizes(g->n, g->nnz, g->edge_w != nullptr, csc_bytes, scratch_bytes);
  return DG_OK;
}

dg_status_t dg_graph_transpose(dg_graph_t g, void* csc_storage, size_t csc_bytes, void* scratch,
                               size_t scratch_bytes, void* stream) {
  if (!g) return invalid("graph handle is NULL");
  if (!csc_storage || !scratch) return invalid("csc_storage or scratch is NULL");
  if (((uintptr_t)csc_storage | (uintptr_t)scratch) & 255)
    return invalid("csc_storage and scratch must be 256-byte aligned");
  size_t need_csc, need_scratch;
  transpose_sizes(g->n, g->nnz, g->edge_w != nullptr, &need_csc, &need_scratch);
  if (csc_bytes < need_csc || scratch_bytes < need_scratch) {
    set_error("workspace smaller than dg_graph_transpose_workspace reports");
    return DG_ERR_WORKSPACE;
  }
  if (overlaps(csc_storage, need_csc, scratch, need_scratch))
    return invalid("csc_storage and scratch overlap");
  g->transposed = false;
  if (dg_status_t st = transpose_run(g, csc_storage, scratch, (cudaStream_t)stream)) return st;
  g->transposed = true;
  return finish_transpose(g, (cudaStream_t)stream);
}

dg_status_t dg_graph_update_weights(dg_graph_t g, void* stream) {
  if (!g) return invalid("graph handle is NULL");
  if (!g->edge_w) return invalid("the graph has no edge weights");
  if (!g->transposed) return DG_OK;  // the CSR is read in place: nothing to refresh
  return refresh_csc_weights(g, (cudaStream_t)stream);
}

dg_status_t dg_graph_get_csc(dg_graph_t g, const int64_t** colptr, const int32_t** rowidx_T,
                             const float** w_T, const int32_t** perm) {
  if (!g) return invalid("graph handle is NULL");
  if (!g->transposed) {
    set_error("dg_graph_transpose has not been called");
    return DG_ERR_NOT_TRANSPOSED;
  }
  if (colptr) *colptr = g->colptr;
  if (rowidx_T) *rowidx_T = g->rowidx_T;
  if (w_T) *w_T = g->w_T;
  if (perm) *perm = g->perm;
  return DG_OK;
}

dg_status_t dg_aggregate_fwd(dg_graph_t g, const float* H, int32_t F, dg_op_t op, float* out,
                             void* stream) {
  return run_forward(g, H, false, F, op, out, stream);
}

dg_status_t dg_aggregate_bwd(dg_graph_t g, const float* dOut, int32_t F, dg_op_t op, float* dH,
                             void* stream) {
  return run_backward(g, dOut, false, F, op, dH, stream);
}

dg_status_t dg_aggregate_fwd_bf16(dg_graph_t g, const uint16_t* H, int32_t F, dg_op_t op,
                                  float* out, void* stream) {
  return run_forward(g, H, true, F, op, out, stream);
}

dg_status_t dg_aggregate_bwd_bf16(dg_graph_t g, const uint16_t* dOut, int32_t F, dg_op_t op,
                                  float* dH, void* stream) {
  return run_backward(g, dOut, true, F, op, dH, stream);
}

size_t dg_aggregate_host_workspace(dg_graph_t g, int32_t F) {
  if (!g || F < 1) return 0;
  const size_t mat = (((size_t)g->n * (size_t)F * sizeof(float)) + 255) & ~(size_t)255;
  return 4 * (mat > 0 ? mat : 256);
}

// Helper streams (upload, download) and a pool of events per handle, created on first use.
static dg_status_t host_pipeline(Graph* g, size_t events) {
  if (!g->aux_ready) {
    for (int i = 0; i < 2; ++i)
      DG_CUDA(cudaStreamCreateWithFlags(&g->aux_stream[i], cudaStreamNonBlocking));
    g->aux_ready = true;
  }
  if (g->aux_event_count < events) {
    cudaEvent_t* grown = (cudaEvent_t*)realloc(g->aux_events, events * sizeof(cudaEvent_t));
    if (!grown) {
      set_error("out of host memory (event pool)");
      return DG_ERR_INVALID_ARG;
    }
    g->aux_events = grown;
    while (g->aux_event_count < events) {
      DG_CUDA(cudaEventCreateWithFlags(&g->aux_events[g->aux_event_count], cudaEventDisableTiming));
      ++g->aux_event_count;
    }
  }
  return DG_OK;
}

// The feature columns are independent of each other in AP, so the host matrices travel in column
// chunks: chunk c of H is uploaded (a strided copy into a compact n x w matrix) while chunk c-1 is
// being aggregated and the result of chunk c-2 is on its way back; then the same for dOut.  PCIe
// carries both directions at once, so a call costs about max(kernel time, copy time) instead of
// their sum.  Two input and two output chunk buffers alternate.
dg_status_t dg_aggregate_host(dg_graph_t g, const float* H_host, const float* dOut_host,
                              int32_t F, dg_op_t op, float* out_host, float* dH_host,
                              void* device_ws, size_t device_ws_bytes, void* stream) {
  if (!g) return invalid("graph handle is NULL");
  if (F < 1) return invalid("F must be >= 1");
  if (!H_host || !out_host) return invalid("H_host or out_host is NULL");
  if ((dOut_host == nullptr) != (dH_host == nullptr))
    return invalid("dOut_host and dH_host must both be given or both be NULL");
  if (!device_ws || ((uintptr_t)device_ws & 255)) return invalid("device_ws is NULL or misaligned");
  if (device_ws_bytes < dg_aggregate_host_workspace(g, F)) {
    set_error("device_ws smaller than dg_aggregate_host_workspace reports");
    return DG_ERR_WORKSPACE;
  }
  if (dOut_host && !g->transposed) {
    set_error("the backward pass needs dg_graph_transpose first");
    return DG_ERR_NOT_TRANSPOSED;
  }
  if (g->n == 0) return DG_OK;
  // chunk width: 128 columns (one 512-byte row slice) once the matrix is wider than 256 columns
  const int32_t W = F > 256 ? 128 : F;
  const int chunks = (F + W - 1) / W;
  const int tasks = chunks * (dOut_host ? 2 : 1);
  if (dg_status_t st = host_pipeline(g, 1 + 3 * (size_t)tasks)) return st;
  cudaStream_t s = (cudaStream_t)stream;
  cudaStream_t up = g->aux_stream[0], down = g->aux_stream[1];
  cudaEvent_t* ev = g->aux_events;
  cudaEvent_t start = ev[0];
  auto uploaded = [&](int t) { return ev[1 + 3 * t]; };
  auto computed = [&](int t) { return ev[2 + 3 * t]; };
  auto downloaded = [&](int t) { return ev[3 + 3 * t]; };

  const size_t buf = (((size_t)g->n * (size_t)W * sizeof(float)) + 255) & ~(size_t)255;
  char* ws = static_cast<char*>(device_ws);
  float* d_in[2] = {reinterpret_cast<float*>(ws), reinterpret_cast<float*>(ws + buf)};
  float* d_out[2] = {reinterpret_cast<float*>(ws + 2 * buf), reinterpret_cast<float*>(ws + 3 * buf)};
  const size_t host_pitch = (size_t)F * sizeof(float);

  // everything queued on `stream` so far (an earlier call may still use the workspace) comes first
  DG_CUDA(cudaEventRecord(start, s));
  DG_CUDA(cudaStreamWaitEvent(up, start, 0));
  DG_CUDA(cudaStreamWaitEvent(down, start, 0));
  for (int t = 0; t < tasks; ++t) {
    const bool bwd = t >= chunks;
    const int c = bwd ? t - chunks : t;
    const int32_t w = (c + 1) * W <= F ? W : F - c * W;
    const float* src = (bwd ? dOut_host : H_host) + (size_t)c * W;
    float* dst = (bwd ? dH_host : out_host) + (size_t)c * W;
    float* in = d_in[t & 1];
    float* out = d_out[t & 1];
    // upload: the input buffer is free once the kernels of task t-2 have read it
    if (t >= 2) DG_CUDA(cudaStreamWaitEvent(up, computed(t - 2), 0));
    DG_CUDA(cudaMemcpy2DAsync(in, (size_t)w * sizeof(float), src, host_pitch,
                              (size_t)w * sizeof(float), (size_t)g->n, cudaMemcpyHostToDevice, up));
    DG_CUDA(cudaEventRecord(uploaded(t), up));
    // compute: needs the upload, and the output buffer back from the download of task t-2
    DG_CUDA(cudaStreamWaitEvent(s, uploaded(t), 0));
    if (t >= 2) DG_CUDA(cudaStreamWaitEvent(s, downloaded(t - 2), 0));
    if (dg_status_t st = bwd ? dg_aggregate_bwd(g, in, w, op, out, stream)
                             : dg_aggregate_fwd(g, in, w, op, out, stream))
      return st;
    DG_CUDA(cudaEventRecord(computed(t), s));
    // download
    DG_CUDA(cudaStreamWaitEvent(down, computed(t), 0));
    DG_CUDA(cudaMemcpy2DAsync(dst, host_pitch, out, (size_t)w * sizeof(float),
                              (size_t)w * sizeof(float), (size_t)g->n, cudaMemcpyDeviceToHost, down));
    DG_CUDA(cudaEventRecord(downloaded(t), down));
  }
  // `stream` finishing means every copy has finished
  DG_CUDA(cudaStreamWaitEvent(s, downloaded(tasks - 1), 0));
  if (tasks >= 2) DG_CUDA(cudaStreamWaitEvent(s, downloaded(tasks - 2), 0));
  return DG_OK;
}

dg_status_t dg_graph_set_param(dg_graph_t g, const char* name, int64_t value) {
  if (!g || !name) return invalid("graph handle or name is NULL");
  if (!strcmp(name, "heavy_threshold")) {
    if (value < 64 || value > (1 << 30)) return invalid("heavy_threshold must be in [64, 2^30]");
    // the lists may be in use, or being built, on any stream: wait for the device on both sides
    DG_CUDA(cudaDeviceSynchronize());
    g->heavy_threshold = value;
    if (dg_status_t st = refresh_heavy(g, true, false, 0)) return st;
    if (dg_status_t st = count_long_rows(g)) return st;
    if (g->transposed)
      if (dg_status_t st = finish_transpose(g, 0)) return st;
    DG_CUDA(cudaDeviceSynchronize());
    return DG_OK;
  }
  if (!strcmp(name, "slice_features")) {
    if (value < 0 || value > (1 << 20)) return invalid("slice_features must be in [0, 2^20]");
    g->slice_features = value;
    return DG_OK;
  }
  if (!strcmp(name, "rows_per_block")) {
    if (value < 0 || value > 248) return invalid("rows_per_block must be in [0, 248]");
    g->rows_per_block = value;
    return DG_OK;
  }
  if (!strcmp(name, "l2_budget_mb")) {
    if (value < 1 || value > 4096) return invalid("l2_budget_mb must be in [1, 4096]");
    g->l2_budget_bytes = value << 20;
    return DG_OK;
  }
  if (!strcmp(name, "heavy_blocks_per_sm")) {
    if (value < 0 || value > 32) return invalid("heavy_blocks_per_sm must be in [0, 32]");
    g->heavy_blocks_per_sm = value;
    return DG_OK;
  }
  if (!strcmp(name, "self_loops")) {
    if (value != 0 && value != 1) return invalid("self_loops must be 0 or 1");
    g->self_loops = value;
    return DG_OK;
  }
  if (!strcmp(name, "source_blocks")) {
    if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8 && value != 16)
      return invalid("source_blocks must be 0 (automatic), 1, 2, 4, 8 or 16");
    g->source_blocks = value;
    return DG_OK;
  }
  return invalid("unknown parameter name");
}

dg_status_t dg_graph_get_param(dg_graph_t g, const char* name, int64_t* value) {
  if (!g || !name || !value) return invalid("graph handle, name or value is NULL");
  if (!strcmp(name, "heavy_threshold")) { *value = g->heavy_threshold; return DG_OK; }
  if (!strcmp(name, "slice_features")) { *value = g->slice_features; return DG_OK; }
  if (!strcmp(name, "rows_per_block")) { *value = g->rows_per_block; return DG_OK; }
  if (!strcmp(name, "l2_budget_mb")) { *value = g->l2_budget_bytes >> 20; return DG_OK; }
  if (!strcmp(name, "source_blocks")) { *value = g->source_blocks; return DG_OK; }
  if (!strcmp(name, "self_loops")) { *value = g->self_loops; return DG_OK; }
  if (!strcmp(name, "heavy_blocks_per_sm")) { *value = g->heavy_blocks_per_sm; return DG_OK; }
  return invalid("unknown parameter name");
}

int64_t dg_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* dg_last_error(void) { return g_last_error; }

const char* dg_version(void) { return "libdgagg 0.8 sm_100a"; }

}  // extern "C"
