// dg_graph_transpose_static: the CSR -> CSC build with its scratch buffers in a fixed array
// that is part of the library image, for callers that have no way to hand over scratch memory.
//
// Who needs this: a host program that reserved the whole device for its own memory pool (so a
// cudaMalloc from a plug-in fails or is forbidden by policy), code that runs where the implicit
// device-wide synchronisation of cudaMalloc/cudaFree is not acceptable (a latency-bound serving
// loop), and small embedders that only own the input and output arrays they were given.  They
// still pass the CSC storage (it is an output), but nothing else.
//
// The price is a fixed size limit and a fixed footprint: every GPU on which a process loads the
// library carries the array below from load until exit, whether or not this entry point is
// ever called.
#include <atomic>

#include "dg_internal.cuh"

namespace {

// Scratch of the radix sort (two key buffers, one value buffer, the digit histogram and its
// chunk sums).  256-byte alignment matches what the sort's layout assumes for its sub-buffers.
static __device__ __align__(256) unsigned char g_transpose_scratch[DG_TRANSPOSE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// device address of the array, per device ordinal (two threads that look it up at the same
// time get the same answer, so a plain atomic slot per device is enough)
std::atomic<void*> g_scratch_addr[kMaxDevices] = {};

// In host code the array's name is only a handle for the runtime, not a pointer a kernel could
// use; the device address has to be asked for, once per device, with that device current.
dg_status_t scratch_address(int graph_device, void** out) {
  int dev = 0;
  DG_CUDA(cudaGetDevice(&dev));
  if (dev != graph_device) {
    // the array of the current device would be paired with another device's graph arrays
    dg::set_error("dg_graph_transpose_static: the handle was created on device %d, the current "
                  "device is %d", graph_device, dev);
    return DG_ERR_INVALID_ARG;
  }
  if (dev < 0 || dev >= kMaxDevices) {
    dg::set_error("dg_graph_transpose_static: device ordinal beyond the table of 64 devices");
    return DG_ERR_UNSUPPORTED;
  }
  void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    DG_CUDA(cudaGetSymbolAddress(&p, g_transpose_scratch));
    g_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return DG_OK;
}

}  // namespace

extern "C" dg_status_t dg_graph_transpose_static(dg_graph_t g, void* csc_storage,
                                                 size_t csc_bytes, void* stream) {
  if (!g) {
    dg::set_error("graph handle is NULL");
    return DG_ERR_INVALID_ARG;
  }
  if (!csc_storage || ((uintptr_t)csc_storage & 255)) {
    dg::set_error("csc_storage is NULL or not 256-byte aligned");
    return DG_ERR_INVALID_ARG;
  }
  size_t need_csc = 0, need_scratch = 0;
  dg::transpose_sizes(g->n, g->nnz, g->edge_w != nullptr, &need_csc, &need_scratch);
  if (need_scratch > (size_t)DG_TRANSPOSE_STATIC_SCRATCH_BYTES) {
    dg::set_error("dg_graph_transpose_static: this graph needs %zu bytes of scratch, the built-in "
                  "array holds %zu; use dg_graph_transpose with caller-supplied scratch",
                  need_scratch, (size_t)DG_TRANSPOSE_STATIC_SCRATCH_BYTES);
    return DG_ERR_UNSUPPORTED;
  }
  if (csc_bytes < need_csc) {
    dg::set_error("csc_storage smaller than dg_graph_transpose_workspace reports");
    return DG_ERR_WORKSPACE;
  }
  void* scratch = nullptr;
  if (dg_status_t st = scratch_address(g->device, &scratch)) return st;
  cudaStream_t s = (cudaStream_t)stream;
  // Every buffer of the sort (keys, values, histogram, chunk sums) is written in full before it
  // is read, so what an earlier call left in the array needs no clearing.
  g->transposed = false;
  if (dg_status_t st = dg::transpose_run(g, csc_storage, scratch, s)) return st;
  g->transposed = true;
  return dg::finish_transpose(g, s);
}
