// The aggregation kernels for graphs with implicit self loops and a segment of 2^15 entries or
// more: self-loop epilogue and two-level sum of the block-per-row path together.
#include "dg_aggregate_kernels.cuh"

namespace dg {

dg_status_t launch_with_self_loops_fold(const Graph* g, const ApArgs& a, const SelfArgs& sa, int vec,
                                        int slices, cudaStream_t s) {
  return dispatch_type<true, true>(g, a, sa, vec, slices, s);
}

}  // namespace dg
