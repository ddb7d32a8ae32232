// The aggregation kernels compiled for graphs with implicit self loops (the row's own input row
// joins its sum): a translation unit of its own, so that the two sets build
// side by side and the plain kernels carry nothing of the extra epilogue.
#include "dg_aggregate_kernels.cuh"

namespace dg {

dg_status_t launch_with_self_loops(const Graph* g, const ApArgs& a, const SelfArgs& sa, int vec,
                                   int slices, cudaStream_t s) {
  return dispatch_type<true>(g, a, sa, vec, slices, s);
}

}  // namespace dg
