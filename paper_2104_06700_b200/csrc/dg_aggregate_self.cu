// The aggregation kernels compiled for graphs with implicit self loops (the row's own input row
// joins its sum): a translation unit of its own, so that the sets build side by side and the plain
// kernels carry nothing of the extra epilogue.
#include "dg_aggregate_kernels.cuh"

namespace dg {

dg_status_t launch_with_self_loops(const Graph* g, const ApArgs& a, const SelfArgs& sa, int vec,
                                   int slices, cudaStream_t s) {
  if (a.long_segments) return launch_with_self_loops_fold(g, a, sa, vec, slices, s);
  return dispatch_type<true, false>(g, a, sa, vec, slices, s);
}

}  // namespace dg
