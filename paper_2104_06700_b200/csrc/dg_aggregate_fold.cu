// The aggregation kernels compiled with the two-level sum of the block-per-row path, for graphs
// that hold a segment of 2^15 entries or more (no implicit self loops).  A translation unit of
// its own: the common kernels stay exactly as they are without it, and the sets build side by side.
#include "dg_aggregate_kernels.cuh"

namespace dg {

dg_status_t launch_plain_fold(const Graph* g, const ApArgs& a, int vec, int slices, cudaStream_t s) {
  return dispatch_type<false, true>(g, a, SelfArgs{}, vec, slices, s);
}

}  // namespace dg
