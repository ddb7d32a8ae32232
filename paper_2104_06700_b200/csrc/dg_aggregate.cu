// Host side of the aggregation: chooses the launch shape of one call (vector width, feature
// slices, source blocks) and runs one launch per source block.  The kernels are in
// dg_aggregate_kernels.cuh; this file compiles them for graphs without implicit self loops and
// without long segments, dg_aggregate_fold.cu, dg_aggregate_self.cu and dg_aggregate_self_fold.cu
// for the other three combinations (four translation units compile side by side).
#include "dg_aggregate_kernels.cuh"

namespace dg {

dg_status_t launch_plain(const Graph* g, const ApArgs& a, int vec, int slices, cudaStream_t s) {
  if (a.long_segments) return launch_plain_fold(g, a, vec, slices, s);
  return dispatch_type<false, false>(g, a, SelfArgs{}, vec, slices, s);
}

// Bytes of L2 one row slice of `slice` elements of `eb` bytes occupies: L2 allocates 128-byte
// lines, and a slice that does not start on a line boundary in every row touches one more line.
static double slice_footprint(int64_t F, int64_t slice, int eb) {
  const int64_t bytes = slice * eb;
  const bool aligned = (F * eb) % 128 == 0 && bytes % 128 == 0;
  return (double)(((bytes + 127) / 128) * 128 + (aligned ? 0 : 128));
}

// Chooses the launch shape, then runs one launch per source block.
//   vector width: the widest both matrices allow (16-byte loads of the gathered matrix when
//     its rows and its base are 16-byte aligned, else 8 or 4 bytes);
//   slice: at most 128 vectors per row slice (4 per lane);
//   source blocks (Algorithm 2 of the paper, with L2 in the role of the CPU cache): when one
//     slice of X over all n rows exceeds the L2 budget and the segments carry split pointers,
//     the neighbour ids are cut into 2, 4, 8 or 16 ranges and each range is a launch of its
//     own, so that the rows of X a launch gathers stay L2-resident; later launches add to Y.
//     Without split pointers the slice is narrowed instead (down to 128 bytes).
dg_status_t aggregate_run(const Graph* g, const ApArgs& a0, const SelfArgs& sa, const int32_t* split,
                          cudaStream_t s) {
  ApArgs a = a0;
  if (a.n == 0) return DG_OK;
  const uintptr_t px = (uintptr_t)a.X, py = (uintptr_t)a.Y;
  const bool bf16 = a.x_bf16 != 0;
  const int eb = bf16 ? 2 : 4;
  int vec = 1;  // elements per lane and vector
  if (bf16) {
    if (a.F % 8 == 0 && px % 16 == 0 && py % 16 == 0) vec = 8;
    else if (a.F % 4 == 0 && px % 8 == 0 && py % 16 == 0) vec = 4;
    else if (a.F % 2 == 0 && px % 4 == 0 && py % 8 == 0) vec = 2;
    else {
      set_error("bf16 feature matrices need an even F and 4-byte (input) / 8-byte (output) alignment");
      return DG_ERR_UNSUPPORTED;
    }
  } else {
    if (a.F % 4 == 0 && px % 16 == 0 && py % 16 == 0) vec = 4;
    else if (a.F % 2 == 0 && px % 8 == 0 && py % 8 == 0) vec = 2;
  }

  const double budget = (double)g->l2_budget_bytes;
  const double avg_len = (double)g->nnz / (double)a.n;
  const int64_t cap = 128LL * vec;
  int64_t slice = g->slice_features > 0 ? g->slice_features : (a.F < cap ? (int64_t)a.F : cap);
  if (slice > cap) slice = cap;
  if (slice > a.F) slice = a.F;
  int nb = 1;
  if (g->source_blocks > 0) {
    nb = split ? (int)g->source_blocks : 1;
  } else if (g->slice_features <= 0 && (double)a.n * slice_footprint(a.F, slice, eb) > budget) {
    if (split) {
      // widest slice first; a candidate is feasible when some block count keeps one block of
      // the slice inside the budget and leaves a row at least 32 edges per block on average
      const int64_t widths[4] = {64LL * vec, 32LL * vec, 16LL * vec, 8LL * vec};
      bool found = false;
      for (int t = 0; t < 4 && !found; ++t) {
        int64_t w = widths[t];
        if (w > slice) w = slice;
        int cand = 1;
        while (cand < kFineBlocks && (double)a.n / cand * slice_footprint(a.F, w, eb) > budget)
          cand *= 2;
        if ((double)a.n / cand * slice_footprint(a.F, w, eb) <= budget && avg_len / cand >= 32.0) {
          slice = w;
          nb = cand;
          found = true;
        }
      }
      if (!found) {  // as many blocks as the row length allows, narrowest slice
        nb = 1;
        while (nb < kFineBlocks && avg_len / (nb * 2) >= 32.0) nb *= 2;
        if (slice > 8LL * vec) slice = 8LL * vec;
      }
    } else {
      int64_t w = (int64_t)(budget / ((double)a.n * eb));
      if (w * eb >= 128) slice = w < slice ? w : slice;  // under 128 bytes is not worth a pass
    }
  }
  slice = (slice / vec) * vec;
  if (slice < vec) slice = vec;
  if ((a.F + slice - 1) / slice > 65535) {  // grid.y limit: widen a (requested) tiny slice
    slice = (a.F + 65534) / 65535;
    slice = ((slice + vec - 1) / vec) * vec;
  }
  // even out the slices: same count, smallest width that covers F
  const int64_t nsl = (a.F + slice - 1) / slice;
  int64_t even = (a.F + nsl - 1) / nsl;
  even = ((even + vec - 1) / vec) * vec;
  if (even <= slice) slice = even;
  a.slice_f = (int32_t)slice;
  const int slices = (int)((a.F + slice - 1) / slice);

  const int per = kFineBlocks / nb;
  for (int j = 0; j < nb; ++j) {
    if (nb > 1) {
      a.seg_lo = split + (size_t)(j * per) * (size_t)a.n;
      a.seg_hi = split + (size_t)((j + 1) * per) * (size_t)a.n;
      a.accumulate = j > 0;
    }
    const dg_status_t st = sa.self_ptr ? launch_with_self_loops(g, a, sa, vec, slices, s)
                                       : launch_plain(g, a, vec, slices, s);
    if (st != DG_OK) return st;
  }
  return DG_OK;
}

}  // namespace dg
