// Diagnostic kernel behind dg_probe_gather: the rate at which this GPU delivers randomly gathered
// rows to its SMs, from a table that is L2-resident or far larger than L2.  It is the access
// pattern of the aggregation kernels with everything else removed (no rows, no weights, one
// output row per warp), so its numbers are the ceilings the aggregation rates are read against.
#include "dg_internal.cuh"

namespace {

constexpr int kProbePerWarp = 512;  // gathered rows per warp
constexpr int kProbeSteps = 4;      // loads in flight per lane

// Rows of 32 float4 (512 bytes) at most: lane c of a group of `row_f4` lanes loads float4 c of
// its group's row; groups take different rows.
__global__ void __launch_bounds__(256)
probe_gather_kernel(const float4* __restrict__ table, const int32_t* __restrict__ idx,
                    int64_t count, int row_f4, float4* __restrict__ sink) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t base = warp * kProbePerWarp;
  if (base >= count) return;
  const int64_t end = base + kProbePerWarp < count ? base + kProbePerWarp : count;
  const int c = lane % row_f4, grp = lane / row_f4, groups = 32 / row_f4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int64_t b = base; b < end; b += 32) {
    const int32_t mine = b + lane < end ? __ldcs(idx + b + lane) : 0;
    const int cnt = (int)(end - b < 32 ? end - b : 32);
    for (int e0 = 0; e0 < cnt; e0 += kProbeSteps * groups) {
      float4 v[kProbeSteps];
#pragma unroll
      for (int j = 0; j < kProbeSteps; ++j) {
        const int e = e0 + j * groups + grp;
        const int32_t u = __shfl_sync(0xffffffffu, mine, e & 31);
        v[j] = e < cnt ? __ldg(table + (size_t)u * row_f4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int j = 0; j < kProbeSteps; ++j) {
        acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w;
      }
    }
  }
  sink[warp * 32 + lane] = acc;
}

}  // namespace

extern "C" dg_status_t dg_probe_gather(const float* table, int64_t rows, int32_t row_floats,
                                       const int32_t* idx, int64_t count, float* sink,
                                       void* stream) {
  if (!table || !idx || !sink || rows < 1 || count < 1) {
    dg::set_error("dg_probe_gather: NULL pointer or empty input");
    return DG_ERR_INVALID_ARG;
  }
  if (row_floats < 4 || row_floats > 128 || (row_floats & (row_floats - 1)) != 0) {
    dg::set_error("dg_probe_gather: row_floats must be a power of two in [4, 128]");
    return DG_ERR_INVALID_ARG;
  }
  if (((uintptr_t)table | (uintptr_t)sink) & 15) {
    dg::set_error("dg_probe_gather: table and sink must be 16-byte aligned");
    return DG_ERR_INVALID_ARG;
  }
  const int64_t warps = (count + kProbePerWarp - 1) / kProbePerWarp;
  const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
  probe_gather_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const float4*>(table), idx, count, row_floats / 4,
      reinterpret_cast<float4*>(sink));
  DG_CUDA(cudaGetLastError());
  dg::count_launches(1);
  return DG_OK;
}
