// Diagnostic kernel behind dg_probe_gather: the rate at which this GPU delivers randomly gathered
// rows to its SMs, from a table that is L2-resident or far larger than L2.  It is the access
// pattern of the aggregation kernels with everything else removed (no rows, no weights, one
// output row per warp), so its numbers are the ceilings the aggregation rates are read against.
#include <cooperative_groups.h>

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
  // the index stream runs kAhead batches (128 gathers) ahead, so that the probe measures the
  // gather and not the latency of its index loads
  constexpr int kAhead = 4;
  int32_t next[kAhead];
#pragma unroll
  for (int t = 0; t < kAhead; ++t)
    next[t] = base + t * 32 + lane < end ? __ldcs(idx + base + t * 32 + lane) : 0;
  for (int64_t b0 = base; b0 < end; b0 += 32 * kAhead) {
    int32_t cur[kAhead];
#pragma unroll
    for (int t = 0; t < kAhead; ++t) {
      cur[t] = next[t];
      const int64_t k = b0 + (kAhead + t) * 32 + lane;
      next[t] = k < end ? __ldcs(idx + k) : 0;
    }
#pragma unroll
    for (int t = 0; t < kAhead; ++t) {
      const int64_t b = b0 + t * 32;
      if (b >= end) break;
      const int cnt = (int)(end - b < 32 ? end - b : 32);
      for (int e0 = 0; e0 < cnt; e0 += kProbeSteps * groups) {
        float4 v[kProbeSteps];
#pragma unroll
        for (int j = 0; j < kProbeSteps; ++j) {
          const int e = e0 + j * groups + grp;
          const int32_t u = __shfl_sync(0xffffffffu, cur[t], e & 31);
          v[j] = e < cnt ? __ldg(table + (size_t)u * row_f4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < kProbeSteps; ++j) {
          acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w;
        }
      }
    }
  }
  sink[warp * 32 + lane] = acc;
}

// The same gather served from shared memory: every block first fills `stage_rows` rows of
// `row_f4` float4 (row r holds the value r in every element), then its warps gather rows named
// by idx from that stage, kSmemPerWarp gathers per warp.  REMOTE: blocks run as clusters of two
// and every gather reads the partner block's stage through distributed shared memory.  What it
// measures is what a kernel could gain by staging a block of the gathered matrix on chip
// instead of fetching every row through the L2 -> SM fabric.
constexpr int kSmemBlock = 1024;
constexpr int kSmemPerWarp = 4096;

template <bool REMOTE>
__global__ void __launch_bounds__(kSmemBlock)
probe_smem_kernel(const int32_t* __restrict__ idx, int64_t count, int row_f4, int stage_rows,
                  float4* __restrict__ sink) {
  extern __shared__ float4 stage[];
  for (int i = threadIdx.x; i < stage_rows * row_f4; i += kSmemBlock) {
    const float r = (float)(i / row_f4);
    stage[i] = make_float4(r, r, r, r);
  }
  const float4* src = stage;
  if (REMOTE) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();
    src = cluster.map_shared_rank(stage, cluster.block_rank() ^ 1u);
  } else {
    __syncthreads();
  }
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * kSmemBlock + threadIdx.x) >> 5;
  const int64_t base = warp * kSmemPerWarp;
  const int64_t end = base + kSmemPerWarp < count ? base + kSmemPerWarp : count;
  const int c = lane % row_f4, grp = lane / row_f4, groups = 32 / row_f4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // The index stream runs kAhead batches (128 gathers) ahead of the gathers: with one block per
  // SM there are too few warps to hide the latency of an index load per 32 gathers otherwise,
  // and the probe would measure that latency instead of the shared-memory gather.
  constexpr int kAhead = 4;
  int32_t next[kAhead];
#pragma unroll
  for (int t = 0; t < kAhead; ++t)
    next[t] = base + t * 32 + lane < end ? __ldcs(idx + base + t * 32 + lane) : 0;
  for (int64_t b0 = base; b0 < end; b0 += 32 * kAhead) {
    int32_t cur[kAhead];
#pragma unroll
    for (int t = 0; t < kAhead; ++t) {
      cur[t] = next[t] < 0 ? 0 : (next[t] >= stage_rows ? stage_rows - 1 : next[t]);
      const int64_t k = b0 + (kAhead + t) * 32 + lane;
      next[t] = k < end ? __ldcs(idx + k) : 0;
    }
#pragma unroll
    for (int t = 0; t < kAhead; ++t) {
      const int64_t b = b0 + t * 32;
      if (b >= end) break;
      const int cnt = (int)(end - b < 32 ? end - b : 32);
      for (int e0 = 0; e0 < cnt; e0 += kProbeSteps * groups) {
        float4 v[kProbeSteps];
#pragma unroll
        for (int j = 0; j < kProbeSteps; ++j) {
          const int e = e0 + j * groups + grp;
          const int32_t u = __shfl_sync(0xffffffffu, cur[t], e & 31);
          v[j] = e < cnt ? src[(size_t)u * row_f4 + c] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < kProbeSteps; ++j) {
          acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w;
        }
      }
    }
  }
  if (base < count) sink[warp * 32 + lane] = acc;
  if (REMOTE) cooperative_groups::this_cluster().sync();  // the partner may still read this stage
}

}  // namespace

extern "C" dg_status_t dg_probe_gather_smem(int32_t row_floats, int32_t stage_rows,
                                            const int32_t* idx, int64_t count, float* sink,
                                            int32_t remote, void* stream) {
  if (!idx || !sink || count < 1 || stage_rows < 1) {
    dg::set_error("dg_probe_gather_smem: NULL pointer or empty input");
    return DG_ERR_INVALID_ARG;
  }
  if (row_floats < 4 || row_floats > 128 || (row_floats & (row_floats - 1)) != 0) {
    dg::set_error("dg_probe_gather_smem: row_floats must be a power of two in [4, 128]");
    return DG_ERR_INVALID_ARG;
  }
  const size_t smem = (size_t)stage_rows * (size_t)row_floats * sizeof(float);
  if (smem > 200 * 1024) {
    dg::set_error("dg_probe_gather_smem: the stage must fit 200 KiB of shared memory");
    return DG_ERR_UNSUPPORTED;
  }
  if ((uintptr_t)sink & 15) {
    dg::set_error("dg_probe_gather_smem: sink must be 16-byte aligned");
    return DG_ERR_INVALID_ARG;
  }
  const int64_t warps = (count + kSmemPerWarp - 1) / kSmemPerWarp;
  int64_t blocks = (warps * 32 + kSmemBlock - 1) / kSmemBlock;
  if (remote) blocks = (blocks + 1) & ~(int64_t)1;  // whole clusters of two
  auto kernel = remote ? probe_smem_kernel<true> : probe_smem_kernel<false>;
  DG_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(kSmemBlock);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = remote ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  DG_CUDA(cudaLaunchKernelEx(&cfg, kernel, idx, count, (int)(row_floats / 4), (int)stage_rows,
                             reinterpret_cast<float4*>(sink)));
  dg::count_launches(1);
  return DG_OK;
}

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
