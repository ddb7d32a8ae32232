// The general aggregation primitive: every operator pair of Table 1 of the paper,
//   f_O[v] = (+)_{edges e_uv into v} ( f_V[u] (x) f_E[e_uv] )          (Eq. 1, Eq. 2, Algorithm 1)
// with (x) in {copylhs, copyrhs, add, sub, mul, div}, (+) in {sum, max, min} and f_E a full
// |E| x F matrix (or |E| x 1, broadcast), its gradients with respect to f_V and f_E, and the
// gradient of the weighted sum / mean with respect to scalar edge weights (message passing onto
// edges, Section 2.2).
//
// These kernels are kept apart from the sum / mean kernels of dg_aggregate_kernels.cuh, which
// stay as they are: here a warp owns one row (one column in the pass over the CSC), its lanes
// are spread along the features in groups of G lanes, and the groups take different edges.  With
// a full edge-feature matrix the edge stream is as large as the gathered rows (nnz x F x 4
// bytes, read once, coalesced), so these passes are bound by HBM streaming rather than by the
// gather.
//
// Determinism: every output element is produced by one warp in a fixed order; the extremum of
// max / min is chosen on (message, edge position) pairs, equal messages going to the lowest
// position, so the order in which lane groups are combined does not matter.  No atomics.
#include "dg_internal.cuh"

namespace dg {
namespace {

constexpr int kGenBlock = 256;
constexpr int kGenWarps = kGenBlock / 32;
constexpr unsigned kAll = 0xffffffffu;
constexpr int kChain = 256;  // a register sum is moved to a second-level sum after this many terms

enum { kCopyLhs = DG_BIN_COPY_LHS, kCopyRhs = DG_BIN_COPY_RHS, kAdd = DG_BIN_ADD,
       kSub = DG_BIN_SUB, kMul = DG_BIN_MUL, kDiv = DG_BIN_DIV };
enum { kSum = DG_RED_SUM, kMax = DG_RED_MAX, kMin = DG_RED_MIN };

struct GenArgs {
  const int64_t* ptr;    // n+1 segment pointers: rowptr, or colptr in the pass over the CSC
  const int32_t* idx;    // colidx, or rowidx_T
  const int32_t* perm;   // CSC pass: CSR position of every CSC entry
  const int64_t* rowptr; // CSR row pointer (the divisor of the mean in the edge-weight gradient)
  const float* X;        // n x F vertex features (fV), or dO in the gradient passes
  const float* V;        // gradient passes: fV
  const float* Y;        // nnz x cols edge features in CSR position order
  const int32_t* arg;    // n x F edge positions of the extrema (max / min)
  float* out;            // n x F, or nnz x cols in the edge-gradient pass
  int32_t* arg_out;
  int64_t n;
  int32_t F, cols;
  int32_t log_g;         // lanes per edge = 1 << log_g
  int32_t row_scale;     // edge-weight gradient: 0 none, 1 = 1/deg(v), 2 = 1/(deg(v)+1)
};

// one fp32 IEEE operation, never contracted into a neighbouring add
template <int BIN>
__device__ __forceinline__ float message(float x, float y) {
  if (BIN == kCopyLhs) return x;
  if (BIN == kCopyRhs) return y;
  if (BIN == kAdd) return __fadd_rn(x, y);
  if (BIN == kSub) return __fsub_rn(x, y);
  if (BIN == kMul) return __fmul_rn(x, y);
  return __fdiv_rn(x, y);
}
template <int BIN>
__device__ __forceinline__ float d_dx(float y) {
  if (BIN == kCopyRhs) return 0.f;
  if (BIN == kMul) return y;
  if (BIN == kDiv) return __fdiv_rn(1.f, y);
  return 1.f;
}
template <int BIN>
__device__ __forceinline__ float d_dy(float x, float y) {
  if (BIN == kCopyLhs) return 0.f;
  if (BIN == kSub) return -1.f;
  if (BIN == kMul) return x;
  if (BIN == kDiv) return -__fdiv_rn(x, __fmul_rn(y, y));
  return 1.f;
}

// (value, position) of the better of two candidates; position < 0 means "none"
template <int RED>
__device__ __forceinline__ void take_better(float& best, int32_t& best_k, float m, int32_t k) {
  if (k < 0) return;
  const bool better = RED == kMax ? m > best : m < best;
  if (best_k < 0 || better || (m == best && k < best_k)) {
    best = m;
    best_k = k;
  }
}

// Forward: warp per destination row; lane (grp, c) takes feature f0 + c of the edges
// lo + grp, lo + grp + NG, ...
template <int BIN, int RED>
__global__ void __launch_bounds__(kGenBlock) general_fwd_kernel(const GenArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kGenWarps + (threadIdx.x >> 5);
  if (row >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int64_t lo = __ldg(a.ptr + row), hi = __ldg(a.ptr + row + 1);
  const int F = a.F, cols = a.cols;
  for (int f0 = 0; f0 < F; f0 += G) {
    const bool jok = f0 + c < F;
    const int j = jok ? f0 + c : 0;
    float acc = 0.f, total = 0.f, best = 0.f;
    int32_t best_k = -1;
    int chain = 0;
#pragma unroll 4
    for (int64_t e = lo + grp; e < hi; e += NG) {
      const float x = BIN != kCopyRhs ? __ldg(a.X + (size_t)__ldg(a.idx + e) * F + j) : 0.f;
      const float y = BIN != kCopyLhs ? __ldg(a.Y + (size_t)e * cols + (cols == 1 ? 0 : j)) : 0.f;
      const float m = message<BIN>(x, y);
      if (RED == kSum) {
        acc += m;
        if (++chain == kChain) { total += acc; acc = 0.f; chain = 0; }
      } else {
        take_better<RED>(best, best_k, m, (int32_t)e);
      }
    }
    total += acc;
    for (int off = G; off < 32; off <<= 1) {
      if (RED == kSum) {
        total += __shfl_xor_sync(kAll, total, off);
      } else {
        const float ob = __shfl_xor_sync(kAll, best, off);
        const int32_t ok = __shfl_xor_sync(kAll, best_k, off);
        take_better<RED>(best, best_k, ob, ok);
      }
    }
    if (grp == 0 && jok) {
      const size_t o = (size_t)row * F + j;
      if (RED == kSum) {
        a.out[o] = total;
      } else {
        a.out[o] = best_k >= 0 ? best : 0.f;
        if (a.arg_out) a.arg_out[o] = best_k;
      }
    }
  }
}

// Gradient with respect to fV: warp per source vertex u over its CSC segment,
//   dV[u][j] = sum_q sel * dO[v_q][j] * d(x (x) y)/dx,   sel = [arg[v_q][j] == perm[q]] (max/min)
// The derivative depends on y only (and not at all for copylhs / add / sub).
template <int BIN, int RED>
__global__ void __launch_bounds__(kGenBlock) general_bwd_vertex_kernel(const GenArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t u = (int64_t)blockIdx.x * kGenWarps + (threadIdx.x >> 5);
  if (u >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int64_t lo = __ldg(a.ptr + u), hi = __ldg(a.ptr + u + 1);
  const int F = a.F, cols = a.cols;
  constexpr bool kNeedsY = BIN == kMul || BIN == kDiv;
  for (int f0 = 0; f0 < F; f0 += G) {
    const bool jok = f0 + c < F;
    const int j = jok ? f0 + c : 0;
    float acc = 0.f, total = 0.f;
    int chain = 0;
#pragma unroll 4
    for (int64_t q = lo + grp; q < hi; q += NG) {
      const size_t vj = (size_t)__ldg(a.idx + q) * F + j;
      float t = __ldg(a.X + vj);  // dO[v][j]
      int32_t k = 0;
      if (kNeedsY || RED != kSum) k = __ldg(a.perm + q);
      if (kNeedsY) t *= d_dx<BIN>(__ldg(a.Y + (size_t)k * cols + (cols == 1 ? 0 : j)));
      if (RED != kSum && __ldg(a.arg + vj) != k) t = 0.f;
      acc += t;
      if (++chain == kChain) { total += acc; acc = 0.f; chain = 0; }
    }
    total += acc;
    for (int off = G; off < 32; off <<= 1) total += __shfl_xor_sync(kAll, total, off);
    if (grp == 0 && jok) a.out[(size_t)u * F + j] = total;
  }
}

// Gradient with respect to fE, full edge features (cols == F): one value per (edge, feature),
//   dE[k][j] = sel * dO[v][j] * d(x (x) y)/dy
template <int BIN, int RED>
__global__ void __launch_bounds__(kGenBlock) general_bwd_edge_full_kernel(const GenArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t v = (int64_t)blockIdx.x * kGenWarps + (threadIdx.x >> 5);
  if (v >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int64_t lo = __ldg(a.ptr + v), hi = __ldg(a.ptr + v + 1);
  const int F = a.F;
  constexpr bool kNeedsX = BIN == kMul || BIN == kDiv;
  for (int f0 = 0; f0 < F; f0 += G) {
    if (f0 + c >= F) continue;
    const int j = f0 + c;
    const float g = __ldg(a.X + (size_t)v * F + j);
    const int32_t sel = RED != kSum ? __ldg(a.arg + (size_t)v * F + j) : 0;
    for (int64_t e = lo + grp; e < hi; e += NG) {
      const float x = kNeedsX ? __ldg(a.V + (size_t)__ldg(a.idx + e) * F + j) : 0.f;
      const float y = BIN == kDiv ? __ldg(a.Y + (size_t)e * F + j) : 0.f;
      float t = g * d_dy<BIN>(x, y);
      if (RED != kSum && sel != (int32_t)e) t = 0.f;
      a.out[(size_t)e * F + j] = t;
    }
  }
}

// Gradient with respect to fE with one column (the broadcast scalar): the feature sum of the
// above, one dot product per edge reduced inside the lane group:
//   dE[k] = s_v * sum_j sel * dO[v][j] * d(x (x) y)/dy
// With (x) = mul and (+) = sum this is the sampled dense-dense product <fV[u_k], dO[v_k]>, the
// gradient with respect to a scalar edge weight; row_scale gives the mean's s_v.
template <int BIN, int RED>
__global__ void __launch_bounds__(kGenBlock) general_bwd_edge_scalar_kernel(const GenArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t v = (int64_t)blockIdx.x * kGenWarps + (threadIdx.x >> 5);
  if (v >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int64_t lo = __ldg(a.ptr + v), hi = __ldg(a.ptr + v + 1);
  const int F = a.F;
  constexpr bool kNeedsX = BIN == kMul || BIN == kDiv;
  float s = 1.f;
  if (a.row_scale) s = 1.0f / (float)(hi - lo + (a.row_scale == 2 ? 1 : 0));
  for (int64_t e0 = lo; e0 < hi; e0 += NG) {   // uniform trip count: the shuffles need all lanes
    const int64_t e = e0 + grp;
    const bool eok = e < hi;
    float dot = 0.f;
    if (eok) {
      const float* xrow = kNeedsX ? a.V + (size_t)__ldg(a.idx + e) * F : nullptr;
      const float y = BIN == kDiv ? __ldg(a.Y + e) : 0.f;
      for (int j = c; j < F; j += G) {
        float t = __ldg(a.X + (size_t)v * F + j) * d_dy<BIN>(kNeedsX ? __ldg(xrow + j) : 0.f, y);
        if (RED != kSum && __ldg(a.arg + (size_t)v * F + j) != (int32_t)e) t = 0.f;
        dot += t;
      }
    }
    for (int off = 1; off < G; off <<= 1) dot += __shfl_xor_sync(kAll, dot, off);
    if (eok && c == 0) a.out[e] = dot * s;
  }
}

// The same dot product with 16-byte loads for the entry point dg_aggregate_edge_grad (rows of
// both matrices 16-byte aligned): lane c of a group takes float4 c, c + G, ... of the two rows.
__global__ void __launch_bounds__(kGenBlock) edge_weight_grad_vec4_kernel(const GenArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t v = (int64_t)blockIdx.x * kGenWarps + (threadIdx.x >> 5);
  if (v >= a.n) return;
  const int G = 1 << a.log_g, NG = 32 >> a.log_g;
  const int grp = lane >> a.log_g, c = lane & (G - 1);
  const int64_t lo = __ldg(a.ptr + v), hi = __ldg(a.ptr + v + 1);
  const int nvec = a.F >> 2;
  float s = 1.f;
  if (a.row_scale) s = 1.0f / (float)(hi - lo + (a.row_scale == 2 ? 1 : 0));
  const float4* grow = reinterpret_cast<const float4*>(a.X + (size_t)v * a.F);
  for (int64_t e0 = lo; e0 < hi; e0 += NG) {
    const int64_t e = e0 + grp;
    const bool eok = e < hi;
    float dot = 0.f;
    if (eok) {
      const float4* xrow = reinterpret_cast<const float4*>(a.V + (size_t)__ldg(a.idx + e) * a.F);
#pragma unroll 4
      for (int j = c; j < nvec; j += G) {
        const float4 x = __ldg(xrow + j), g = __ldg(grow + j);
        dot += x.x * g.x + x.y * g.y + x.z * g.z + x.w * g.w;
      }
    }
    for (int off = 1; off < G; off <<= 1) dot += __shfl_xor_sync(kAll, dot, off);
    if (eok && c == 0) a.out[e] = dot * s;
  }
}

int log_group(int32_t width) {  // lanes per edge: the power of two covering `width`, at most 32
  int lg = 0;
  while (lg < 5 && (1 << lg) < width) ++lg;
  return lg;
}

inline unsigned warp_blocks(int64_t n) { return (unsigned)((n + kGenWarps - 1) / kGenWarps); }

template <template <int, int> class L>
dg_status_t dispatch_ops(int bin, int red, const GenArgs& a, cudaStream_t s) {
#define DG_GEN_CASE(B)                                                   \
  case B:                                                                \
    if (red == kSum) return L<B, kSum>::run(a, s);                       \
    if (red == kMax) return L<B, kMax>::run(a, s);                       \
    return L<B, kMin>::run(a, s);
  switch (bin) {
    DG_GEN_CASE(kCopyLhs)
    DG_GEN_CASE(kCopyRhs)
    DG_GEN_CASE(kAdd)
    DG_GEN_CASE(kSub)
    DG_GEN_CASE(kMul)
    default:
      DG_GEN_CASE(kDiv)
  }
#undef DG_GEN_CASE
}

#define DG_GEN_LAUNCHER(NAME, KERNEL)                                         \
  template <int BIN, int RED>                                                 \
  struct NAME {                                                               \
    static dg_status_t run(const GenArgs& a, cudaStream_t s) {                \
      KERNEL<BIN, RED><<<warp_blocks(a.n), kGenBlock, 0, s>>>(a);             \
      DG_CUDA(cudaGetLastError());                                            \
      count_launches(1);                                                      \
      return DG_OK;                                                           \
    }                                                                         \
  };
DG_GEN_LAUNCHER(FwdLauncher, general_fwd_kernel)
DG_GEN_LAUNCHER(BwdVertexLauncher, general_bwd_vertex_kernel)
DG_GEN_LAUNCHER(BwdEdgeFullLauncher, general_bwd_edge_full_kernel)
DG_GEN_LAUNCHER(BwdEdgeScalarLauncher, general_bwd_edge_scalar_kernel)
#undef DG_GEN_LAUNCHER

dg_status_t bad(const char* msg) {
  set_error("%s", msg);
  return DG_ERR_INVALID_ARG;
}

dg_status_t check_operands(const dg_graph* g, const float* fV, const float* fE, int32_t fE_cols,
                           int32_t F, int bin, int red) {
  if (!g) return bad("graph handle is NULL");
  if (F < 1) return bad("F must be >= 1");
  if (F > (1 << 20)) {
    set_error("F must be at most 2^20");
    return DG_ERR_UNSUPPORTED;
  }
  if (bin < kCopyLhs || bin > kDiv) return bad("binary must be one of the dg_binary_t values");
  if (red < kSum || red > kMin) return bad("reduce must be one of the dg_reduce_t values");
  if (bin != kCopyRhs && !fV && g->n > 0) return bad("fV is NULL (only copyrhs works without it)");
  if (bin != kCopyLhs) {
    if (!fE && g->nnz > 0) return bad("fE is NULL (only copylhs works without it)");
    if (fE_cols != 1 && fE_cols != F) return bad("fE_cols must be 1 or F");
  }
  return DG_OK;
}

}  // namespace
}  // namespace dg

using namespace dg;

extern "C" {

dg_status_t dg_ap_fwd(dg_graph_t g, const float* fV, const float* fE, int32_t fE_cols, int32_t F,
                      dg_binary_t binary, dg_reduce_t reduce, float* fO, int32_t* arg,
                      void* stream) {
  if (dg_status_t st = check_operands(g, fV, fE, fE_cols, F, (int)binary, (int)reduce)) return st;
  if (g->n == 0) return DG_OK;
  if (!fO) return bad("fO is NULL");
  GenArgs a{};
  a.ptr = g->rowptr;
  a.idx = g->colidx;
  a.X = fV;
  a.Y = fE;
  a.out = fO;
  a.arg_out = reduce == DG_RED_SUM ? nullptr : arg;
  a.n = g->n;
  a.F = F;
  a.cols = binary == DG_BIN_COPY_LHS ? 1 : fE_cols;
  a.log_g = log_group(F);
  return dispatch_ops<FwdLauncher>((int)binary, (int)reduce, a, (cudaStream_t)stream);
}

dg_status_t dg_ap_bwd(dg_graph_t g, const float* dO, const float* fV, const float* fE,
                      int32_t fE_cols, int32_t F, dg_binary_t binary, dg_reduce_t reduce,
                      const int32_t* arg, float* dV, float* dE, void* stream) {
  if (dg_status_t st = check_operands(g, fV, fE, fE_cols, F, (int)binary, (int)reduce)) return st;
  if (g->n == 0) return DG_OK;
  if (!dO) return bad("dO is NULL");
  if (reduce != DG_RED_SUM && !arg) return bad("max / min need the arg output of dg_ap_fwd");
  if (dE && binary == DG_BIN_COPY_LHS) return bad("copylhs has no edge operand: dE must be NULL");
  cudaStream_t s = (cudaStream_t)stream;
  const int32_t cols = binary == DG_BIN_COPY_LHS ? 1 : fE_cols;
  if (dV) {
    if (binary == DG_BIN_COPY_RHS) {  // the result does not depend on fV
      DG_CUDA(cudaMemsetAsync(dV, 0, (size_t)g->n * (size_t)F * sizeof(float), s));
    } else {
      if (!g->transposed) {
        set_error("the gradient with respect to fV gathers over the CSC: call dg_graph_transpose first");
        return DG_ERR_NOT_TRANSPOSED;
      }
      GenArgs a{};
      a.ptr = g->colptr;
      a.idx = g->rowidx_T;
      a.perm = g->perm;
      a.X = dO;
      a.Y = fE;
      a.arg = arg;
      a.out = dV;
      a.n = g->n;
      a.F = F;
      a.cols = cols;
      a.log_g = log_group(F);
      if (dg_status_t st = dispatch_ops<BwdVertexLauncher>((int)binary, (int)reduce, a, s)) return st;
    }
  }
  if (dE && g->nnz > 0) {
    GenArgs a{};
    a.ptr = g->rowptr;
    a.idx = g->colidx;
    a.X = dO;
    a.V = fV;
    a.Y = fE;
    a.arg = arg;
    a.out = dE;
    a.n = g->n;
    a.F = F;
    a.cols = cols;
    a.log_g = log_group(F);
    if (cols == 1)
      return dispatch_ops<BwdEdgeScalarLauncher>((int)binary, (int)reduce, a, s);
    return dispatch_ops<BwdEdgeFullLauncher>((int)binary, (int)reduce, a, s);
  }
  return DG_OK;
}

dg_status_t dg_aggregate_edge_grad(dg_graph_t g, const float* H, const float* dOut, int32_t F,
                                   dg_op_t op, float* dW, void* stream) {
  if (!g) return bad("graph handle is NULL");
  if (F < 1) return bad("F must be >= 1");
  if (F > (1 << 20)) {
    set_error("F must be at most 2^20");
    return DG_ERR_UNSUPPORTED;
  }
  if (op != DG_OP_SUM && op != DG_OP_MEAN) return bad("op must be DG_OP_SUM or DG_OP_MEAN");
  if (g->nnz == 0) return DG_OK;
  if (!H || !dOut || !dW) return bad("H, dOut or dW is NULL");
  GenArgs a{};
  a.ptr = g->rowptr;
  a.idx = g->colidx;
  a.X = dOut;
  a.V = H;
  a.out = dW;
  a.n = g->n;
  a.F = F;
  a.cols = 1;
  a.row_scale = op == DG_OP_MEAN ? (g->self_loops ? 2 : 1) : 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (F % 4 == 0 && (((uintptr_t)H | (uintptr_t)dOut) & 15) == 0) {
    a.log_g = log_group(F / 4);
    edge_weight_grad_vec4_kernel<<<warp_blocks(a.n), kGenBlock, 0, s>>>(a);
    DG_CUDA(cudaGetLastError());
    count_launches(1);
    return DG_OK;
  }
  a.log_g = log_group(F);
  return BwdEdgeScalarLauncher<kMul, kSum>::run(a, s);
}

}  // extern "C"
