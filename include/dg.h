/*
 * libdgagg -- the aggregation primitive (AP) of full-batch GraphSAGE training on one B200.
 *
 * AP is the sparse-times-dense product f_O = A x f_V of Section 2.1 of the paper (Eq. 1 with
 * the binary operator "multiply by the edge's scalar weight", Eq. 2 with the unary copy, both
 * with the reducer "sum" of Table 1), computed in the pull form of Algorithm 1: the CSR row of
 * a destination vertex v lists the source vertices u that have an edge u -> v (Section 3.1).
 * "mean" divides the sum by the in-degree of v, the normalisation of Section 5.1 (Models and
 * Parameters).  The backward pass dH = A^T x dOut and the CSR -> CSC build it needs are not
 * written in the paper; they are the adjoint of the forward pass and a stable counting sort.
 *
 * Conventions for every entry point
 *   - plain C ABI, no exceptions cross it; every call returns a dg_status_t, and
 *     dg_last_error() gives a message for the last failure on the calling thread;
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers are
 *     ordinary process memory; the library never takes ownership of a caller's buffer;
 *   - `stream` is a CUDA stream handle (cudaStream_t / CUstream passed as void*); NULL is the
 *     legacy default stream.  Calls that take a stream only enqueue work on it;
 *   - feature matrices are dense, row-major, fp32, leading dimension F, 1 <= F <= 2^20;
 *   - rowptr/colptr are int64, vertex ids are int32 (n < 2^31), nnz < 2^31;
 *   - no call aborts, traps or waits without bound on the device;
 *   - a handle may be used from any thread, by one thread at a time; different handles are
 *     independent.  Calls on one handle that are queued on different streams are not ordered
 *     against each other by the library (source-blocked passes read what the previous launch
 *     of the same call wrote, so one call's launches all go to the stream it was given).
 */
#ifndef DG_H_
#define DG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DG_OK = 0,
  DG_ERR_INVALID_ARG = 1,     /* null pointer, negative size, aliasing, bad enum            */
  DG_ERR_UNSUPPORTED = 2,     /* a size beyond the limits stated above                      */
  DG_ERR_CUDA = 3,            /* a CUDA runtime call failed; dg_last_error() has its text   */
  DG_ERR_NOT_TRANSPOSED = 4,  /* backward pass or CSC query before dg_graph_transpose       */
  DG_ERR_WORKSPACE = 5,       /* csc_storage or scratch smaller than the workspace query    */
  DG_ERR_INVALID_GRAPH = 6    /* dg_graph_create or dg_graph_validate found a malformed CSR */
} dg_status_t;

/* Reducer of Table 1 ("sum"), and the sum divided by the in-degree (Section 5.1). */
typedef enum { DG_OP_SUM = 0, DG_OP_MEAN = 1 } dg_op_t;

typedef struct dg_graph* dg_graph_t;

/*
 * Graph ingest: records the CSR of A (Section 3.1: rows = destination vertices, column
 * indices = source vertices, any order inside a row, duplicates and self-loops allowed).
 *   n       number of vertices, 0 <= n < 2^31
 *   nnz     number of directed edges, 0 <= nnz < 2^31
 *   rowptr  device, n+1 entries, rowptr[0] = 0, non-decreasing, rowptr[n] = nnz
 *   colidx  device, nnz entries in [0, n)
 *   edge_w  device, nnz fp32 scalars (the edge feature of Eq. 1 reduced to one value per
 *           edge and broadcast over the F features), or NULL for the unary copy of Eq. 2
 * The handle BORROWS the three arrays: they must stay valid and unchanged until
 * dg_graph_destroy.  The call allocates a few small device arrays that it owns (the lists of
 * heavy rows and, for graphs with at least 64 edges per vertex, 17 int32 split pointers per
 * vertex for source blocking).  It waits for the whole device before it reads the arrays (so
 * they may have been produced on any stream) and again before it returns.
 * The arrays are checked here, in one streaming pass (rowptr[0] = 0, rowptr non-decreasing,
 * rowptr[n] = nnz, every colidx in [0, n)): the aggregation kernels index the feature matrix
 * with colidx without a range check, so a malformed CSR is refused with DG_ERR_INVALID_GRAPH
 * and no handle is made.  Arrays that are changed afterwards are the caller's responsibility;
 * dg_graph_validate repeats the check on request.
 */
dg_status_t dg_graph_create(int64_t n, int64_t nnz, const int64_t* rowptr,
                            const int32_t* colidx, const float* edge_w, dg_graph_t* out_graph);

/* Frees what dg_graph_create allocated.  The borrowed CSR and the caller's CSC storage are
 * not touched.  NULL is accepted. */
dg_status_t dg_graph_destroy(dg_graph_t g);

/* Synchronous check of the borrowed CSR on `stream`: rowptr[0] = 0, rowptr non-decreasing,
 * rowptr[n] = nnz, every colidx in [0, n).  Returns DG_ERR_INVALID_GRAPH if not. */
dg_status_t dg_graph_validate(dg_graph_t g, void* stream);

/* Sizes in bytes of the two device buffers dg_graph_transpose needs for this graph. */
dg_status_t dg_graph_transpose_workspace(dg_graph_t g, size_t* csc_bytes, size_t* scratch_bytes);

/*
 * CSR -> CSC on the GPU (the paper works on the CSR only and leaves this step implicit).
 * The result is the stable counting sort of the edge positions k = 0..nnz-1 by colidx[k]:
 *   colptr[u]   number of edges with source < u (int64, n+1 entries)
 *   perm[q]     CSR position of the q-th edge in (source, position) order (int32)
 *   rowidx_T[q] destination vertex of edge perm[q] (int32)
 *   w_T[q]      edge_w[perm[q]], copied bit for bit (absent when the graph is unweighted)
 * There is exactly one correct result; it is integer work and bit-exact.
 * Next to these the storage holds two internal arrays: the per-edge factor w_T[q]/deg(rowidx_T[q])
 * that the backward pass of the mean streams (deg + 1 when the graph attribute "self_loops" is
 * set at the time of this call), and (for graphs with at least 64 edges per vertex) the split
 * pointers of the CSC for source blocking.
 *   csc_storage  device, 256-byte aligned, >= csc_bytes; holds all these arrays, is borrowed
 *                by the handle until destroy (or the next transpose) and is what
 *                dg_graph_get_csc points into
 *   scratch      device, 256-byte aligned, >= scratch_bytes; free for reuse once the work
 *                enqueued on `stream` has finished
 * Asynchronous on `stream`.
 */
dg_status_t dg_graph_transpose(dg_graph_t g, void* csc_storage, size_t csc_bytes,
                               void* scratch, size_t scratch_bytes, void* stream);

/*
 * (The paper has no counterpart of this entry point; it exists for deployment reasons.)
 * dg_graph_transpose for callers that cannot provide scratch memory: a plug-in inside a host
 * program that has claimed the whole device for its own pool, a serving loop that must not hit
 * the device-wide synchronisation of cudaMalloc/cudaFree, an embedder that owns nothing but the
 * arrays it was handed.  The sort's scratch lives in an array of
 * DG_TRANSPOSE_STATIC_SCRATCH_BYTES bytes inside the library image: every GPU on which the
 * process loads the library holds that much from load to exit.  The call allocates and frees
 * nothing, neither directly nor through a library.
 *   - Same result, arguments and errors as dg_graph_transpose (csc_storage is still the
 *     caller's: it is an output), minus the scratch pair.
 *   - Limit: graphs whose scratch_bytes (dg_graph_transpose_workspace) exceed the array are
 *     rejected with DG_ERR_UNSUPPORTED and a message that states both sizes; that is a little
 *     under 1.4 million edges.
 *   - The first call on a device looks up the array's device address (the device must be
 *     current; the result is cached per device).  Make that first call before any stream
 *     capture begins.
 *   - All calls of a process on one device share the one array.  It keeps whatever the last
 *     call left, which is harmless (every part is rewritten before it is read), but two calls
 *     whose work overlaps on the GPU (different streams, or different threads) race on it and
 *     give wrong CSC arrays: serialise them.
 */
#define DG_TRANSPOSE_STATIC_SCRATCH_BYTES (16u << 20)
dg_status_t dg_graph_transpose_static(dg_graph_t g, void* csc_storage, size_t csc_bytes,
                                      void* stream);

/*
 * Learnable edge weights: after the caller has changed the values of edge_w in place (an
 * optimiser step on them, with the gradient of dg_aggregate_edge_grad), this call copies them
 * into the CSC again (w_T[q] = edge_w[perm[q]] and the mean's per-edge factors), so that the
 * backward pass uses the new weights.  The forward pass reads edge_w in place and needs nothing.
 * A no-op before dg_graph_transpose; DG_ERR_INVALID_ARG for an unweighted graph.
 * Asynchronous on `stream`.
 */
dg_status_t dg_graph_update_weights(dg_graph_t g, void* stream);

/* Device pointers to the CSC arrays inside csc_storage (any output pointer may be NULL).
 * *w_T is set to NULL for an unweighted graph. */
dg_status_t dg_graph_get_csc(dg_graph_t g, const int64_t** colptr, const int32_t** rowidx_T,
                             const float** w_T, const int32_t** perm);

/*
 * Forward AP (Algorithm 1 with the operators above):
 *   out[v][j] = s_v * sum over the CSR row of v of  w_k * H[colidx[k]][j],   0 <= j < F
 * w_k = edge_w[k] (1 if unweighted); s_v = 1 for DG_OP_SUM, 1/deg(v) for DG_OP_MEAN with
 * deg(v) = rowptr[v+1]-rowptr[v]; a vertex without in-edges gets zeros (the output of
 * Algorithm 1 starts at zero).
 *   H    device, n x F fp32 row-major, read only
 *   out  device, n x F fp32 row-major, OVERWRITTEN (no need to clear it); must not overlap H
 * With the graph attribute "self_loops" = 1 (dg_graph_set_param) every vertex counts as its own
 * in-neighbour with weight 1 without such edges being stored: H[v][j] joins the sum and the
 * mean divides by deg(v) + 1.  DG_OP_MEAN is then the GCN aggregator of GraphSAGE, Section 5.1
 * (Models and Parameters): (sum of the neighbours' rows + own row) / (in-degree + 1), in one
 * pass, without a second read and write of the n x F matrix.
 * fp32 accumulation in a fixed order: the same call on the same data gives the same bits.
 * Asynchronous on `stream`.
 */
dg_status_t dg_aggregate_fwd(dg_graph_t g, const float* H, int32_t F, dg_op_t op, float* out,
                             void* stream);

/*
 * Backward AP, the adjoint of dg_aggregate_fwd with the same (F, op):
 *   dH[u][j] = sum over the CSC segment of u of  w_T[q] * s_{v_q} * dOut[v_q][j],
 *   v_q = rowidx_T[q]
 * (the mean's 1/deg belongs to the destination vertex v_q).  Gathers over the CSC built by
 * dg_graph_transpose, without atomics, in a fixed order.  dH is OVERWRITTEN and must not
 * overlap dOut.  Returns DG_ERR_NOT_TRANSPOSED before dg_graph_transpose.
 * With "self_loops" = 1 the term s_u * dOut[u][j] joins the sum and s_v = 1/(deg(v) + 1) for
 * DG_OP_MEAN.  The mean's per-edge factors are tabulated by dg_graph_transpose: set
 * "self_loops" before it; DG_OP_MEAN returns DG_ERR_NOT_TRANSPOSED if the attribute has changed
 * since (DG_OP_SUM does not use the table).
 * Asynchronous on `stream`.
 */
dg_status_t dg_aggregate_bwd(dg_graph_t g, const float* dOut, int32_t F, dg_op_t op, float* dH,
                             void* stream);

/*
 * The same two passes with the gathered matrix stored as bf16 (two bytes per element, the
 * upper half of an fp32; the paper's Conclusion names reduced precision as future work).  Every
 * gathered byte is halved; products and sums are fp32 (a bf16 value converts to fp32 exactly)
 * and the output is fp32, so the result equals the fp32 entry point's on the same values and
 * the same error bound holds.  F must be even (16-byte loads need F % 8 == 0 and a 16-byte
 * aligned H; narrower loads are used otherwise); DG_ERR_UNSUPPORTED for an odd F.
 */
dg_status_t dg_aggregate_fwd_bf16(dg_graph_t g, const uint16_t* H, int32_t F, dg_op_t op,
                                  float* out, void* stream);
dg_status_t dg_aggregate_bwd_bf16(dg_graph_t g, const uint16_t* dOut, int32_t F, dg_op_t op,
                                  float* dH, void* stream);

/*
 * Forward and backward AP with the feature matrices in HOST memory (pinned memory makes the
 * copies asynchronous and lets them overlap the kernels; pageable memory works but serialises).
 * Computes what dg_aggregate_fwd on H_host and dg_aggregate_bwd on dOut_host compute and leaves
 * the results in out_host and dH_host.  The feature columns are independent in AP, so matrices
 * wider than 256 columns travel in chunks of 128 columns: a chunk is uploaded while the previous
 * one is aggregated and the one before that is downloaded, on two helper streams the handle
 * creates at its first call of this function.  (The summation order inside an output element
 * can therefore differ from a full-width call; both are within the stated error bound.)
 * Everything is ordered after the work already queued on `stream`, and `stream` finishing means
 * all copies are done.  dOut_host/dH_host may both be NULL to run the forward pass only.
 *   device_ws  device, 256-byte aligned, >= dg_aggregate_host_workspace(g, F) bytes (four
 *              n x F matrices at most)
 */
size_t dg_aggregate_host_workspace(dg_graph_t g, int32_t F);
dg_status_t dg_aggregate_host(dg_graph_t g, const float* H_host, const float* dOut_host,
                              int32_t F, dg_op_t op, float* out_host, float* dH_host,
                              void* device_ws, size_t device_ws_bytes, void* stream);

/*
 * Vertex reordering as graph pre-processing: the same graph with its vertices renamed, so that
 * the rows of the feature matrix that the aggregation gathers most often form one contiguous
 * range (the GPU counterpart of the per-block CSRs the paper builds for its cache blocking,
 * Section 3.2; Table 3 there measures the cache reuse such a layout can exploit).
 *   order   DG_ORDER_OUT_DEGREE  hub-first by the number of edges a vertex is the source of
 *                                (the rows the forward pass gathers most), largest first, equal
 *                                counts by ascending old id
 *           DG_ORDER_IN_DEGREE   the same by in-degree (the rows the backward pass gathers most)
 *           DG_ORDER_GIVEN       the caller's permutation (from a clustering or partitioning
 *                                tool, or community labels it already has)
 *   given_new_of_old  device, n int32, a permutation of 0..n-1 (DG_ORDER_GIVEN only; checked:
 *                     DG_ERR_INVALID_ARG if it is not one)
 * The result is exact integer work with one correct answer: old vertex v becomes new_of_old[v];
 * new row new_of_old[v] holds the entries of old row v with every source u replaced by
 * new_of_old[u], sorted by new source id, duplicate edges in the order of their old positions;
 * weights follow their edges bit for bit.  Aggregating the renamed features on the renamed graph
 * gives the renamed result: AP'(P H) = P AP(H).
 *   storage  device, 256-byte aligned, >= storage_bytes: receives new_of_old, the new rowptr,
 *            colidx, edge_w and pos (pos[k'] = old CSR position of new position k', the order an
 *            edge-feature matrix must be permuted into); borrowed by the new handle until it is
 *            destroyed
 *   scratch  device, 256-byte aligned, >= scratch_bytes; free again when the call returns
 *   out_graph  a new handle over the renamed CSR (the attribute "self_loops" is carried over,
 *            tuning knobs are not); the old handle stays valid and independent
 * Synchronous (it ends like dg_graph_create).  dg_graph_get_order returns device pointers into
 * `storage` (any output pointer may be NULL); dg_permute_rows renames the rows of a feature
 * matrix: out[new_of_old[v]] = in[v] (to_old = 0), or out[v] = in[new_of_old[v]] (to_old = 1,
 * results back in the old numbering); not in place.
 */
typedef enum { DG_ORDER_GIVEN = 0, DG_ORDER_OUT_DEGREE = 1, DG_ORDER_IN_DEGREE = 2 } dg_order_t;
dg_status_t dg_graph_reorder_workspace(dg_graph_t g, size_t* storage_bytes, size_t* scratch_bytes);
dg_status_t dg_graph_reorder(dg_graph_t g, dg_order_t order, const int32_t* given_new_of_old,
                             void* storage, size_t storage_bytes, void* scratch,
                             size_t scratch_bytes, void* stream, dg_graph_t* out_graph);
dg_status_t dg_graph_get_order(dg_graph_t reordered, const int32_t** new_of_old,
                               const int64_t** rowptr, const int32_t** colidx,
                               const float** edge_w, const int32_t** pos);
dg_status_t dg_permute_rows(const int32_t* new_of_old, int64_t n, int32_t F, const float* in,
                            float* out, int to_old, void* stream);

/*
 * The general aggregation primitive: every operator pair of Table 1 of the paper,
 *   fO[v][j] = (+) over the CSR row of v of  ( fV[colidx[k]][j] (x) fE[k][j] ),   0 <= j < F
 * (Eq. 1; with one operand absent the unary copy of Eq. 2), in the pull form of Algorithm 1.
 *   binary  (x): copylhs (the vertex feature alone), copyrhs (the edge feature alone), add, sub,
 *           mul, div, with x = the source vertex's feature and y = the edge's feature
 *   reduce  (+): sum, max, min
 *   fV      device, n x F fp32 row-major; may be NULL for copyrhs
 *   fE      device, nnz x fE_cols fp32 row-major, row k belongs to the edge at CSR position k;
 *           fE_cols is F (the |E| x d edge features of Section 2.1) or 1 (one scalar per edge,
 *           broadcast over the features); may be NULL for copylhs.  The edge_w given to
 *           dg_graph_create plays no part in these calls.
 *   fO      device, n x F fp32, OVERWRITTEN
 *   arg     device, n x F int32, or NULL; written for max / min only: the CSR position of the
 *           edge whose message is the extremum
 * The paper does not say what max / min do on a vertex without in-edges, nor how ties are
 * resolved.  Here the extremum runs over the messages of the row only (the zero the output of
 * Algorithm 1 starts from is not a candidate), a vertex without in-edges gets 0 and arg = -1,
 * and among equal messages the one at the lowest edge position wins.  A message is one fp32
 * IEEE operation on the two fp32 operands, so the result of max / min is exact and the same on
 * every run; sums are fp32 in a fixed order.
 * Where fV does not fit the handle's L2 budget and the rows are long and sorted, the call runs
 * as one launch per (range of source ids, slice of 128 features) as the sum / mean calls do
 * (attributes "l2_budget_mb", "source_blocks"); each launch folds its piece into fO, for max /
 * min through arg, so a caller who passes arg = NULL gets feature slices only.  fO and arg must
 * not overlap the inputs.  copylhs / sum and mul / sum with fE_cols = 1 are the plain and the
 * weighted sum: these two pairs run on the kernels of dg_aggregate_fwd (fE as the weights).
 * Asynchronous on `stream`.
 */
typedef enum {
  DG_BIN_COPY_LHS = 0, DG_BIN_COPY_RHS = 1, DG_BIN_ADD = 2, DG_BIN_SUB = 3, DG_BIN_MUL = 4,
  DG_BIN_DIV = 5
} dg_binary_t;
typedef enum { DG_RED_SUM = 0, DG_RED_MAX = 1, DG_RED_MIN = 2 } dg_reduce_t;

dg_status_t dg_ap_fwd(dg_graph_t g, const float* fV, const float* fE, int32_t fE_cols, int32_t F,
                      dg_binary_t binary, dg_reduce_t reduce, float* fO, int32_t* arg,
                      void* stream);

/*
 * Gradients of <dg_ap_fwd(fV, fE), dO> (the paper writes no backward pass; this is calculus on
 * the definition above).  With sel(k, j) = 1 for sum and [arg[v_k][j] == k] for max / min:
 *   dV[u][j] = sum over the edges k out of u of  sel * dO[v_k][j] * d(x (x) y)/dx
 *   dE[k][j] =                                   sel * dO[v_k][j] * d(x (x) y)/dy
 * (dE summed over j when fE_cols is 1: for mul / sum that is the sampled dense-dense product
 * <fV[u_k], dO[v_k]> of Section 2.2).  The sum for dV is a gather over the CSC with an equality
 * test on arg, without atomics and in a fixed order, so it needs dg_graph_transpose first
 * (DG_ERR_NOT_TRANSPOSED otherwise).
 *   dO       device, n x F
 *   fV, fE   the operands of the forward call (those the derivative needs must be given)
 *   arg      the forward call's arg output; required for max / min
 *   dV       device, n x F, OVERWRITTEN; NULL to skip (all zeros for copyrhs)
 *   dE       device, nnz x fE_cols, OVERWRITTEN; NULL to skip; must be NULL for copylhs
 * Asynchronous on `stream`.
 */
dg_status_t dg_ap_bwd(dg_graph_t g, const float* dO, const float* fV, const float* fE,
                      int32_t fE_cols, int32_t F, dg_binary_t binary, dg_reduce_t reduce,
                      const int32_t* arg, float* dV, float* dE, void* stream);

/*
 * Gradient of <dg_aggregate_fwd(H), dOut> with respect to the scalar edge weights (message
 * passing onto edges, Section 2.2: one sampled dot product per edge):
 *   dW[k] = s_v * sum_j H[colidx[k]][j] * dOut[v][j]      for the edge at CSR position k into v
 * s_v = 1 for DG_OP_SUM, 1/deg(v) for DG_OP_MEAN (deg(v) + 1 with "self_loops"; the implicit
 * loops carry no weight and get no gradient).  Works on the CSR alone; the graph's own weights
 * do not enter (the sum is linear in them).
 *   H, dOut  device, n x F;   dW  device, nnz fp32, OVERWRITTEN
 * Asynchronous on `stream`.
 */
dg_status_t dg_aggregate_edge_grad(dg_graph_t g, const float* H, const float* dOut, int32_t F,
                                   dg_op_t op, float* dW, void* stream);

/*
 * Tuning knobs (defaults come from the device's L2 size and SM count):
 *   "heavy_threshold"  rows longer than this are summed by a whole thread block
 *   "heavy_blocks_per_sm"  thread blocks per SM that walk the list of heavy rows (longest first)
 *                      before the launch turns to the light rows; 0 = as many as are resident
 *   "slice_features"   features per pass over the graph (0 = choose from the L2 size; a value
 *                      that would need more than 65535 passes is widened)
 *   "rows_per_block"   destination rows per thread block in the light-row kernel (1..248,
 *                      rounded up to a multiple of 8: each of the 8 warps owns a run of rows;
 *                      0 = about 1024 edges per warp, between 32 and 248 rows per block)
 *   "l2_budget_mb"     MiB of the gathered matrix one launch may keep L2-resident
 *   "source_blocks"    number of source-vertex ranges the pass is cut into, one launch each
 *                      (the blocking of Algorithm 2; 0 = choose from the L2 budget, else 1, 2,
 *                      4, 8 or 16; ignored for graphs without split pointers, i.e. with fewer
 *                      than 64 edges per vertex or unsorted rows)
 * Graph attribute (not a tuning knob: it changes the result):
 *   "self_loops"       0 (default) or 1: every vertex is its own in-neighbour with weight 1, see
 *                      dg_aggregate_fwd / dg_aggregate_bwd; set it before dg_graph_transpose
 * Changing "heavy_threshold" waits for the whole device, rebuilds the heavy lists and waits
 * again: a rare, synchronous call.
 * Returns DG_ERR_INVALID_ARG for an unknown name or a value out of range.
 */
dg_status_t dg_graph_set_param(dg_graph_t g, const char* name, int64_t value);
dg_status_t dg_graph_get_param(dg_graph_t g, const char* name, int64_t* value);

/*
 * Diagnostic: gathers `count` rows table[idx[i]] (rows of row_floats fp32, a power of two in
 * [4, 128]; idx values in [0, rows)) and sums them per warp, 512 gathers per warp, with the
 * load pattern of the aggregation kernels and nothing else.  Timed by the caller, it gives the
 * rate at which this GPU delivers gathered rows from L2 (small table) or from HBM (table far
 * larger than L2): the ceilings the aggregation rates are compared with.
 *   table  device, rows x row_floats fp32, 16-byte aligned
 *   idx    device, count int32
 *   sink   device, 16-byte aligned, >= ceil(count / 512) * 128 floats; receives the warp sums
 * Asynchronous on `stream`.
 */
dg_status_t dg_probe_gather(const float* table, int64_t rows, int32_t row_floats,
                            const int32_t* idx, int64_t count, float* sink, void* stream);

/*
 * Diagnostic: the same gather served from SHARED memory.  Every thread block (1024 threads) fills a
 * stage of stage_rows rows of row_floats fp32 (row r holds the value r everywhere; the stage
 * must fit 200 KiB), then each warp gathers 4096 rows named by idx (values in [0, stage_rows),
 * clamped) and sums them.  remote = 1 runs the blocks as clusters of two and reads every row
 * from the partner block's stage (distributed shared memory).  Timed by the caller, it says what
 * staging a block of the gathered matrix on chip could deliver, next to the L2 figure of
 * dg_probe_gather.
 *   idx   device, count int32;   sink  device, 16-byte aligned, >= ceil(count / 4096) * 128 floats
 * Asynchronous on `stream`.
 */
dg_status_t dg_probe_gather_smem(int32_t row_floats, int32_t stage_rows, const int32_t* idx,
                                 int64_t count, float* sink, int32_t remote, void* stream);

/* Number of kernels the library has launched from this process (all handles, all threads). */
int64_t dg_kernel_launch_count(void);

/* Message of the last failure on this thread ("" if none).  Valid until the next failing call
 * on the same thread. */
const char* dg_last_error(void);

/* "libdgagg <version> sm_100a". */
const char* dg_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DG_H_ */
