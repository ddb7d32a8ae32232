/*
 * CPU oracle for the aggregation primitive (AP).  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain definition of what the CUDA library must compute.  It is slow on
 * purpose, accumulates in fp64, and shares no code, header, table or helper with the CUDA
 * path.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * What it follows:
 *   - Forward AP: the pull loop of Algorithm 1 of the paper (Section 3.1), with the binary
 *     operator of Eq. 1 taken as "multiply the source row by one scalar edge weight" or the
 *     unary copy of Eq. 2, and the reducer "sum" (Table 1).  "mean" is that sum divided by the
 *     in-degree, the post-processing named in Section 5.1 (Models and Parameters).
 *   - The GCN aggregator of GraphSAGE (Section 5.1, Models and Parameters) adds the vertex's
 *     own row to the sum of its neighbours' rows and divides by in-degree + 1.  Here that is the
 *     `self_loops` switch: every vertex v counts as its own in-neighbour with weight 1, so that
 *     "mean" becomes (sum_{u in N(v)} w h_u + h_v) / (deg(v) + 1) and "sum" the numerator alone.
 *   - The matrix A is CSR with rows = destination vertices and column indices = source
 *     vertices (Section 3.1: A[v] lists the vertices with an edge incident on v).
 *   - The paper never writes the backward pass or the CSR->CSC build.  They are defined here
 *     from calculus (dH = A^T dOut, with the mean's 1/deg belonging to the destination row)
 *     and as a stable counting sort of edge positions by source vertex.
 *
 * Parity pins (tests/test_oracle_pins.py): dense fp64 A*H on graphs with <= 64 vertices,
 * closed-form graphs (identity, ring, star, complete, all-ones features), the column-sum
 * invariant, the adjoint identity <AP(H),G> = <H,AP^T(G)>, (A^T)^T = A, an O(n^2) brute-force
 * transpose, and scipy.sparse as a third party; for `self_loops`, the same operators on the
 * graph with the edges v -> v written out, and constant features (every vertex keeps the
 * constant).  Every function below has at least one pin.
 *
 * The loop over destination vertices is the paper's own parallel loop ("for v in V in
 * parallel", Algorithm 1) with the dynamic chunked schedule of Section 3.2 (Multithreading).
 * Nothing else of Section 3.2 (blocking, loop reordering) is applied.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OP_SUM 0
#define ORACLE_OP_MEAN 1

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int t) {
#ifdef _OPENMP
  if (t > 0) omp_set_num_threads(t);
#else
  (void)t;
#endif
}

/*
 * Forward AP (Algorithm 1).  For every requested destination vertex v:
 *   ref[v][j] = s_v * sum_{k in row v} w_k * H[colidx[k]][j]
 *   mag[v][j] = s_v * sum_{k in row v} |w_k * H[colidx[k]][j]|
 * w_k = edge_w[k] (1 when edge_w is NULL); s_v = 1 for sum, 1/deg(v) for mean (0 if deg = 0).
 * With self_loops != 0 the term H[v][j] joins both sums and the mean divides by deg(v) + 1.
 * rows == NULL means all n rows in order (nrows is then ignored); otherwise output row i
 * belongs to vertex rows[i].  ref and mag are (count x F) row-major doubles.
 * Returns 0, or 1 on an invalid argument.
 */
int oracle_ap_forward(int64_t n, const int64_t* rowptr, const int32_t* colidx,
                      const float* edge_w, const float* H, int32_t F, int op, int self_loops,
                      const int64_t* rows, int64_t nrows, double* ref, double* mag) {
  if (n < 0 || F < 1 || (op != ORACLE_OP_SUM && op != ORACLE_OP_MEAN)) return 1;
  const int64_t count = rows ? nrows : n;
#pragma omp parallel for schedule(dynamic, 64)
  for (int64_t i = 0; i < count; ++i) {
    const int64_t v = rows ? rows[i] : i;
    double* acc = ref + i * (int64_t)F;
    double* am = mag + i * (int64_t)F;
    for (int32_t j = 0; j < F; ++j) { acc[j] = 0.0; am[j] = 0.0; }
    const int64_t lo = rowptr[v], hi = rowptr[v + 1];
    for (int64_t k = lo; k < hi; ++k) {
      const int64_t u = colidx[k];
      const double w = edge_w ? (double)edge_w[k] : 1.0;
      const float* hu = H + u * (int64_t)F;
      for (int32_t j = 0; j < F; ++j) {
        const double t = w * (double)hu[j];
        acc[j] += t;
        am[j] += fabs(t);
      }
    }
    if (self_loops) {
      const float* hv = H + v * (int64_t)F;
      for (int32_t j = 0; j < F; ++j) {
        acc[j] += (double)hv[j];
        am[j] += fabs((double)hv[j]);
      }
    }
    if (op == ORACLE_OP_MEAN) {
      const int64_t deg = hi - lo + (self_loops ? 1 : 0);
      const double s = deg > 0 ? 1.0 / (double)deg : 0.0;
      for (int32_t j = 0; j < F; ++j) { acc[j] *= s; am[j] *= s; }
    }
  }
  return 0;
}

/*
 * CSR -> CSC as a stable counting sort of the edge positions k = 0..nnz-1 by key colidx[k].
 *   colptr[u]   = number of edges whose source is < u          (n+1 entries, colptr[n] = nnz)
 *   perm[q]     = position in the CSR of the q-th edge in (source, position) order
 *   rowidx_T[q] = destination vertex (CSR row) of edge perm[q]
 *   w_T[q]      = edge_w[perm[q]] copied bit for bit (skipped when edge_w is NULL)
 * Serial on purpose: walking the CSR in position order makes the fill stable by construction.
 * Returns 0, 1 on an invalid argument, 2 when memory runs out.
 */
int oracle_transpose(int64_t n, int64_t nnz, const int64_t* rowptr, const int32_t* colidx,
                     const float* edge_w, int64_t* colptr, int32_t* rowidx_T, float* w_T,
                     int64_t* perm) {
  if (n < 0 || nnz < 0) return 1;
  for (int64_t u = 0; u <= n; ++u) colptr[u] = 0;
  for (int64_t k = 0; k < nnz; ++k) {
    const int64_t u = colidx[k];
    if (u < 0 || u >= n) return 1;
    colptr[u + 1] += 1;
  }
  for (int64_t u = 0; u < n; ++u) colptr[u + 1] += colptr[u];
  int64_t* cursor = (int64_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(int64_t));
  if (!cursor) return 2;
  for (int64_t u = 0; u < n; ++u) cursor[u] = colptr[u];
  for (int64_t v = 0; v < n; ++v) {
    for (int64_t k = rowptr[v]; k < rowptr[v + 1]; ++k) {
      const int64_t q = cursor[colidx[k]]++;
      perm[q] = k;
      rowidx_T[q] = (int32_t)v;
      if (edge_w) memcpy(&w_T[q], &edge_w[k], sizeof(float));
    }
  }
  free(cursor);
  return 0;
}

/*
 * Backward AP: dH = A^T dOut, the adjoint of oracle_ap_forward.  For every requested source
 * vertex u, with q running over the CSC segment of u and v_q = rowidx_T[q]:
 *   ref[u][j] = sum_q  w_T[q] * s_{v_q} * dOut[v_q][j],   mag likewise with absolute values
 * s_v = 1 for sum, 1/deg(v) for mean, deg(v) = rowptr[v+1]-rowptr[v] taken from the CSR
 * (the divisor of the forward mean belongs to the destination vertex, not to the source).
 * With self_loops != 0 the divisor is deg(v) + 1 and the term s_u * dOut[u][j] joins the sum:
 * u is then a destination of itself, with weight 1.
 * cols == NULL means all n vertices in order.
 */
int oracle_ap_backward(int64_t n, const int64_t* rowptr, const int64_t* colptr,
                       const int32_t* rowidx_T, const float* w_T, const float* dOut, int32_t F,
                       int op, int self_loops, const int64_t* cols, int64_t ncols, double* ref,
                       double* mag) {
  if (n < 0 || F < 1 || (op != ORACLE_OP_SUM && op != ORACLE_OP_MEAN)) return 1;
  const int64_t count = cols ? ncols : n;
#pragma omp parallel for schedule(dynamic, 64)
  for (int64_t i = 0; i < count; ++i) {
    const int64_t u = cols ? cols[i] : i;
    double* acc = ref + i * (int64_t)F;
    double* am = mag + i * (int64_t)F;
    for (int32_t j = 0; j < F; ++j) { acc[j] = 0.0; am[j] = 0.0; }
    for (int64_t q = colptr[u]; q < colptr[u + 1]; ++q) {
      const int64_t v = rowidx_T[q];
      double s = w_T ? (double)w_T[q] : 1.0;
      if (op == ORACLE_OP_MEAN) {
        const int64_t deg = rowptr[v + 1] - rowptr[v] + (self_loops ? 1 : 0);
        s *= deg > 0 ? 1.0 / (double)deg : 0.0;
      }
      const float* gv = dOut + v * (int64_t)F;
      for (int32_t j = 0; j < F; ++j) {
        const double t = s * (double)gv[j];
        acc[j] += t;
        am[j] += fabs(t);
      }
    }
    if (self_loops) {
      double s = 1.0;
      if (op == ORACLE_OP_MEAN) s = 1.0 / (double)(rowptr[u + 1] - rowptr[u] + 1);
      const float* gu = dOut + u * (int64_t)F;
      for (int32_t j = 0; j < F; ++j) {
        const double t = s * (double)gu[j];
        acc[j] += t;
        am[j] += fabs(t);
      }
    }
  }
  return 0;
}
