/*
 * CPU oracle, second part: the general aggregation primitive, its gradients, the gradient with
 * respect to scalar edge weights, and vertex relabelling.  TEST INFRASTRUCTURE ONLY.
 *
 * Like ap_oracle.c this file is the plain definition of what the CUDA library must compute: slow
 * on purpose, no blocking, no code shared with the CUDA path.  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may load it.
 *
 * What it follows:
 *   - The general AP of Section 2.1 of the paper, Eq. 1 and Eq. 2, in the pull loop of
 *     Algorithm 1 (Section 3.1):  f_O[v] = (+)_{edges e_uv into v} ( f_V[u] (x) f_E[e_uv] ),
 *     element-wise over the d features, with the operators of Table 1:
 *       (x) in {add, sub, mul, div} on (x, y) = (f_V[u], f_E[e]), copylhs (x alone, Eq. 2),
 *           copyrhs (y alone);
 *       (+) in {sum, max, min}.
 *     f_E is |E| x d (Section 2.1); a |E| x 1 matrix is broadcast over the features (the scalar
 *     edge weight of the other entry points).
 *   - Readings where the paper is silent: max and min run over the messages of the row only (the
 *     zero the output starts from in Algorithm 1 is not a candidate); a vertex without in-edges
 *     gets 0; among equal extremal messages the one at the LOWEST edge position is the arg.  The
 *     message of max/min is formed in fp32 (one IEEE operation on the fp32 inputs), because the
 *     choice of the extremum is a discrete decision that both sides must take in the same
 *     precision; the result is then one of those fp32 messages, exactly.  For sum the messages
 *     and their sum are fp64.
 *   - The gradients are calculus on that definition (the paper writes no backward pass):
 *       dV[u][j] = sum over edges k out of u of  sel(k,j) * dO[v_k][j] * d(x (x) y)/dx
 *       dE[k][j] =                               sel(k,j) * dO[v_k][j] * d(x (x) y)/dy
 *     (summed over j when f_E has one column), sel = 1 for sum and [arg[v_k][j] == k] for
 *     max/min.
 *   - Gradient with respect to scalar edge weights of the weighted sum / mean of ap_oracle.c
 *     (message passing onto edges, Section 2.2: the sampled dense-dense product):
 *       dW[k] = s_v * <H[u_k], dOut[v_k]>,  s_v as in oracle_ap_forward.
 *   - Relabelling: given new_of_old, the CSR of P A P^T with every row sorted by new source id
 *     (ties, i.e. duplicate edges, by old position).  The paper's counterpart is the
 *     pre-processing that makes its cache blocks effective (Section 3.2); the definition here is
 *     just "the same graph with the vertices renamed".
 *   - Hub-first order: vertices by degree, largest first, ties by ascending id.
 *
 * Parity pins (tests/test_oracle_general_pins.py): brute-force dense evaluation of every
 * operator pair on tiny graphs written with numpy masks; reductions to the pinned
 * oracle_ap_forward (mul/sum with one column = weighted sum, copylhs/sum = plain sum);
 * algebraic identities (add/sum = A X + row sums of Y, min = -max of negated inputs, copyrhs/sum
 * = segment sums); directional derivatives of <AP(X, Y), G> for the gradients (exact for the
 * bilinear cases, finite differences otherwise); linearity in w for the edge-weight gradient;
 * P A P^T on dense tiny graphs and AP(relabelled)(P H) = P AP(H) for the relabelling.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { BIN_COPY_LHS = 0, BIN_COPY_RHS = 1, BIN_ADD = 2, BIN_SUB = 3, BIN_MUL = 4, BIN_DIV = 5 };
enum { RED_SUM = 0, RED_MAX = 1, RED_MIN = 2 };

static int ops_valid(int bin, int red) {
  return bin >= BIN_COPY_LHS && bin <= BIN_DIV && red >= RED_SUM && red <= RED_MIN;
}

/* x (x) y in fp64 (exact inputs, one fp64 rounding) */
static double message_f64(int bin, double x, double y) {
  switch (bin) {
    case BIN_COPY_LHS: return x;
    case BIN_COPY_RHS: return y;
    case BIN_ADD: return x + y;
    case BIN_SUB: return x - y;
    case BIN_MUL: return x * y;
    default: return x / y;
  }
}

/* x (x) y as one fp32 IEEE operation */
static float message_f32(int bin, float x, float y) {
  volatile float r;
  switch (bin) {
    case BIN_COPY_LHS: r = x; break;
    case BIN_COPY_RHS: r = y; break;
    case BIN_ADD: r = x + y; break;
    case BIN_SUB: r = x - y; break;
    case BIN_MUL: r = x * y; break;
    default: r = x / y; break;
  }
  return r;
}

static double d_message_dx(int bin, double x, double y) {
  (void)x;
  switch (bin) {
    case BIN_COPY_LHS: case BIN_ADD: case BIN_SUB: return 1.0;
    case BIN_COPY_RHS: return 0.0;
    case BIN_MUL: return y;
    default: return 1.0 / y;
  }
}

static double d_message_dy(int bin, double x, double y) {
  switch (bin) {
    case BIN_COPY_RHS: case BIN_ADD: return 1.0;
    case BIN_COPY_LHS: return 0.0;
    case BIN_SUB: return -1.0;
    case BIN_MUL: return x;
    default: return -x / (y * y);
  }
}

/*
 * General forward AP.  For every destination v and feature j:
 *   sum:      ref[v][j] = sum_k m_k,  mag[v][j] = sum_k |m_k|,  m_k = x_k (x) y_k in fp64
 *   max/min:  ref[v][j] = the extremal fp32 message, arg[v][j] = its edge position (lowest
 *             among equals), mag[v][j] = |ref|; empty row: ref = 0, arg = -1
 * x_k = fV[colidx[k]][j] (ignored for copyrhs, fV may be NULL); y_k = fE[k][j], or fE[k][0] when
 * fE_cols == 1 (ignored for copylhs, fE may be NULL).  arg may be NULL.
 * Returns 0, or 1 on an invalid argument.
 */
int oracle_general_forward(int64_t n, const int64_t* rowptr, const int32_t* colidx,
                           const float* fV, const float* fE, int32_t fE_cols, int32_t F, int bin,
                           int red, double* ref, double* mag, int64_t* arg) {
  if (n < 0 || F < 1 || !ops_valid(bin, red)) return 1;
  if (bin != BIN_COPY_LHS && (!fE || (fE_cols != 1 && fE_cols != F))) return 1;
  if (bin != BIN_COPY_RHS && !fV) return 1;
#pragma omp parallel for schedule(dynamic, 64)
  for (int64_t v = 0; v < n; ++v) {
    for (int32_t j = 0; j < F; ++j) {
      double acc = 0.0, am = 0.0;
      float best = 0.0f;
      int64_t best_k = -1;
      for (int64_t k = rowptr[v]; k < rowptr[v + 1]; ++k) {
        const float x = bin != BIN_COPY_RHS ? fV[(int64_t)colidx[k] * F + j] : 0.0f;
        const float y = bin != BIN_COPY_LHS ? fE[k * (int64_t)fE_cols + (fE_cols == 1 ? 0 : j)] : 0.0f;
        if (red == RED_SUM) {
          const double m = message_f64(bin, (double)x, (double)y);
          acc += m;
          am += fabs(m);
        } else {
          const float m = message_f32(bin, x, y);
          if (best_k < 0 || (red == RED_MAX ? m > best : m < best)) {
            best = m;
            best_k = k;
          }
        }
      }
      if (red != RED_SUM) {
        acc = best_k >= 0 ? (double)best : 0.0;
        am = fabs(acc);
      }
      ref[v * (int64_t)F + j] = acc;
      mag[v * (int64_t)F + j] = am;
      if (arg) arg[v * (int64_t)F + j] = red == RED_SUM ? -1 : best_k;
    }
  }
  return 0;
}

/*
 * Gradients of the general AP.  Walks the edges in CSR order (serial: the sum into dV[u] is a
 * scatter) and adds, for edge k = (u -> v) and feature j with sel(k,j) != 0,
 *   dV[u][j]  += dO[v][j] * d(x (x) y)/dx        magV likewise with absolute values
 *   dE[k][jj] += dO[v][j] * d(x (x) y)/dy        magE likewise; jj = j, or 0 when fE_cols == 1
 * sel = 1 for sum, [arg[v][j] == k] for max/min (arg as returned by oracle_general_forward).
 * dV/magV are n x F, dE/magE are nnz x fE_cols; either pair may be NULL.
 */
int oracle_general_backward(int64_t n, const int64_t* rowptr, const int32_t* colidx,
                            const float* fV, const float* fE, int32_t fE_cols, int32_t F, int bin,
                            int red, const int64_t* arg, const float* dO, double* dV,
                            double* magV, double* dE, double* magE) {
  if (n < 0 || F < 1 || !ops_valid(bin, red) || !dO) return 1;
  if (red != RED_SUM && !arg) return 1;
  if (bin != BIN_COPY_LHS && (!fE || (fE_cols != 1 && fE_cols != F))) return 1;
  if (bin != BIN_COPY_RHS && !fV) return 1;
  if (dE && bin == BIN_COPY_LHS) return 1; /* no edge operand to differentiate */
  const int64_t nnz = rowptr[n];
  if (dV) for (int64_t i = 0; i < n * (int64_t)F; ++i) { dV[i] = 0.0; magV[i] = 0.0; }
  if (dE) for (int64_t i = 0; i < nnz * (int64_t)fE_cols; ++i) { dE[i] = 0.0; magE[i] = 0.0; }
  for (int64_t v = 0; v < n; ++v) {
    for (int64_t k = rowptr[v]; k < rowptr[v + 1]; ++k) {
      const int64_t u = colidx[k];
      for (int32_t j = 0; j < F; ++j) {
        if (red != RED_SUM && arg[v * (int64_t)F + j] != k) continue;
        const double x = bin != BIN_COPY_RHS ? (double)fV[u * (int64_t)F + j] : 0.0;
        const int64_t ej = k * (int64_t)fE_cols + (fE_cols == 1 ? 0 : j);
        const double y = bin != BIN_COPY_LHS ? (double)fE[ej] : 0.0;
        const double g = (double)dO[v * (int64_t)F + j];
        if (dV) {
          const double t = g * d_message_dx(bin, x, y);
          dV[u * (int64_t)F + j] += t;
          magV[u * (int64_t)F + j] += fabs(t);
        }
        if (dE) {
          const double t = g * d_message_dy(bin, x, y);
          dE[ej] += t;
          magE[ej] += fabs(t);
        }
      }
    }
  }
  return 0;
}

/*
 * Gradient of <AP(H), dOut> with respect to the scalar edge weights of the weighted sum / mean
 * (oracle_ap_forward of ap_oracle.c): for the edge at CSR position k, from u = colidx[k] into v,
 *   dW[k]  = s_v * sum_j H[u][j] * dOut[v][j],   mag[k] = s_v * sum_j |H[u][j] * dOut[v][j]|
 * s_v = 1 for sum (op 0); 1 / deg(v) for mean (op 1), deg(v) + 1 with self_loops.
 */
int oracle_edge_weight_grad(int64_t n, const int64_t* rowptr, const int32_t* colidx,
                            const float* H, const float* dOut, int32_t F, int op, int self_loops,
                            double* dW, double* mag) {
  if (n < 0 || F < 1 || (op != 0 && op != 1)) return 1;
#pragma omp parallel for schedule(dynamic, 64)
  for (int64_t v = 0; v < n; ++v) {
    const int64_t deg = rowptr[v + 1] - rowptr[v] + (self_loops ? 1 : 0);
    const double s = op == 1 ? (deg > 0 ? 1.0 / (double)deg : 0.0) : 1.0;
    for (int64_t k = rowptr[v]; k < rowptr[v + 1]; ++k) {
      const float* hu = H + (int64_t)colidx[k] * F;
      const float* gv = dOut + v * (int64_t)F;
      double acc = 0.0, am = 0.0;
      for (int32_t j = 0; j < F; ++j) {
        const double t = (double)hu[j] * (double)gv[j];
        acc += t;
        am += fabs(t);
      }
      dW[k] = s * acc;
      mag[k] = s * am;
    }
  }
  return 0;
}

/*
 * new_of_old for the hub-first order: vertices sorted by degree[v], largest first, equal degrees
 * by ascending old id; the vertex in place i of that order gets the new id i.
 * Written as a counting sort over the degree values (stable by construction).
 */
int oracle_order_by_degree(int64_t n, const int64_t* degree, int32_t* new_of_old) {
  if (n < 0) return 1;
  int64_t dmax = 0;
  for (int64_t v = 0; v < n; ++v) {
    if (degree[v] < 0) return 1;
    if (degree[v] > dmax) dmax = degree[v];
  }
  int64_t* start = (int64_t*)calloc((size_t)dmax + 2, sizeof(int64_t));
  if (!start) return 2;
  /* start[d] = number of vertices with a degree larger than d */
  for (int64_t v = 0; v < n; ++v) start[degree[v]] += 1;
  int64_t run = 0;
  for (int64_t d = dmax; d >= 0; --d) {
    const int64_t c = start[d];
    start[d] = run;
    run += c;
  }
  for (int64_t v = 0; v < n; ++v) new_of_old[v] = (int32_t)(start[degree[v]]++);
  free(start);
  return 0;
}

typedef struct { int32_t src; int64_t pos; } relabel_entry;

static int relabel_cmp(const void* a, const void* b) {
  const relabel_entry* x = (const relabel_entry*)a;
  const relabel_entry* y = (const relabel_entry*)b;
  if (x->src != y->src) return x->src < y->src ? -1 : 1;
  return x->pos < y->pos ? -1 : (x->pos > y->pos ? 1 : 0);
}

/*
 * The graph with its vertices renamed: old vertex v becomes new_of_old[v] (a permutation of
 * 0..n-1).  New row new_of_old[v] holds the entries of old row v with every source u replaced by
 * new_of_old[u], sorted by new source id, duplicates in the order of their old positions.
 *   rowptr2 (n+1), colidx2 (nnz): the relabelled CSR
 *   pos2 (nnz): old CSR position of every new position (what an edge-feature matrix must be
 *               permuted with); edge_w2[k'] = edge_w[pos2[k']] bit for bit (skipped if NULL)
 * Returns 0, 1 when new_of_old is not a permutation, 2 when memory runs out.
 */
int oracle_relabel(int64_t n, const int64_t* rowptr, const int32_t* colidx, const float* edge_w,
                   const int32_t* new_of_old, int64_t* rowptr2, int32_t* colidx2, float* edge_w2,
                   int64_t* pos2) {
  if (n < 0) return 1;
  int32_t* old_of_new = (int32_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(int32_t));
  if (!old_of_new) return 2;
  for (int64_t i = 0; i < n; ++i) old_of_new[i] = -1;
  for (int64_t v = 0; v < n; ++v) {
    const int32_t p = new_of_old[v];
    if (p < 0 || p >= n || old_of_new[p] != -1) { free(old_of_new); return 1; }
    old_of_new[p] = (int32_t)v;
  }
  rowptr2[0] = 0;
  for (int64_t i = 0; i < n; ++i) {
    const int64_t v = old_of_new[i];
    rowptr2[i + 1] = rowptr2[i] + (rowptr[v + 1] - rowptr[v]);
  }
  int64_t longest = 0;
  for (int64_t v = 0; v < n; ++v)
    if (rowptr[v + 1] - rowptr[v] > longest) longest = rowptr[v + 1] - rowptr[v];
  relabel_entry* row = (relabel_entry*)malloc((size_t)(longest > 0 ? longest : 1) * sizeof(relabel_entry));
  if (!row) { free(old_of_new); return 2; }
  for (int64_t i = 0; i < n; ++i) {
    const int64_t v = old_of_new[i];
    const int64_t len = rowptr[v + 1] - rowptr[v];
    for (int64_t t = 0; t < len; ++t) {
      row[t].src = new_of_old[colidx[rowptr[v] + t]];
      row[t].pos = rowptr[v] + t;
    }
    qsort(row, (size_t)len, sizeof(relabel_entry), relabel_cmp);
    for (int64_t t = 0; t < len; ++t) {
      const int64_t k2 = rowptr2[i] + t;
      colidx2[k2] = row[t].src;
      pos2[k2] = row[t].pos;
      if (edge_w) memcpy(&edge_w2[k2], &edge_w[row[t].pos], sizeof(float));
    }
  }
  free(row);
  free(old_of_new);
  return 0;
}
