/*
 * CPU ORACLE -- TEST INFRASTRUCTURE ONLY.  Not part of the product path.
 *
 * Plain, slow, single-threaded reference for what DB-SpMSpV computes.  The blocked method
 * reaches exactly the mathematical result y = A*x (up to rounding order), so the oracle is
 * the plain definition written out: the textbook push and pull loops of Algorithm 1
 * (Section 2.1), accumulated in fp64, plus a queue BFS.  There is no blocking, fusion or
 * reordering here.  It shares no code with the CUDA library.
 *
 * Output convention (the paper returns a dense y and is silent on the rest): a row i is
 * reported iff some stored A[i][j] meets some listed x_j -- a *structural* hit, whatever the
 * numeric sum -- in ascending row order.  Beside each value the oracle returns
 * scale_i = sum_k |a_ik * x_k|, the denominator of the value tolerance.
 *
 * Pins (tests/test_oracle_pins.py): brute-force dense mat-vec, identity and permutation
 * matrices, exact integer linearity, pull == push, queue BFS == level-synchronous Boolean
 * SpMSpV BFS, path/star/two-component/directed-cycle graphs, Chebyshev-distance closed form
 * on the 27-point grid graph.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Algorithm 1, bottom half (pull over CSR): for every row scan its stored entries and use
 * those whose input entry is listed.  val == NULL or x_val == NULL -> Boolean (pattern).   */
int64_t ref_pull(int64_t m, int64_t n, const int64_t *row_ptr, const int32_t *col_idx,
                 const float *val, int64_t nnz_x, const int32_t *x_idx, const float *x_val,
                 int32_t *y_idx, double *y_val, double *y_scale)
{
    uint8_t *present = (uint8_t *)calloc((size_t)(n > 0 ? n : 1), 1);
    double *xs = (double *)calloc((size_t)(n > 0 ? n : 1), sizeof(double));
    if (!present || !xs) { free(present); free(xs); return -1; }
    for (int64_t k = 0; k < nnz_x; ++k) {
        present[x_idx[k]] = 1;
        xs[x_idx[k]] = x_val ? (double)x_val[k] : 1.0;
    }
    int64_t cnt = 0;
    for (int64_t i = 0; i < m; ++i) {
        double acc = 0.0, scale = 0.0;
        int hit = 0;
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            int32_t j = col_idx[p];
            if (present[j]) {
                double a = val ? (double)val[p] : 1.0;
                double t = a * xs[j];
                hit = 1;
                acc += t;
                scale += fabs(t);
            }
        }
        if (hit) {
            y_idx[cnt] = (int32_t)i;
            if (y_val) y_val[cnt] = acc;
            if (y_scale) y_scale[cnt] = scale;
            ++cnt;
        }
    }
    free(present);
    free(xs);
    return cnt;
}

/* Plain transposition CSR -> CSC by counting (the oracle's own; used by push and BFS).     */
void ref_csr_to_csc(int64_t m, int64_t n, const int64_t *row_ptr, const int32_t *col_idx,
                    const float *val, int64_t *col_ptr, int32_t *row_idx, float *cval)
{
    memset(col_ptr, 0, (size_t)(n + 1) * sizeof(int64_t));
    int64_t nnz = row_ptr[m];
    for (int64_t p = 0; p < nnz; ++p) col_ptr[col_idx[p] + 1]++;
    for (int64_t j = 0; j < n; ++j) col_ptr[j + 1] += col_ptr[j];
    int64_t *next = (int64_t *)malloc((size_t)(n > 0 ? n : 1) * sizeof(int64_t));
    memcpy(next, col_ptr, (size_t)n * sizeof(int64_t));
    for (int64_t i = 0; i < m; ++i)
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            int64_t q = next[col_idx[p]]++;
            row_idx[q] = (int32_t)i;
            if (val && cval) cval[q] = val[p];
        }
    free(next);
}

/* Algorithm 1, top half (push over CSC): for every listed x_j walk column j and scatter
 * into a dense accumulator; touched rows are gathered in ascending order.                   */
int64_t ref_push(int64_t m, int64_t n, const int64_t *col_ptr, const int32_t *row_idx,
                 const float *cval, int64_t nnz_x, const int32_t *x_idx, const float *x_val,
                 int32_t *y_idx, double *y_val, double *y_scale)
{
    (void)n;
    double *acc = (double *)calloc((size_t)(m > 0 ? m : 1), sizeof(double));
    double *scl = (double *)calloc((size_t)(m > 0 ? m : 1), sizeof(double));
    uint8_t *touched = (uint8_t *)calloc((size_t)(m > 0 ? m : 1), 1);
    if (!acc || !scl || !touched) { free(acc); free(scl); free(touched); return -1; }
    for (int64_t k = 0; k < nnz_x; ++k) {
        int32_t j = x_idx[k];
        double xj = x_val ? (double)x_val[k] : 1.0;
        for (int64_t p = col_ptr[j]; p < col_ptr[j + 1]; ++p) {
            int32_t i = row_idx[p];
            double t = (cval ? (double)cval[p] : 1.0) * xj;
            acc[i] += t;
            scl[i] += fabs(t);
            touched[i] = 1;
        }
    }
    int64_t cnt = 0;
    for (int64_t i = 0; i < m; ++i)
        if (touched[i]) {
            y_idx[cnt] = (int32_t)i;
            if (y_val) y_val[cnt] = acc[i];
            if (y_scale) y_scale[cnt] = scl[i];
            ++cnt;
        }
    free(acc); free(scl); free(touched);
    return cnt;
}

/* Queue BFS.  Edge orientation: a stored A[i][j] is the edge j -> i (this is what y = A*x
 * with a frontier x propagates, Section 2.1 push), so the out-neighbours of j are the rows
 * of column j: the CSC arrays.  levels: source 0, unreachable -1.  Returns reached count.   */
int64_t ref_bfs(int64_t n, const int64_t *col_ptr, const int32_t *row_idx, int32_t src,
                int32_t *levels)
{
    for (int64_t v = 0; v < n; ++v) levels[v] = -1;
    int32_t *queue = (int32_t *)malloc((size_t)(n > 0 ? n : 1) * sizeof(int32_t));
    if (!queue) return -1;
    int64_t head = 0, tail = 0;
    levels[src] = 0;
    queue[tail++] = src;
    while (head < tail) {
        int32_t j = queue[head++];
        for (int64_t p = col_ptr[j]; p < col_ptr[j + 1]; ++p) {
            int32_t i = row_idx[p];
            if (levels[i] < 0) {
                levels[i] = levels[j] + 1;
                queue[tail++] = i;
            }
        }
    }
    free(queue);
    return tail;
}

/* Single-token linear layer (Section 4.3): dense x in, dense y out.  Structural x = entries
 * with x[j] != 0 (so -0.0 counts as zero); rows without a structural hit are exactly 0.
 * Same loop as ref_pull.  Operands arrive already rounded to bf16 and widened.              */
void ref_decode(int64_t m, int64_t n, const int64_t *row_ptr, const int32_t *col_idx,
                const float *val, const float *x, double *y, double *y_scale)
{
    (void)n;
    for (int64_t i = 0; i < m; ++i) {
        double acc = 0.0, scale = 0.0;
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            float xj = x[col_idx[p]];
            if (xj != 0.0f) {
                double t = (double)val[p] * (double)xj;
                acc += t;
                scale += fabs(t);
            }
        }
        y[i] = acc;
        if (y_scale) y_scale[i] = scale;
    }
}

/* (min, +) SpMSpV: Algorithm 1 (pull half) with the sum of products replaced by the minimum
 * of sums, y_i = min over stored A[i][j] with x_j listed of (A[i][j] + x_j) -- the product
 * that GraphBLAS-style systems (Sections 1 and 6) iterate for single-source shortest paths.
 * A listed x_j = 0 takes part (an absent entry is +infinity, not 0); val == NULL: every
 * stored element has weight 1.  Row i is reported iff a stored element meets a listed entry.
 * Pins: brute force over a dense matrix, x = {j: 0} returns column j, pattern matrix with a
 * zero-valued frontier gives hop counts (BFS levels).                                       */
int64_t ref_minplus(int64_t m, int64_t n, const int64_t *row_ptr, const int32_t *col_idx,
                    const float *val, int64_t nnz_x, const int32_t *x_idx, const float *x_val,
                    int32_t *y_idx, double *y_val)
{
    uint8_t *present = (uint8_t *)calloc((size_t)(n > 0 ? n : 1), 1);
    double *xs = (double *)calloc((size_t)(n > 0 ? n : 1), sizeof(double));
    if (!present || !xs) { free(present); free(xs); return -1; }
    for (int64_t k = 0; k < nnz_x; ++k) {
        present[x_idx[k]] = 1;
        xs[x_idx[k]] = x_val ? (double)x_val[k] : 0.0;
    }
    int64_t cnt = 0;
    for (int64_t i = 0; i < m; ++i) {
        double best = INFINITY;
        int hit = 0;
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            int32_t j = col_idx[p];
            if (present[j]) {
                double t = (val ? (double)val[p] : 1.0) + xs[j];
                if (!hit || t < best) best = t;
                hit = 1;
            }
        }
        if (hit) {
            y_idx[cnt] = (int32_t)i;
            y_val[cnt] = best;
            ++cnt;
        }
    }
    free(present);
    free(xs);
    return cnt;
}

/* Single-source shortest paths by Bellman-Ford sweeps: dist[src] = 0, everything else
 * +infinity; every sweep relaxes every edge (a stored A[i][j] is the edge j -> i of weight
 * A[i][j], as in ref_bfs) until a sweep changes nothing.  Weights must not close a negative
 * cycle (at most n sweeps are made).  Returns the number of sweeps, -1 if it did not settle.
 * Pins: a library Dijkstra, path and star graphs in closed form, unit weights == BFS levels. */
int64_t ref_sssp(int64_t n, const int64_t *col_ptr, const int32_t *row_idx, const float *cval,
                 int32_t src, double *dist)
{
    for (int64_t v = 0; v < n; ++v) dist[v] = INFINITY;
    dist[src] = 0.0;
    for (int64_t sweep = 1; sweep <= n + 1; ++sweep) {
        int changed = 0;
        for (int64_t j = 0; j < n; ++j) {
            if (isinf(dist[j])) continue;
            for (int64_t p = col_ptr[j]; p < col_ptr[j + 1]; ++p) {
                double t = dist[j] + (cval ? (double)cval[p] : 1.0);
                if (t < dist[row_idx[p]]) { dist[row_idx[p]] = t; changed = 1; }
            }
        }
        if (!changed) return sweep;
    }
    return -1;
}
