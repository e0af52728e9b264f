/*
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, FP64 CPU statement of the ExactOBS / OBQ layer solver of
 * "Optimal Brain Compression".  It exists to check the CUDA library and to be timed as a CPU baseline;
 * nothing in the product path may call it, and it shares no code with the CUDA sources.
 *
 * Every function follows the passage it cites, in the paper's order and notation, with no blocking,
 * fusion or reordering.  Matrices are row-major doubles.  Indices are 0-based.
 *
 * Pins (see tests/test_oracle_*.py): masked least-squares optimum after every step, Lemma 1 against a
 * direct inverse of the reduced Hessian, brute force over all single removals, the telescoping loss
 * identity, the diagonal-Hessian special case, hand-computed d_col = 1 and 2 cases, a brute-force
 * simulation of the global step.  Every function here is pinned by at least one of them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_FLAG_OUTLIERS 1

/* ---- Hessian: H = 2 X X^T  (Section 3, "ExactOBS": the per-row least-squares Hessian) ---------------
 * X is d x n float (the same FP32 array the GPU sees), widened to double before any arithmetic. */
void oracle_hessian(const float *X, int d, int64_t n, double *H)
{
    for (int i = 0; i < d; ++i)
        for (int j = 0; j < d; ++j) {
            double s = 0.0;
            for (int64_t c = 0; c < n; ++c)
                s += (double)X[(int64_t)i * n + c] * (double)X[(int64_t)j * n + c];
            H[(int64_t)i * d + j] = 2.0 * s;
        }
}

/* ---- Dampened inverse (Section 3, "Implementation Details": small diagonal term before inverting) -----
 * lambda = damp_rel * mean(diag H);  A = H + lambda I = L L^T;  Hinv = L^-T L^-1, then symmetrised.
 * Returns 0, or 1 + index of the first non-positive pivot. */
int oracle_inverse(const double *H, int d, double damp_rel, double *Hinv)
{
    double tr = 0.0;
    for (int i = 0; i < d; ++i) tr += H[(int64_t)i * d + i];
    const double lambda = damp_rel * tr / (double)d;
    double *L = (double *)calloc((size_t)d * d, sizeof(double));
    double *Li = (double *)calloc((size_t)d * d, sizeof(double));
    int info = 0;
    for (int j = 0; j < d && !info; ++j) {
        double s = H[(int64_t)j * d + j] + lambda;
        for (int k = 0; k < j; ++k) s -= L[(int64_t)j * d + k] * L[(int64_t)j * d + k];
        if (!(s > 0.0)) { info = j + 1; break; }
        const double ljj = sqrt(s);
        L[(int64_t)j * d + j] = ljj;
#pragma omp parallel for schedule(static)
        for (int i = j + 1; i < d; ++i) {
            double t = H[(int64_t)i * d + j];
            for (int k = 0; k < j; ++k) t -= L[(int64_t)i * d + k] * L[(int64_t)j * d + k];
            L[(int64_t)i * d + j] = t / ljj;
        }
    }
    if (!info) {
        /* Li = L^-1 by forward substitution, one column of the identity at a time */
#pragma omp parallel for schedule(dynamic, 8)
        for (int c = 0; c < d; ++c)
            for (int i = c; i < d; ++i) {
                double t = (i == c) ? 1.0 : 0.0;
                for (int k = c; k < i; ++k) t -= L[(int64_t)i * d + k] * Li[(int64_t)k * d + c];
                Li[(int64_t)i * d + c] = t / L[(int64_t)i * d + i];
            }
        /* Hinv = Li^T Li */
#pragma omp parallel for schedule(dynamic, 8)
        for (int i = 0; i < d; ++i)
            for (int j = 0; j <= i; ++j) {
                double t = 0.0;
                for (int k = i; k < d; ++k) t += Li[(int64_t)k * d + i] * Li[(int64_t)k * d + j];
                Hinv[(int64_t)i * d + j] = t;
                Hinv[(int64_t)j * d + i] = t;
            }
    }
    free(L);
    free(Li);
    return info;
}

/* ---- quant(.) : uniform affine grid of width Delta = scale with integer offset zero and codes in
 * [0, maxq]; round-half-to-even on the true quotient (Section 4: "fixed grid of width Delta"). -------- */
static double grid_code(double x, double scale, double zero, int maxq)
{
    double c = rint(x / scale) + zero;
    if (c < 0.0) c = 0.0;
    if (c > (double)maxq) c = (double)maxq;
    return c;
}
static double grid_quant(double x, double scale, double zero, int maxq)
{
    return scale * (grid_code(x, scale, zero, maxq) - zero);
}

/*
 * ---- One row of Algorithm 1 (mode 0, pruning) or Algorithm 3 (mode 1, OBQ) ---------------------------
 *   M = {all active};  for t = 0..steps-1:
 *      p    = argmin_{p in M} (q(w_p) - w_p)^2 / [Hinv]_pp         (Eq. 3 / Eq. 7; q == 0 when pruning)
 *      w   -= Hinv[:,p] * (w_p - q(w_p)) / [Hinv]_pp               (then w_p = q(w_p) exactly)
 *      Hinv-= Hinv[:,p] Hinv[p,:] / [Hinv]_pp                      (Lemma 1)
 *      M   -= {p}                                                  (row and column p are zeroed)
 * Ties in the argmin go to the lowest index.  The recorded loss is (q(w_p)-w_p)^2/[Hinv]_pp as printed
 * in Section 3 ("Step 2").
 *
 * forced (nullable): take forced[t] instead of the argmin (teacher forcing); best[], margin[] and
 * forced_gap[] still describe the oracle's own choice at that state.
 *   margin[t]     = (s_second - s_best) / max(s_second, tiny)   (1 when a single candidate is left)
 *   forced_gap[t] = (s_forced - s_best) / max(s_forced, tiny)
 * N:M pattern (Section 3, "N:M Sparsity"; mode 0 only): with nm_block = M > 0 the argmin runs only over weights
 * whose block of M consecutive columns has lost fewer than nm_prune = M - N weights so far (every block keeps
 * exactly N non-zeros once steps = d (M - N) / M eliminations are done); nm_block = 0 switches it off.
 * With ORACLE_FLAG_OUTLIERS (Section 4, "Quantization Outliers"): if any active weight has
 * |q(w_j)-w_j| > Delta/2, the one with the largest such error is taken first (ties: lowest index).
 *
 * active0 (nullable): 1 = in M at the start.  Hi is the row's private d x d copy of Hinv and is
 * modified in place (so the caller can inspect it).  pivot_diag[t] (nullable) records [Hinv]_pp of step t.
 * w_trace (nullable) is (steps+1) x d with
 * w_trace[0] = w on entry.  Returns 0, or 1+t if [Hinv]_pp was not positive and finite at step t.
 */
int oracle_row(double *Hi, int d, double *w, int steps, int mode,
               double scale, double zero, int maxq, int flags,
               const int32_t *forced, const uint8_t *active0,
               int32_t *order, double *loss, double *margin, int32_t *best, double *forced_gap,
               double *round_dist, double *pivot_diag, double *w_trace, int32_t *codes,
               int nm_prune, int nm_block)
{
    const double tiny = 1e-300;
    int32_t *blk_pruned = nm_block > 0 ? (int32_t *)calloc((size_t)(d / nm_block + 1), sizeof(int32_t)) : NULL;
    int32_t *M = (int32_t *)malloc((size_t)d * sizeof(int32_t));   /* the remaining set, ascending */
    uint8_t *in_M = (uint8_t *)calloc((size_t)d, 1);
    double *err = (double *)malloc((size_t)d * sizeof(double));
    int m = 0;
    for (int j = 0; j < d; ++j)
        if (!active0 || active0[j]) { M[m++] = j; in_M[j] = 1; }
    if (w_trace) memcpy(w_trace, w, (size_t)d * sizeof(double));
    int ret = 0;
    for (int t = 0; t < steps; ++t) {
        /* scores over M */
        int b = -1, b2 = -1;
        double sb = 0.0, sb2 = 0.0;
        for (int a = 0; a < m; ++a) {
            const int j = M[a];
            const double q = mode ? grid_quant(w[j], scale, zero, maxq) : 0.0;
            err[j] = q - w[j];
            if (blk_pruned && blk_pruned[j / nm_block] >= nm_prune) continue;   /* block already at N non-zeros */
            const double s = err[j] * err[j] / Hi[(int64_t)j * d + j];
            if (b < 0 || s < sb) { b2 = b; sb2 = sb; b = j; sb = s; }
            else if (b2 < 0 || s < sb2) { b2 = j; sb2 = s; }
        }
        if (b < 0) { ret = ret ? ret : 1 + t; break; }       /* nothing left to eliminate */
        double mg = (b2 < 0) ? 1.0 : (sb2 - sb) / fmax(sb2, tiny);
        if (mode && (flags & ORACLE_FLAG_OUTLIERS)) {
            int ob = -1, ob2 = -1;
            double eb = 0.0, eb2 = 0.0, close = 1.0;
            for (int a = 0; a < m; ++a) {
                const int j = M[a];
                const double ae = fabs(err[j]);
                const double c = fabs(ae - 0.5 * scale) / (0.5 * scale);
                if (c < close) close = c;
                if (ae > 0.5 * scale) {
                    if (ob < 0 || ae > eb) { ob2 = ob; eb2 = eb; ob = j; eb = ae; }
                    else if (ob2 < 0 || ae > eb2) { ob2 = j; eb2 = ae; }
                }
            }
            if (ob >= 0) {
                b = ob;
                sb = err[b] * err[b] / Hi[(int64_t)b * d + b];
                mg = (ob2 < 0) ? 1.0 : (eb - eb2) / fmax(eb, tiny);
            }
            if (close < mg) mg = close;
        }
        int p = b;
        if (forced) {
            p = forced[t];
            if (p < 0 || p >= d || !in_M[p]) { ret = ret ? ret : 1 + t; break; }
        }
        if (blk_pruned) blk_pruned[p / nm_block] += 1;
        const double dpp = Hi[(int64_t)p * d + p];
        if (!(dpp > 0.0) || !isfinite(dpp)) { ret = ret ? ret : 1 + t; break; }
        const double sp = err[p] * err[p] / dpp;
        if (best) best[t] = b;
        if (margin) margin[t] = mg;
        if (forced_gap) forced_gap[t] = (sp - sb) / fmax(sp, tiny);
        order[t] = p;
        loss[t] = sp;
        if (pivot_diag) pivot_diag[t] = dpp;
        const double qp = mode ? grid_quant(w[p], scale, zero, maxq) : 0.0;
        if (mode) {
            const double xq = w[p] / scale;
            if (round_dist) round_dist[t] = fabs(fabs(xq - floor(xq)) - 0.5);
            if (codes) codes[p] = (int32_t)grid_code(w[p], scale, zero, maxq);
        }
        /* weight update, Eq. 3 / Eq. 7:  w -= Hinv[:,p] (w_p - q(w_p)) / [Hinv]_pp */
        const double f = -err[p] / dpp;
        for (int a = 0; a < m; ++a) { const int j = M[a]; w[j] -= f * Hi[(int64_t)j * d + p]; }
        w[p] = qp;
        /* Lemma 1 on the rows and columns of M, then drop row and column p */
        for (int a = 0; a < m; ++a) {
            const int i = M[a];
            if (i == p) continue;
            const double g = Hi[(int64_t)i * d + p] / dpp;
            for (int c = 0; c < m; ++c) { const int j = M[c]; Hi[(int64_t)i * d + j] -= g * Hi[(int64_t)p * d + j]; }
        }
        for (int a = 0; a < m; ++a) { const int j = M[a]; Hi[(int64_t)p * d + j] = 0.0; Hi[(int64_t)j * d + p] = 0.0; }
        int pos = 0;
        while (M[pos] != p) ++pos;
        for (int a = pos; a + 1 < m; ++a) M[a] = M[a + 1];
        --m;
        in_M[p] = 0;
        if (w_trace) memcpy(w_trace + (int64_t)(t + 1) * d, w, (size_t)d * sizeof(double));
    }
    free(M);
    free(in_M);
    free(err);
    free(blk_pruned);
    return ret;
}

/* ---- Block pruning (Section 3, "Block-Sparsity", Eq. 5) ------------------------------------------------------
 * Zeros appear in blocks of c consecutive weights.  Per step, over the remaining blocks P:
 *      P*  = argmin_P  w_P^T ((Hinv)_P)^-1 w_P                       (ties: lowest block)
 *      w  -= Hinv[:,P*] ((Hinv)_P*)^-1 w_P*                          (then w_P* = 0 exactly)
 *      Hinv: Lemma 1 applied successively for every p in P* (ascending), rows/columns of P* zeroed.
 * The c x c systems are solved directly by Gaussian elimination with partial pivoting.
 * order[c*t .. c*t+c) = the members of the t-th block (ascending), loss[c*t] = its score w_P^T((Hinv)_P)^-1 w_P and
 * loss[c*t+1 .. c*t+c) = 0, so that the per-weight global step (Algorithm 2) takes a block's members together.
 * forced_blocks (nullable): block index to take at step t instead of the argmin; best_block/forced_gap/margin describe
 * the oracle's own choice as in oracle_row.  Returns 0, or 1+t when a block matrix is not positive definite. */
static int solve_small(int c, const double *A, const double *b, double *x)
{
    double M[8][9];
    for (int i = 0; i < c; ++i) { for (int j = 0; j < c; ++j) M[i][j] = A[i * c + j]; M[i][c] = b[i]; }
    for (int k = 0; k < c; ++k) {
        int piv = k;
        for (int i = k + 1; i < c; ++i) if (fabs(M[i][k]) > fabs(M[piv][k])) piv = i;
        if (!(fabs(M[piv][k]) > 0.0) || !isfinite(M[piv][k])) return 1;
        if (piv != k) for (int j = 0; j <= c; ++j) { double t = M[k][j]; M[k][j] = M[piv][j]; M[piv][j] = t; }
        for (int i = k + 1; i < c; ++i) {
            const double f = M[i][k] / M[k][k];
            for (int j = k; j <= c; ++j) M[i][j] -= f * M[k][j];
        }
    }
    for (int i = c - 1; i >= 0; --i) {
        double t = M[i][c];
        for (int j = i + 1; j < c; ++j) t -= M[i][j] * x[j];
        x[i] = t / M[i][i];
    }
    return 0;
}

int oracle_row_blocks(double *Hi, int d, double *w, int c, int steps, const int32_t *forced_blocks,
                      int32_t *order, double *loss, double *margin, int32_t *best_block, double *forced_gap)
{
    const double tiny = 1e-300;
    const int nblk = d / c;
    uint8_t *gone = (uint8_t *)calloc((size_t)nblk, 1);
    double A[64], x[8], wp[8];
    int ret = 0;
    for (int t = 0; t < steps; ++t) {
        int b = -1, b2 = -1;
        double sb = 0.0, sb2 = 0.0, sforced = 0.0;
        const int fb = forced_blocks ? forced_blocks[t] : -1;
        for (int q = 0; q < nblk; ++q) {
            if (gone[q]) continue;
            for (int i = 0; i < c; ++i) {
                wp[i] = w[q * c + i];
                for (int j = 0; j < c; ++j) A[i * c + j] = Hi[(int64_t)(q * c + i) * d + q * c + j];
            }
            if (solve_small(c, A, wp, x)) { ret = ret ? ret : 1 + t; break; }
            double s = 0.0;
            for (int i = 0; i < c; ++i) s += wp[i] * x[i];
            if (!(s >= 0.0) || !isfinite(s)) { ret = ret ? ret : 1 + t; break; }
            if (q == fb) sforced = s;
            if (b < 0 || s < sb) { b2 = b; sb2 = sb; b = q; sb = s; }
            else if (b2 < 0 || s < sb2) { b2 = q; sb2 = s; }
        }
        if (ret || b < 0) { ret = ret ? ret : 1 + t; break; }
        int P = b;
        double sp = sb;
        if (forced_blocks) {
            if (fb < 0 || fb >= nblk || gone[fb]) { ret = 1 + t; break; }
            P = fb; sp = sforced;
        }
        if (best_block) best_block[t] = b;
        if (margin) margin[t] = (b2 < 0) ? 1.0 : (sb2 - sb) / fmax(sb2, tiny);
        if (forced_gap) forced_gap[t] = (sp - sb) / fmax(sp, tiny);
        for (int i = 0; i < c; ++i) { order[t * c + i] = P * c + i; loss[t * c + i] = 0.0; }
        loss[t * c] = sp;
        /* weight update with the block formula (Eq. 5) */
        for (int i = 0; i < c; ++i) {
            wp[i] = w[P * c + i];
            for (int j = 0; j < c; ++j) A[i * c + j] = Hi[(int64_t)(P * c + i) * d + P * c + j];
        }
        if (solve_small(c, A, wp, x)) { ret = 1 + t; break; }
        for (int j = 0; j < d; ++j) {
            double acc = 0.0;
            for (int i = 0; i < c; ++i) acc += Hi[(int64_t)j * d + P * c + i] * x[i];
            w[j] -= acc;
        }
        for (int i = 0; i < c; ++i) w[P * c + i] = 0.0;
        /* Lemma 1, successively for every member of the block */
        for (int i = 0; i < c; ++i) {
            const int p = P * c + i;
            const double dpp = Hi[(int64_t)p * d + p];
            if (!(dpp > 0.0) || !isfinite(dpp)) { ret = 1 + t; break; }
            for (int a = 0; a < d; ++a) {
                if (a == p) continue;
                const double g = Hi[(int64_t)a * d + p] / dpp;
                if (g == 0.0) continue;
                for (int e = 0; e < d; ++e) Hi[(int64_t)a * d + e] -= g * Hi[(int64_t)p * d + e];
            }
            for (int a = 0; a < d; ++a) { Hi[(int64_t)p * d + a] = 0.0; Hi[(int64_t)a * d + p] = 0.0; }
        }
        if (ret) break;
        gone[P] = 1;
    }
    free(gone);
    return ret;
}

/* Many independent rows (Section 3: no Hessian interaction between rows); OpenMP over rows.
 * Per-row arrays are strided by `steps` (order, loss, margin, best, forced_gap, round_dist, pivot_diag),
 * by d (w, codes, active0) and by (steps+1)*d (w_trace).  scale/zero are per row.  Each row works on
 * its own copy of Hinv.  status[r] receives oracle_row's return value. */
void oracle_rows(const double *Hinv, int d, int rows, double *W, int steps, int mode,
                 const double *scale, const double *zero, int maxq, int flags,
                 const int32_t *forced, const uint8_t *active0,
                 int32_t *order, double *loss, double *margin, int32_t *best, double *forced_gap,
                 double *round_dist, double *pivot_diag, double *w_trace, int32_t *codes, int32_t *status,
                 int nm_prune, int nm_block)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < rows; ++r) {
        double *Hi = (double *)malloc((size_t)d * d * sizeof(double));
        memcpy(Hi, Hinv, (size_t)d * d * sizeof(double));
        const int64_t so = (int64_t)r * steps;
        status[r] = oracle_row(Hi, d, W + (int64_t)r * d, steps, mode,
                               scale ? scale[r] : 1.0, zero ? zero[r] : 0.0, maxq, flags,
                               forced ? forced + so : NULL, active0 ? active0 + (int64_t)r * d : NULL,
                               order + so, loss + so, margin ? margin + so : NULL, best ? best + so : NULL,
                               forced_gap ? forced_gap + so : NULL, round_dist ? round_dist + so : NULL,
                               pivot_diag ? pivot_diag + so : NULL,
                               w_trace ? w_trace + (int64_t)r * (steps + 1) * d : NULL,
                               codes ? codes + (int64_t)r * d : NULL, nm_prune, nm_block);
        free(Hi);
    }
}

/* ---- Global step, Algorithm 2 (appendix "ExactOBS Global Step Pseudocode") ---------------------------
 * Q holds, per row i, the number j of weights already pruned there.  k times: take the (i, j) whose next
 * loss L[i][j] is smallest (infinity once a row is exhausted; ties go to the lowest row) and advance it.
 * Q is a binary min-heap keyed by (value, row).  mask[i][P[i][t]] = 0 for t < counts[i], else 1. */
typedef struct { double v; int32_t row; } heap_item;
static int item_less(heap_item a, heap_item b) { return a.v < b.v || (a.v == b.v && a.row < b.row); }
static void sift_down(heap_item *h, int n, int i)
{
    for (;;) {
        int l = 2 * i + 1, r = l + 1, m = i;
        if (l < n && item_less(h[l], h[m])) m = l;
        if (r < n && item_less(h[r], h[m])) m = r;
        if (m == i) return;
        heap_item t = h[i]; h[i] = h[m]; h[m] = t;
        i = m;
    }
}
int oracle_global_mask(const double *L, const int32_t *P, int rows, int d, int64_t k,
                       int32_t *counts, uint8_t *mask)
{
    if (k < 0 || k > (int64_t)rows * d) return 1;
    heap_item *h = (heap_item *)malloc((size_t)rows * sizeof(heap_item));
    for (int i = 0; i < rows; ++i) { counts[i] = 0; h[i].v = d > 0 ? L[(int64_t)i * d] : INFINITY; h[i].row = i; }
    for (int i = rows / 2 - 1; i >= 0; --i) sift_down(h, rows, i);
    for (int64_t it = 0; it < k; ++it) {
        const int i = h[0].row;
        const int j = ++counts[i];
        h[0].v = (j < d) ? L[(int64_t)i * d + j] : INFINITY;
        sift_down(h, rows, 0);
    }
    free(h);
    for (int i = 0; i < rows; ++i) {
        for (int j = 0; j < d; ++j) mask[(int64_t)i * d + j] = 1;
        for (int t = 0; t < counts[i]; ++t) mask[(int64_t)i * d + P[(int64_t)i * d + t]] = 0;
    }
    return 0;
}

/* ---- Per-row min-max grid over the kept entries (the benchmark configurations' grid; the paper only
 * fixes "symmetric / asymmetric per-channel").  Range always contains 0.
 *   asymmetric: maxq = 2^bits - 1, Delta = (hi - lo)/maxq, zero = rne(-lo/Delta)
 *   symmetric : Q = 2^(bits-1) - 1, Delta = max|w|/Q, zero = Q, maxq = 2Q
 *   degenerate (hi == lo): Delta = 1. */
void oracle_minmax_grid(const double *W, int rows, int d, const uint8_t *mask, int bits, int symmetric,
                        double *scale, double *zero, int32_t *maxq_out)
{
    for (int r = 0; r < rows; ++r) {
        double lo = 0.0, hi = 0.0;
        for (int j = 0; j < d; ++j) {
            if (mask && !mask[(int64_t)r * d + j]) continue;
            const double x = W[(int64_t)r * d + j];
            if (x < lo) lo = x;
            if (x > hi) hi = x;
        }
        if (symmetric) {
            const double Q = (double)((1 << (bits - 1)) - 1);
            const double a = fmax(hi, -lo);
            scale[r] = (a > 0.0) ? a / Q : 1.0;
            zero[r] = Q;
            *maxq_out = 2 * (int32_t)Q;
        } else {
            const int mq = (1 << bits) - 1;
            scale[r] = (hi > lo) ? (hi - lo) / (double)mq : 1.0;
            zero[r] = rint(-lo / scale[r]);
            *maxq_out = mq;
        }
    }
}
