/*
 * CPU oracle for block-wise multi-hop feature aggregation  X_k = A^ X_{k-1}, k = 1..K.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA
 * library is checked against.  It shares no code with that library, is never
 * linked into it, and only the tests, the smoke check and the benchmark's CPU
 * baseline may call it.
 *
 * Everything is written from the paper's definitions (arXiv 2207.12000):
 *   - Section 2 (Preliminaries): A in {0,1}^{n x n} undirected, D_i = degree of node i,
 *     A~ = A + I.
 *   - Eq. 1:  S = D~^{-1/2} A~ D~^{-1/2}   (D~_ii = sum_j A~_ij = D_i + 1).
 *   - Section 3.2 "Precomputation on GPU": edge list E of A~ split into disjoint sets of
 *     similar size; Eq. 10: S = sum_l D~^{-1/2} A~^(l) D~^{-1/2}.
 *   - Algorithm 1 (block-wise feature aggregation): b edge blocks x c column slabs x K hops.
 *   - Eq. 12: min b*c subject to beta_S B_S / b + beta_X B_X / c <= B_GPU, by exhaustive search.
 * Two further constant filters are supported beside Eq. 1's, both linear and fixed before
 * precomputation as Section 3.1 "Limitation" and the related-work note on GIN require:
 *   SAGE row-mean  A^ = D^{-1} A          (rows with D_i = 0 are zero rows)
 *   GIN sum        A^ = A + (1 + eps) I   (eps a fixed constant)
 *
 * Floating point is fp64 throughout; X_0 is the fp32 input widened to fp64 and no hop is
 * rounded back to fp32.  Sums run over a row's support in ascending column order.
 *
 * Parity pins (tests/test_oracle_pins.py): closed forms on complete, cycle, star and regular
 * graphs, fixed points and conservation laws of each operator, brute-force dense A^^k X,
 * an independent scipy.sparse product, and exhaustive checks of the block partition.
 * The fixed-weight sum of hops, orc_weighted_hop_sum, is pinned by unit weights (one hop each), by the
 * identity that turns the K-step PageRank iteration into such a sum, and by a closed form on a complete graph.
 * The first dense stage of an LC model (Eq. 9), orc_lc_first_layer, is pinned by a library matrix
 * product, by one-hot / identity weights and by the commutation S^k (X W) = (S^k X) W on integers.
 * Absolute speed is the one thing with no pin: the paper prints ratios only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_OP_GCN = 0, ORC_OP_SAGE = 1, ORC_OP_GIN = 2 };

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* Section 2: D_i is the degree of node i, i.e. the number of ones in row i of A. */
void orc_degrees(int64_t n, const int64_t* rowptr, int32_t* deg) {
    for (int64_t i = 0; i < n; ++i) deg[i] = (int32_t)(rowptr[i + 1] - rowptr[i]);
}

/* Does the operator's support contain the diagonal?  (A~ = A + I for Eq. 1; the GIN self term.) */
static int has_diagonal(int op) { return op == ORC_OP_GCN || op == ORC_OP_GIN; }

/*
 * Entry A^_ij for an edge (i, j) of the support.
 *   GCN  (Eq. 1): A~_ij / sqrt(D~_i D~_j), evaluated as (1/sqrt(D~_i)) * (1/sqrt(D~_j)).
 *   SAGE: A_ij / D_i.
 *   GIN : 1 off the diagonal, 1 + eps on it.
 */
static double entry(int op, double eps, const int32_t* deg, int64_t i, int64_t j) {
    switch (op) {
    case ORC_OP_GCN:
        return (1.0 / sqrt((double)deg[i] + 1.0)) * (1.0 / sqrt((double)deg[j] + 1.0));
    case ORC_OP_SAGE:
        return 1.0 / (double)deg[i];
    default:
        return i == j ? 1.0 + eps : 1.0;
    }
}

/*
 * The per-node factors the operator separates into, A^_ij = r_i * c_j (times the GIN
 * diagonal weight), rounded once from fp64 to fp32.  The CUDA library exposes its own
 * copies of these arrays and the two must agree bit for bit.
 *   GCN : r_i = c_i = D~_i^{-1/2}        SAGE: r_i = 1/D_i (0 when D_i = 0), c = 1
 *   GIN : r = c = 1
 */
void orc_scales_f32(int op, int64_t n, const int32_t* deg, float* rscale, float* cscale) {
    for (int64_t i = 0; i < n; ++i) {
        double r = 1.0, c = 1.0;
        if (op == ORC_OP_GCN) {
            r = c = 1.0 / sqrt((double)deg[i] + 1.0);
        } else if (op == ORC_OP_SAGE) {
            r = deg[i] > 0 ? 1.0 / (double)deg[i] : 0.0;
        }
        rscale[i] = (float)r;
        cscale[i] = (float)c;
    }
}

/* Number of edges in E, the edge list of the operator's support (Section 3.2: E lists A~). */
int64_t orc_support_nnz(int op, int64_t n, int64_t nnz) { return has_diagonal(op) ? nnz + n : nnz; }

/*
 * CSR of the support: A with the diagonal entry inserted at its column-sorted position
 * when the operator has one.  Input rows hold strictly ascending columns and no diagonal.
 */
void orc_support(int op, int64_t n, const int64_t* rowptr, const int32_t* colidx, int64_t* rowptr_t,
                 int32_t* colidx_t) {
    int64_t w = 0;
    rowptr_t[0] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int placed = !has_diagonal(op);
        for (int64_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
            if (!placed && colidx[e] > i) {
                colidx_t[w++] = (int32_t)i;
                placed = 1;
            }
            colidx_t[w++] = colidx[e];
        }
        if (!placed) colidx_t[w++] = (int32_t)i;
        rowptr_t[i + 1] = w;
    }
}

/* Dense A^ (row-major n x n), for tiny graphs only. */
void orc_dense_operator(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx,
                        double* Ahat) {
    int32_t* deg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    orc_degrees(n, rowptr, deg);
    memset(Ahat, 0, sizeof(double) * (size_t)n * (size_t)n);
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t e = rowptr[i]; e < rowptr[i + 1]; ++e) Ahat[i * n + colidx[e]] = entry(op, eps, deg, i, colidx[e]);
        if (has_diagonal(op)) Ahat[i * n + i] = entry(op, eps, deg, i, i);
    }
    free(deg);
}

/*
 * One output row of one hop: y[f] = sum_j A^_ij x[j, f], with j running in ascending order
 * over the support of row i (the columns of A merged with the diagonal when the operator
 * has one).  `absy`, when given, receives sum_j |A^_ij| |x[j, f]|, the scale of the sum,
 * which the componentwise error measure divides by.  Two copies: fp32 and fp64 input.
 */
#define DEFINE_ROW(NAME, T)                                                                              \
    static void NAME(int op, double eps, const int32_t* deg, const int64_t* rowptr, const int32_t* colidx,  \
                     int64_t F, const T* x, int64_t ldx, int64_t i, double* y, double* absy) {           \
        for (int64_t f = 0; f < F; ++f) y[f] = 0.0;                                                      \
        if (absy)                                                                                        \
            for (int64_t f = 0; f < F; ++f) absy[f] = 0.0;                                               \
        int64_t e = rowptr[i];                                                                           \
        const int64_t end = rowptr[i + 1];                                                               \
        int diag_pending = has_diagonal(op);                                                             \
        while (e < end || diag_pending) {                                                                \
            int64_t j;                                                                                   \
            if (diag_pending && (e == end || colidx[e] > i)) {                                           \
                j = i; /* the diagonal entry, at its sorted position */                                  \
                diag_pending = 0;                                                                        \
            } else {                                                                                     \
                j = colidx[e++];                                                                         \
            }                                                                                            \
            const double w = entry(op, eps, deg, i, j);                                                  \
            const T* xj = x + j * ldx;                                                                   \
            for (int64_t f = 0; f < F; ++f) y[f] += w * (double)xj[f];                                   \
            if (absy)                                                                                    \
                for (int64_t f = 0; f < F; ++f) absy[f] += fabs(w) * fabs((double)xj[f]);                \
        }                                                                                                \
    }
DEFINE_ROW(row_f32, float)
DEFINE_ROW(row_f64, double)

/* One hop over all rows from an fp64 previous hop (rows are independent: OpenMP over rows). */
void orc_hop_f64(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx, int64_t F,
                 const double* xprev, double* xnext) {
    int32_t* deg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    orc_degrees(n, rowptr, deg);
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < n; ++i) row_f64(op, eps, deg, rowptr, colidx, F, xprev, F, i, xnext + i * F, NULL);
    free(deg);
}

/*
 * The definition: out[k-1] = A^ out[k-2], out[-1] = X (fp32 widened), for k = 1..K.
 * `out` is K consecutive row-major n x F fp64 matrices.  A^k itself is never formed
 * (the appendix on GPRGNN notes its fill-in); each hop multiplies the previous one.
 */
void orc_propagate(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx, int64_t F,
                   const float* X, int64_t ldx, int K, double* out) {
    int32_t* deg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    orc_degrees(n, rowptr, deg);
    for (int k = 0; k < K; ++k) {
        double* xk = out + (size_t)k * (size_t)n * (size_t)F;
        if (k == 0) {
#pragma omp parallel for schedule(dynamic, 256)
            for (int64_t i = 0; i < n; ++i) row_f32(op, eps, deg, rowptr, colidx, F, X, ldx, i, xk + i * F, NULL);
        } else {
            const double* xp = out + (size_t)(k - 1) * (size_t)n * (size_t)F;
#pragma omp parallel for schedule(dynamic, 256)
            for (int64_t i = 0; i < n; ++i) row_f64(op, eps, deg, rowptr, colidx, F, xp, F, i, xk + i * F, NULL);
        }
    }
    free(deg);
}

/*
 * Personalised-PageRank style propagation, one of the constant filters Section 3.1 ("Limitation")
 * names as precomputable:  X_k = (1 - alpha) A^ X_{k-1} + alpha X_0,  k = 1..K  (the power
 * iteration of APPNP).  alpha = 0 is orc_propagate.  `out` as in orc_propagate.
 */
void orc_propagate_teleport(int op, double eps, double alpha, int64_t n, const int64_t* rowptr, const int32_t* colidx,
                            int64_t F, const float* X, int64_t ldx, int K, double* out) {
    orc_propagate(op, eps, n, rowptr, colidx, F, X, ldx, 1, out); /* A^ X_0 */
    for (int k = 0; k < K; ++k) {
        double* xk = out + (size_t)k * (size_t)n * (size_t)F;
        if (k > 0) orc_hop_f64(op, eps, n, rowptr, colidx, F, out + (size_t)(k - 1) * (size_t)n * (size_t)F, xk);
        for (int64_t i = 0; i < n; ++i)
            for (int64_t f = 0; f < F; ++f) xk[i * F + f] = (1.0 - alpha) * xk[i * F + f] + alpha * (double)X[i * ldx + f];
    }
}

/*
 * Generalised-PageRank filter with FIXED weights (the appendix on GPRGNN, Eq. 13: H = sum_k gamma_k S^k (...);
 * with gamma fixed before training it is one more constant filter in the sense of Section 3.1 "Limitation"):
 *     Z = sum_{k=0..K} gamma[k] A^^k X_0 ,
 * evaluated hop by hop (A^^k is never formed: same appendix), fp64.  Z is [n, F].
 */
void orc_weighted_hop_sum(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx, int64_t F,
                          const float* X, int64_t ldx, int K, const double* gamma, double* Z) {
    const size_t nf = (size_t)n * (size_t)F;
    double* cur = (double*)malloc(sizeof(double) * nf);
    double* nxt = (double*)malloc(sizeof(double) * nf);
    for (int64_t i = 0; i < n; ++i)
        for (int64_t f = 0; f < F; ++f) {
            cur[i * F + f] = (double)X[i * ldx + f];
            Z[i * F + f] = gamma[0] * cur[i * F + f];
        }
    for (int k = 1; k <= K; ++k) {
        orc_hop_f64(op, eps, n, rowptr, colidx, F, cur, nxt);
        for (size_t t = 0; t < nf; ++t) Z[t] += gamma[k] * nxt[t];
        double* tmp = cur;
        cur = nxt;
        nxt = tmp;
    }
    free(nxt);
    free(cur);
}

/*
 * One hop evaluated on chosen rows only, from an fp32 previous hop: the exact fp64 value
 * of (A^ xprev)[rows[r], :] and, optionally, of (|A^| |xprev|)[rows[r], :].
 */
void orc_hop_rows_f32(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx, int64_t F,
                      const float* xprev, int64_t ldx, int64_t nrows, const int64_t* rows, double* y, double* absy) {
    int32_t* deg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    orc_degrees(n, rowptr, deg);
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t r = 0; r < nrows; ++r)
        row_f32(op, eps, deg, rowptr, colidx, F, xprev, ldx, rows[r], y + r * F, absy ? absy + r * F : NULL);
    free(deg);
}

/* ------------------------------------------------------------------ edge decomposition */

/*
 * Section 3.2: E is cut into b disjoint sets of similar size.  The reading fixed here:
 * block l is the contiguous range [floor(l m / b), floor((l+1) m / b)) of the CSR-ordered
 * edge list (m = |E|), so sizes differ by at most one edge.  Returns -1 when a block would
 * be empty (b > m) or b < 1.
 */
int orc_block_offsets(int64_t m, int32_t b, int64_t* e_off) {
    if (b < 1 || (int64_t)b > m) return -1;
    for (int32_t l = 0; l <= b; ++l) {
        /* l*m can exceed 63 bits only for m > 2^31 * 2^31 / b; split to stay exact anyway */
        const int64_t q = m / b, r = m % b;
        e_off[l] = (int64_t)l * q + ((int64_t)l * r) / b;
    }
    return 0;
}

/*
 * Rows a block touches: row_lo = row holding its first edge, row_hi = row holding its last
 * edge; a flag tells whether that row also has edges in the neighbouring block (the paper's
 * limitation paragraph: a node's edges may fall into different groups).
 * Linear scan over rows, no search tricks.
 */
void orc_block_rows(int64_t n, const int64_t* rowptr_t, int32_t b, const int64_t* e_off, int32_t* row_lo,
                    int32_t* row_hi, int32_t* first_partial, int32_t* last_partial) {
    for (int32_t l = 0; l < b; ++l) {
        const int64_t lo = e_off[l], hi = e_off[l + 1] - 1; /* first and last edge of the block */
        for (int64_t i = 0; i < n; ++i) {
            if (rowptr_t[i] <= lo && lo < rowptr_t[i + 1]) {
                row_lo[l] = (int32_t)i;
                first_partial[l] = rowptr_t[i] < lo;
            }
            if (rowptr_t[i] <= hi && hi < rowptr_t[i + 1]) {
                row_hi[l] = (int32_t)i;
                last_partial[l] = hi + 1 < rowptr_t[i + 1];
            }
        }
    }
}

/* ceil(a / b) for positive integers */
static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/*
 * Eq. 12 by exhaustive search over natural (b, c), b <= max_b, c <= max_c:
 *   ceil(beta_S B_S / b) + ceil(beta_X B_X / c) + B_fixed <= B_GPU,  minimise b c,
 * ties broken towards the smaller c, then the smaller b.  B_fixed is the part of the
 * working set that no split shrinks (the per-node scale arrays; Eq. 11's alpha_D B_D term
 * plays the same role there).  Returns 0 and (b, c), or -1 if nothing is feasible.
 */
int orc_solve_budget(int64_t B_S, int64_t B_X, int64_t B_fixed, int64_t beta_S, int64_t beta_X, int64_t B_GPU,
                     int64_t max_b, int64_t max_c, int64_t* b_out, int64_t* c_out) {
    int found = 0;
    int64_t best_b = 0, best_c = 0;
    for (int64_t c = 1; c <= max_c; ++c) {
        for (int64_t b = 1; b <= max_b; ++b) {
            if (ceil_div(beta_S * B_S, b) + ceil_div(beta_X * B_X, c) + B_fixed > B_GPU) continue;
            if (!found || b * c < best_b * best_c || (b * c == best_b * best_c && c < best_c)) {
                found = 1;
                best_b = b;
                best_c = c;
            }
        }
    }
    if (!found) return -1;
    *b_out = best_b;
    *c_out = best_c;
    return 0;
}

/* Eq. 11: least a with ceil((alpha_A B_A + alpha_S B_S) / a) + alpha_D B_D <= B_GPU, or -1. */
int64_t orc_solve_normalisation_blocks(int64_t B_A, int64_t B_S, int64_t B_D, int64_t alpha_A, int64_t alpha_S,
                                       int64_t alpha_D, int64_t B_GPU, int64_t max_a) {
    for (int64_t a = 1; a <= max_a; ++a)
        if (ceil_div(alpha_A * B_A + alpha_S * B_S, a) + alpha_D * B_D <= B_GPU) return a;
    return -1;
}

/*
 * The normalised adjacency itself (Eq. 1; block-wise Eq. 10): the value A^_ij of every edge of the
 * support, in the support's CSR order (orc_support gives the matching structure).  With b blocks,
 * block l holds the values of edges [e_off[l], e_off[l+1]); the blocks are disjoint, so their
 * union is the whole matrix.  vals has orc_support_nnz entries.
 */
void orc_normalized_values(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx, double* vals) {
    int32_t* deg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    orc_degrees(n, rowptr, deg);
    int64_t w = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t e = rowptr[i];
        const int64_t end = rowptr[i + 1];
        int diag_pending = has_diagonal(op);
        while (e < end || diag_pending) {
            int64_t j;
            if (diag_pending && (e == end || colidx[e] > i)) {
                j = i;
                diag_pending = 0;
            } else {
                j = colidx[e++];
            }
            vals[w++] = entry(op, eps, deg, i, j);
        }
    }
    free(deg);
}

/* Width of a column slab: ceil(F / c) rounded up to a multiple of 4 columns. */
int64_t orc_slab_width(int64_t F, int64_t c) { return 4 * ceil_div(F, 4 * c); }

/*
 * Algorithm 1, step by step: split S into b edge blocks, and for every hop split X_prev into
 * c column slabs; for each slab start X_tmp at zero, and for each block form Z = S^(j) X^(i)
 * and add it to X_tmp; concatenate the slabs, append to the list, and make the result the
 * next X_prev.  S^(j) is held as explicit triplets (row, col, value) so that the block
 * products are literal sparse-times-dense products.  `out` as in orc_propagate.
 * Returns -1 for an impossible (b, c).
 */
int orc_propagate_blocked(int op, double eps, int64_t n, const int64_t* rowptr, const int32_t* colidx, int64_t F,
                          const float* X, int64_t ldx, int K, int32_t b, int32_t c, double* out) {
    const int64_t m = orc_support_nnz(op, n, rowptr[n]);
    if (c < 1 || 4 * (int64_t)(c - 1) >= F + 3) return -1; /* a slab would be empty */
    int64_t* e_off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(b + 1));
    if (orc_block_offsets(m, b, e_off) != 0) {
        free(e_off);
        return -1;
    }
    int32_t* deg = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    orc_degrees(n, rowptr, deg);
    int64_t* rowptr_t = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int32_t* col_t = (int32_t*)malloc(sizeof(int32_t) * (size_t)m);
    orc_support(op, n, rowptr, colidx, rowptr_t, col_t);
    /* S as triplets in E's order */
    int32_t* row_t = (int32_t*)malloc(sizeof(int32_t) * (size_t)m);
    double* val_t = (double*)malloc(sizeof(double) * (size_t)m);
    for (int64_t i = 0; i < n; ++i)
        for (int64_t e = rowptr_t[i]; e < rowptr_t[i + 1]; ++e) {
            row_t[e] = (int32_t)i;
            val_t[e] = entry(op, eps, deg, i, col_t[e]);
        }
    const int64_t w = orc_slab_width(F, c);
    double* xprev = (double*)malloc(sizeof(double) * (size_t)n * (size_t)F);
    double* xtmp = (double*)malloc(sizeof(double) * (size_t)n * (size_t)w);
    double* ztmp = (double*)malloc(sizeof(double) * (size_t)n * (size_t)w);
    for (int64_t i = 0; i < n; ++i)
        for (int64_t f = 0; f < F; ++f) xprev[i * F + f] = (double)X[i * ldx + f];
    for (int k = 0; k < K; ++k) {
        double* xconc = out + (size_t)k * (size_t)n * (size_t)F;
        for (int32_t i = 0; i < c; ++i) {
            const int64_t f_lo = i * w, f_hi = (i + 1) * w < F ? (i + 1) * w : F;
            const int64_t wi = f_hi - f_lo;
            memset(xtmp, 0, sizeof(double) * (size_t)n * (size_t)w);
            for (int32_t j = 0; j < b; ++j) {
                memset(ztmp, 0, sizeof(double) * (size_t)n * (size_t)w);
                for (int64_t e = e_off[j]; e < e_off[j + 1]; ++e) /* Z = S^(j) X^(i) */
                    for (int64_t f = 0; f < wi; ++f)
                        ztmp[(int64_t)row_t[e] * w + f] += val_t[e] * xprev[(int64_t)col_t[e] * F + f_lo + f];
                for (int64_t t = 0; t < n * w; ++t) xtmp[t] += ztmp[t]; /* X_tmp = X_tmp + Z */
            }
            for (int64_t r = 0; r < n; ++r) /* concat: slab i occupies columns [f_lo, f_hi) */
                for (int64_t f = 0; f < wi; ++f) xconc[r * F + f_lo + f] = xtmp[r * w + f];
        }
        memcpy(xprev, xconc, sizeof(double) * (size_t)n * (size_t)F);
    }
    free(ztmp);
    free(xtmp);
    free(xprev);
    free(val_t);
    free(row_t);
    free(col_t);
    free(rowptr_t);
    free(deg);
    free(e_off);
    return 0;
}

/* ------------------------------------------------------------------ first dense stage of an LC model */

/*
 * Eq. 9 (the LC version of JKNet): every term of COMB starts with  S^k X W_1 , the k-th
 * precomputed hop times the first weight matrix, followed by the activation sigma (ReLU in
 * the paper's experimental settings) whenever another layer follows.  Training runs on
 * mini-batches of rows (batch size 4096 in the settings), so the stage is
 *     Y[i][h] = act( sum_f  Xk[batch[i]][f] * Wt[h][f] ),   i < B, h < H,
 * with Wt the weight stored as [H, F] (one row per output unit).  `batch` == NULL means rows
 * 0..B-1.  Yabs, when given, receives sum_f |Xk| |Wt| (the scale of the rounding error of any
 * finite-precision evaluation).  fp64 throughout, f ascending.
 */
void orc_lc_first_layer(int64_t B, const int64_t* batch, int64_t F, const float* Xk, int64_t ldx, int64_t H,
                        const float* Wt, int64_t ldw, int relu, double* Y, double* Yabs) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < B; ++i) {
        const float* x = Xk + (batch ? batch[i] : i) * ldx;
        for (int64_t h = 0; h < H; ++h) {
            const float* w = Wt + h * ldw;
            double s = 0.0, a = 0.0;
            for (int64_t f = 0; f < F; ++f) {
                s += (double)x[f] * (double)w[f];
                a += fabs((double)x[f]) * fabs((double)w[f]);
            }
            if (relu && s < 0.0) s = 0.0;
            Y[i * H + h] = s;
            if (Yabs) Yabs[i * H + h] = a;
        }
    }
}
