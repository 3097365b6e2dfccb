/*
 * CPU oracle for HDT hierarchical attention.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain, slow definition the CUDA path is checked against.
 * It shares no code, header, table or helper with the CUDA library and must
 * never be used by the product path; only tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may load it.
 *
 * What it computes (paper, section "Hierarchical Document Transformer",
 * paragraph "Hierarchical Attention"):
 *   mask      M_ij = 1 iff token j is token i's parent, one of its siblings
 *             (same parent, same level, i itself included) or one of its
 *             children; tokens of different sequences and PAD tokens never
 *             interact.  This is the parent/sibling/child rule stated in the
 *             text; for 3-level documents it equals the OR of the per-level
 *             masks of the attention-mask equation (checked in the tests).
 *   forward   A = Q K^T / sqrt(d_k); masked entries are -inf; S = softmax(A)
 *             row-wise; O = S V   (the hierarchical attention equation).
 *             LSE_i = log sum_j exp(A_ij) over unmasked j.
 *   backward  the derivative of the forward map (the paper prints none):
 *             dV = S^T dO; dP = dO V^T; delta_i = sum_j S_ij dP_ij;
 *             dS = S o (dP - delta); dQ = scale dS K; dK = scale dS^T Q.
 *
 * The n x n mask of a sequence is materialised as bytes, attention is written
 * as "for i, for j if M[i][j]" in fp64 with no tiling, no online softmax and
 * no reordering.  PAD rows give O = 0, LSE = -inf and zero gradients.
 *
 * Every function here is pinned by tests/test_oracle_pins.py (hand-worked
 * hierarchy, closed forms, reductions to dense softmax attention, finite
 * differences, brute-force tree walks); no part is parity-unpinned.
 *
 * Layouts: q,k,v,do and outputs o,dq,dk,dv are [T, H, d] (token-major,
 * packed); lse is [H, T].  Inputs are fp64 (in_f32 = 0) or fp32 (in_f32 = 1)
 * arrays; every output is fp64.  parent[] is relative to the start of the
 * token's own sequence.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double ld(const void *p, size_t idx, int f32) {
    return f32 ? (double)((const float *)p)[idx] : ((const double *)p)[idx];
}

/*
 * Directed variants of the rule (paper, "Mathematical Reasoning Tasks": the ListOps attention
 * patterns).  Three groups of entries can be switched off: a token attending to its parent
 * (bit 0; the variant where operands do not attend to their operators clears it), a token
 * attending to its other siblings (bit 1; the variant where operands do not attend to each
 * other clears it as well), a token attending to its children (bit 2).  The diagonal always
 * stays.  7 = the full rule of the section "Hierarchical Attention"; every function below uses
 * the value set here.
 */
static int g_directions = 7;
void hdt_oracle_set_directions(int bits) { g_directions = bits & 7; }

/* Parent / sibling / child rule on sequence-relative indices i, j. */
static int mask_rule(const int8_t *lv, const int32_t *pa, int i, int j) {
    if (lv[i] < 0 || lv[j] < 0) return 0;                 /* PAD */
    if (i == j) return 1;                                 /* a token is its own sibling */
    if (pa[i] == j) return (g_directions & 1) != 0;       /* j is the parent of i */
    if (pa[j] == i) return (g_directions & 4) != 0;       /* j is a child of i */
    if (pa[i] >= 0 && pa[i] == pa[j] && lv[i] == lv[j])   /* siblings */
        return (g_directions & 2) != 0;
    return 0;
}

int hdt_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Dense mask of sequence b: out[n*n] bytes, n = cu[b+1]-cu[b]. */
int hdt_oracle_mask(const int8_t *level, const int32_t *parent, const int32_t *cu,
                    int b, uint8_t *out) {
    const int s0 = cu[b], n = cu[b + 1] - cu[b];
    const int8_t *lv = level + s0;
    const int32_t *pa = parent + s0;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j)
            out[(size_t)i * n + j] = (uint8_t)mask_rule(lv, pa, i, j);
    return 0;
}

/* One mask row (sequence-relative i) of sequence b. */
static void mask_row(const int8_t *lv, const int32_t *pa, int n, int i, uint8_t *row) {
    for (int j = 0; j < n; ++j) row[j] = (uint8_t)mask_rule(lv, pa, i, j);
}

/* Softmax row i of one (sequence, head): S[j] for all j, returns LSE.  S is zero where masked. */
static double softmax_row(const void *q, const void *k, int f32, size_t s0, int n, int H, int d,
                          int h, int i, const uint8_t *mrow, double scale, double *S) {
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        S[j] = 0.0;
        if (!mrow[j]) continue;
        double a = 0.0;
        for (int c = 0; c < d; ++c)
            a += ld(q, ((s0 + i) * H + h) * (size_t)d + c, f32) *
                 ld(k, ((s0 + j) * H + h) * (size_t)d + c, f32);
        a *= scale;
        S[j] = a;
        if (a > m) m = a;
    }
    if (m == -INFINITY) return -INFINITY; /* PAD row: no key */
    double l = 0.0;
    for (int j = 0; j < n; ++j)
        if (mrow[j]) { S[j] = exp(S[j] - m); l += S[j]; }
    for (int j = 0; j < n; ++j)
        if (mrow[j]) S[j] /= l;
    return m + log(l);
}

/* Full forward over the batch. */
int hdt_oracle_fwd(const int8_t *level, const int32_t *parent, const int32_t *cu, int B,
                   int H, int d, const void *q, const void *k, const void *v, int in_f32,
                   double scale, double *o, double *lse) {
    const size_t T = (size_t)cu[B];
    for (int b = 0; b < B; ++b) {
        const size_t s0 = (size_t)cu[b];
        const int n = cu[b + 1] - cu[b];
        if (n == 0) continue;
        uint8_t *M = (uint8_t *)malloc((size_t)n * n);
        if (!M) return -1;
        hdt_oracle_mask(level, parent, cu, b, M);
#pragma omp parallel
        {
            double *S = (double *)malloc(sizeof(double) * n);
#pragma omp for collapse(2) schedule(dynamic, 16)
            for (int h = 0; h < H; ++h)
                for (int i = 0; i < n; ++i) {
                    const uint8_t *mrow = M + (size_t)i * n;
                    double L = softmax_row(q, k, in_f32, s0, n, H, d, h, i, mrow, scale, S);
                    lse[(size_t)h * T + s0 + i] = L;
                    double *oi = o + ((s0 + i) * H + h) * (size_t)d;
                    for (int c = 0; c < d; ++c) oi[c] = 0.0;
                    for (int j = 0; j < n; ++j)
                        if (mrow[j])
                            for (int c = 0; c < d; ++c)
                                oi[c] += S[j] * ld(v, ((s0 + j) * H + h) * (size_t)d + c, in_f32);
                }
            free(S);
        }
        free(M);
    }
    return 0;
}

/* Full backward over the batch (recomputes S from q, k). */
int hdt_oracle_bwd(const int8_t *level, const int32_t *parent, const int32_t *cu, int B,
                   int H, int d, const void *q, const void *k, const void *v, const void *d_o,
                   int in_f32, double scale, double *dq, double *dk, double *dv) {
    const size_t T = (size_t)cu[B];
    memset(dq, 0, sizeof(double) * T * H * d);
    memset(dk, 0, sizeof(double) * T * H * d);
    memset(dv, 0, sizeof(double) * T * H * d);
    for (int b = 0; b < B; ++b) {
        const size_t s0 = (size_t)cu[b];
        const int n = cu[b + 1] - cu[b];
        if (n == 0) continue;
        uint8_t *M = (uint8_t *)malloc((size_t)n * n);
        if (!M) return -1;
        hdt_oracle_mask(level, parent, cu, b, M);
#pragma omp parallel
        {
            double *S = (double *)malloc(sizeof(double) * n);
            double *dP = (double *)malloc(sizeof(double) * n);
#pragma omp for schedule(dynamic, 1)
            for (int h = 0; h < H; ++h)
                for (int i = 0; i < n; ++i) {
                    const uint8_t *mrow = M + (size_t)i * n;
                    double L = softmax_row(q, k, in_f32, s0, n, H, d, h, i, mrow, scale, S);
                    if (L == -INFINITY) continue;
                    const size_t ri = ((s0 + i) * H + h) * (size_t)d;
                    double delta = 0.0;
                    for (int j = 0; j < n; ++j) {
                        if (!mrow[j]) continue;
                        const size_t rj = ((s0 + j) * H + h) * (size_t)d;
                        double p = 0.0;
                        for (int c = 0; c < d; ++c) p += ld(d_o, ri + c, in_f32) * ld(v, rj + c, in_f32);
                        dP[j] = p;
                        delta += S[j] * p;
                    }
                    for (int j = 0; j < n; ++j) {
                        if (!mrow[j]) continue;
                        const size_t rj = ((s0 + j) * H + h) * (size_t)d;
                        const double dS = S[j] * (dP[j] - delta);
                        for (int c = 0; c < d; ++c) {
                            dv[rj + c] += S[j] * ld(d_o, ri + c, in_f32);
                            dq[ri + c] += scale * dS * ld(k, rj + c, in_f32);
                            dk[rj + c] += scale * dS * ld(q, ri + c, in_f32);
                        }
                    }
                }
            free(S);
            free(dP);
        }
        free(M);
    }
    return 0;
}

static int find_seq(const int32_t *cu, int B, int g) {
    for (int b = 0; b < B; ++b)
        if (g >= cu[b] && g < cu[b + 1]) return b;
    return -1;
}

/*
 * Sampled forward / dQ: for each global token id rows[r] compute, for every head,
 * O (o_rows [nrows,H,d]), LSE (lse_rows [nrows,H]) and, if d_o != NULL, dQ
 * (dq_rows [nrows,H,d]).  Only the sampled mask rows are materialised.
 */
int hdt_oracle_rows(const int8_t *level, const int32_t *parent, const int32_t *cu, int B,
                    int H, int d, const void *q, const void *k, const void *v, const void *d_o,
                    int in_f32, double scale, const int32_t *rows, int nrows,
                    double *o_rows, double *lse_rows, double *dq_rows) {
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < nrows; ++r) {
        const int b = find_seq(cu, B, rows[r]);
        if (b < 0) { err = 1; continue; }
        const size_t s0 = (size_t)cu[b];
        const int n = cu[b + 1] - cu[b], i = rows[r] - cu[b];
        uint8_t *mrow = (uint8_t *)malloc(n);
        double *S = (double *)malloc(sizeof(double) * n);
        mask_row(level + s0, parent + s0, n, i, mrow);
        for (int h = 0; h < H; ++h) {
            double L = softmax_row(q, k, in_f32, s0, n, H, d, h, i, mrow, scale, S);
            lse_rows[(size_t)r * H + h] = L;
            double *oi = o_rows + ((size_t)r * H + h) * d;
            for (int c = 0; c < d; ++c) oi[c] = 0.0;
            for (int j = 0; j < n; ++j)
                if (mrow[j])
                    for (int c = 0; c < d; ++c)
                        oi[c] += S[j] * ld(v, ((s0 + j) * H + h) * (size_t)d + c, in_f32);
            if (d_o && dq_rows) {
                double *dqi = dq_rows + ((size_t)r * H + h) * d;
                for (int c = 0; c < d; ++c) dqi[c] = 0.0;
                if (L == -INFINITY) continue;
                const size_t ri = ((s0 + i) * H + h) * (size_t)d;
                double delta = 0.0;
                for (int j = 0; j < n; ++j) {
                    if (!mrow[j]) continue;
                    const size_t rj = ((s0 + j) * H + h) * (size_t)d;
                    double p = 0.0;
                    for (int c = 0; c < d; ++c) p += ld(d_o, ri + c, in_f32) * ld(v, rj + c, in_f32);
                    delta += S[j] * p;
                }
                for (int j = 0; j < n; ++j) {
                    if (!mrow[j]) continue;
                    const size_t rj = ((s0 + j) * H + h) * (size_t)d;
                    double p = 0.0;
                    for (int c = 0; c < d; ++c) p += ld(d_o, ri + c, in_f32) * ld(v, rj + c, in_f32);
                    const double dS = S[j] * (p - delta);
                    for (int c = 0; c < d; ++c) dqi[c] += scale * dS * ld(k, rj + c, in_f32);
                }
            }
        }
        free(mrow);
        free(S);
    }
    return err ? -2 : 0;
}

/*
 * Sampled dK / dV: for each global token id cols[r] (as a key), for every head,
 * dK and dV ([ncols,H,d]).  Every query row i with M_ij = 1 gets its own full
 * softmax row.
 */
int hdt_oracle_cols(const int8_t *level, const int32_t *parent, const int32_t *cu, int B,
                    int H, int d, const void *q, const void *k, const void *v, const void *d_o,
                    int in_f32, double scale, const int32_t *cols, int ncols,
                    double *dk_cols, double *dv_cols) {
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < ncols; ++r) {
        const int b = find_seq(cu, B, cols[r]);
        if (b < 0) { err = 1; continue; }
        const size_t s0 = (size_t)cu[b];
        const int n = cu[b + 1] - cu[b], j = cols[r] - cu[b];
        const int8_t *lv = level + s0;
        const int32_t *pa = parent + s0;
        uint8_t *mrow = (uint8_t *)malloc(n);
        double *S = (double *)malloc(sizeof(double) * n);
        for (int h = 0; h < H; ++h) {
            double *dkj = dk_cols + ((size_t)r * H + h) * d;
            double *dvj = dv_cols + ((size_t)r * H + h) * d;
            for (int c = 0; c < d; ++c) dkj[c] = dvj[c] = 0.0;
            const size_t rj = ((s0 + j) * H + h) * (size_t)d;
            for (int i = 0; i < n; ++i) {
                if (!mask_rule(lv, pa, i, j)) continue;
                mask_row(lv, pa, n, i, mrow);
                double L = softmax_row(q, k, in_f32, s0, n, H, d, h, i, mrow, scale, S);
                if (L == -INFINITY) continue;
                const size_t ri = ((s0 + i) * H + h) * (size_t)d;
                double delta = 0.0, pj = 0.0;
                for (int jj = 0; jj < n; ++jj) {
                    if (!mrow[jj]) continue;
                    const size_t rjj = ((s0 + jj) * H + h) * (size_t)d;
                    double p = 0.0;
                    for (int c = 0; c < d; ++c) p += ld(d_o, ri + c, in_f32) * ld(v, rjj + c, in_f32);
                    delta += S[jj] * p;
                    if (jj == j) pj = p;
                }
                const double dS = S[j] * (pj - delta);
                for (int c = 0; c < d; ++c) {
                    dvj[c] += S[j] * ld(d_o, ri + c, in_f32);
                    dkj[c] += scale * dS * ld(q, ri + c, in_f32);
                }
            }
        }
        free(mrow);
        free(S);
    }
    return err ? -2 : 0;
}

/* Softmax matrix S of one (sequence, head), dense n x n, for invariant tests. */
int hdt_oracle_probs(const int8_t *level, const int32_t *parent, const int32_t *cu, int b,
                     int H, int d, const void *q, const void *k, int in_f32, double scale,
                     int h, double *S_out) {
    const size_t s0 = (size_t)cu[b];
    const int n = cu[b + 1] - cu[b];
    uint8_t *M = (uint8_t *)malloc((size_t)n * n);
    if (!M) return -1;
    hdt_oracle_mask(level, parent, cu, b, M);
    for (int i = 0; i < n; ++i)
        softmax_row(q, k, in_f32, s0, n, H, d, h, i, M + (size_t)i * n, scale, S_out + (size_t)i * n);
    free(M);
    return 0;
}
