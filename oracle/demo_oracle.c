/*
 * DeMo per-step optimizer transform -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, fp64 restatement of what the path computes, written from the paper
 * (arXiv 2411.19870) step by step: Algorithm 1 (main body), the appendix algorithm
 * "Decoupled Momentum Optimization", CompressChunks and Decompress&Aggregate.
 * It shares no code, table or constant with the CUDA library; only tests/, the smoke
 * check and the benchmark's cpu-baseline leg may call it.
 *
 * Conventions: s = chunk size, rows = s for a 2-D tile and 1 for a 1-D segment,
 * M = rows*s elements per chunk, k_eff = min(k, M), C = s x s orthonormal DCT-II matrix.
 * Everything is double precision; inputs are the exact values of the fp32 / bf16 bits the
 * GPU sees, upcast by the caller.  The only parallelism is an OpenMP loop ACROSS chunks;
 * inside a chunk there is no blocking, fusion or reordering beyond the definitions.
 *
 * Readings taken where the paper is silent or at odds with itself (listed in the design
 * notes too):
 *   - momentum update is m <- beta*m + g (every algorithm listing), not the (1-beta) form
 *     of the Section 2.1 text equation;
 *   - aggregation is the plain sum over workers, in worker order (Decompress&Aggregate) by default;
 *     the mean over workers (Section 2.1, AvgAllGather) and the per-coordinate count-normalised
 *     mean with 0/0 = 0 (appendix algorithm "Sparse Top-k Averaging") are selectable, as is the
 *     identity in place of the sign for the transform phi of Section 2.1;
 *   - momentum subtraction m <- B - alpha * IDCT(kept) (Section 2.1, "Momentum Subtraction as Error
 *     Feedback", alpha in (0, 1]); alpha = 1 is what every algorithm listing uses and the default;
 *   - exactly k_eff coefficients per chunk (||Q_hat||_0 = k, Section 2.1); ties at the
 *     k-th magnitude go to the lowest flat index;
 *   - sign(0) = 0 (the sign lemmas of the appendix treat sign(y) = 0 as a legal case);
 *   - the DCT is the orthonormal DCT-II ("unitary", P^T = P^-1, appendix Sec. B.1.2);
 *   - any other orthonormal basis (identity, Gram-Schmidt of a Gaussian matrix: Section 4.2) is passed
 *     in as an s x s matrix whose ROWS are the basis vectors, and is used for both axes of a 2-D chunk.
 *
 * Parity pins live in tests/test_oracle_pins.py (closed forms, scipy's DCT, Parseval,
 * brute force on 8x8, the paper's 128x512 blocking example, the sqrt(1-k/M) bound with its
 * equality case, the lossless k = M case).  The particular choice among exactly tied
 * magnitudes is this repo's convention: "parity unpinned" by the paper for that choice.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t idx;
    float val;
} oracle_record; /* 8 bytes, little-endian: flat index inside the chunk, fp32 value */

/* ---------------------------------------------------------------------------------------
 * DCT basis.  Orthonormal DCT-II of dimension s:
 *   C[u][n] = a_u * cos(pi*(2n+1)*u / (2s)),  a_0 = sqrt(1/s), a_u = sqrt(2/s) for u > 0.
 * (Section 2.1 "DCT ... precomputed only once"; appendix B.1.2: unitary, P^T = P^-1.)
 * ------------------------------------------------------------------------------------- */
void oracle_dct_matrix(int s, double *C)
{
    const double pi = 3.14159265358979323846264338327950288;
    for (int u = 0; u < s; ++u) {
        double a = (u == 0) ? sqrt(1.0 / (double)s) : sqrt(2.0 / (double)s);
        for (int n = 0; n < s; ++n)
            C[(size_t)u * s + n] = a * cos(pi * (double)(2 * n + 1) * (double)u / (2.0 * (double)s));
    }
}

/* The transform of a chunk is any orthonormal s x s matrix P with rows as basis vectors (Q = P B P^T,
 * inverse P^T Q P): the DCT above, the identity ("no transformation") or a random orthonormal matrix
 * (Section 4.2, "Choice of Linear Projections").  `basis` NULL selects the DCT. */
static void chunk_basis(int s, const double *basis, double *C)
{
    if (basis)
        memcpy(C, basis, sizeof(double) * (size_t)s * s);
    else
        oracle_dct_matrix(s, C);
}

/* Gram-Schmidt process on the rows of G (s x s, entries drawn from N(0,1) by the caller with the step
 * number as the seed, Section 4.2): row j of P is row j of G minus its components along rows 0..j-1 of
 * P, scaled to unit length.  The components are removed one after the other from the running vector
 * (the "modified" ordering, identical in exact arithmetic).  Returns -1 when a row has no component
 * left (G singular to rounding), 0 otherwise. */
int oracle_gram_schmidt(int s, const double *G, double *P)
{
    for (int j = 0; j < s; ++j) {
        double *p = P + (size_t)j * s;
        double scale = 0.0;
        for (int n = 0; n < s; ++n) {
            p[n] = G[(size_t)j * s + n];
            scale += p[n] * p[n];
        }
        for (int i = 0; i < j; ++i) {
            const double *q = P + (size_t)i * s;
            double dot = 0.0;
            for (int n = 0; n < s; ++n) dot += p[n] * q[n];
            for (int n = 0; n < s; ++n) p[n] -= dot * q[n];
        }
        double nrm = 0.0;
        for (int n = 0; n < s; ++n) nrm += p[n] * p[n];
        if (!(nrm > 1e-24 * scale)) return -1;
        nrm = sqrt(nrm);
        for (int n = 0; n < s; ++n) p[n] /= nrm;
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * Blocking operator (appendix B.1.2):
 *   (B_{k0,k1}(X))[j0][j1] = X[k0*s0 + j0][k1*s1 + j1],   X is n0 x n1 row-major, n1 = c1*s1.
 * General rectangular chunk s0 x s1 so that the paper's 128x512 / 16x32 example can be
 * checked; the hot path uses s0 = s1 = s (2-D) or s0 = 1 (1-D, n0 = 1).
 * ------------------------------------------------------------------------------------- */
void oracle_block_extract(const double *X, int64_t n1, int s0, int s1, int64_t k0, int64_t k1, double *B)
{
    for (int j0 = 0; j0 < s0; ++j0)
        for (int j1 = 0; j1 < s1; ++j1)
            B[(size_t)j0 * s1 + j1] = X[(size_t)(k0 * s0 + j0) * (size_t)n1 + (size_t)(k1 * s1 + j1)];
}

void oracle_block_insert(double *X, int64_t n1, int s0, int s1, int64_t k0, int64_t k1, const double *B)
{
    for (int j0 = 0; j0 < s0; ++j0)
        for (int j1 = 0; j1 < s1; ++j1)
            X[(size_t)(k0 * s0 + j0) * (size_t)n1 + (size_t)(k1 * s1 + j1)] = B[(size_t)j0 * s1 + j1];
}

/* ---------------------------------------------------------------------------------------
 * Separable transform T (Section 2.1, appendix B.1.2), d in {1, 2}, P = C:
 *   2-D: Q[u][v] = sum_i sum_j C[u][i] * C[v][j] * B[i][j]        (= C B C^T)
 *   1-D: q[v]    = sum_j C[v][j] * b[j]
 * Inverse uses the transposes (C is unitary):
 *   2-D: R[i][j] = sum_u sum_v C[u][i] * C[v][j] * Q[u][v]        (= C^T Q C)
 *   1-D: r[j]    = sum_v C[v][j] * q[v]
 * Written as the product of two plain matrix products (rows first, then columns).
 * ------------------------------------------------------------------------------------- */
void oracle_forward(int s, int rows, const double *C, const double *B, double *Q)
{
    double *T = (double *)malloc(sizeof(double) * (size_t)rows * s);
    /* along the last axis: T[i][v] = sum_j C[v][j] B[i][j] */
    for (int i = 0; i < rows; ++i)
        for (int v = 0; v < s; ++v) {
            double acc = 0.0;
            for (int j = 0; j < s; ++j) acc += C[(size_t)v * s + j] * B[(size_t)i * s + j];
            T[(size_t)i * s + v] = acc;
        }
    if (rows == 1) {
        memcpy(Q, T, sizeof(double) * (size_t)s);
    } else {
        /* along the first axis: Q[u][v] = sum_i C[u][i] T[i][v] */
        for (int u = 0; u < s; ++u)
            for (int v = 0; v < s; ++v) {
                double acc = 0.0;
                for (int i = 0; i < s; ++i) acc += C[(size_t)u * s + i] * T[(size_t)i * s + v];
                Q[(size_t)u * s + v] = acc;
            }
    }
    free(T);
}

void oracle_inverse(int s, int rows, const double *C, const double *Q, double *R)
{
    double *T = (double *)malloc(sizeof(double) * (size_t)rows * s);
    /* along the last axis with C^T: T[u][j] = sum_v C[v][j] Q[u][v] */
    for (int u = 0; u < rows; ++u)
        for (int j = 0; j < s; ++j) {
            double acc = 0.0;
            for (int v = 0; v < s; ++v) acc += C[(size_t)v * s + j] * Q[(size_t)u * s + v];
            T[(size_t)u * s + j] = acc;
        }
    if (rows == 1) {
        memcpy(R, T, sizeof(double) * (size_t)s);
    } else {
        /* along the first axis with C^T: R[i][j] = sum_u C[u][i] T[u][j] */
        for (int i = 0; i < s; ++i)
            for (int j = 0; j < s; ++j) {
                double acc = 0.0;
                for (int u = 0; u < s; ++u) acc += C[(size_t)u * s + i] * T[(size_t)u * s + j];
                R[(size_t)i * s + j] = acc;
            }
    }
    free(T);
}

/* ---------------------------------------------------------------------------------------
 * Top-k (Section 2.1 "Top-k Sparsification"; appendix algorithm: thr = k-th largest
 * magnitude).  Definition written out: order ALL M coefficients by (|q| descending, flat
 * index ascending) with a full sort, keep the first k_eff, report them by ascending index.
 * a_k / a_k1 receive the k_eff-th and (k_eff+1)-th magnitudes of that order (a_k1 = 0 when
 * k_eff = M).
 * ------------------------------------------------------------------------------------- */
typedef struct {
    double mag;
    int32_t idx;
} mag_idx;

static int cmp_mag_desc_idx_asc(const void *pa, const void *pb)
{
    const mag_idx *a = (const mag_idx *)pa, *b = (const mag_idx *)pb;
    if (a->mag > b->mag) return -1;
    if (a->mag < b->mag) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

static int cmp_int32_asc(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

void oracle_topk(int M, int k, const double *Q, int32_t *idx_out, double *a_k, double *a_k1)
{
    int k_eff = k < M ? k : M;
    mag_idx *order = (mag_idx *)malloc(sizeof(mag_idx) * (size_t)M);
    for (int i = 0; i < M; ++i) {
        order[i].mag = fabs(Q[i]);
        order[i].idx = i;
    }
    qsort(order, (size_t)M, sizeof(mag_idx), cmp_mag_desc_idx_asc);
    for (int i = 0; i < k_eff; ++i) idx_out[i] = order[i].idx;
    qsort(idx_out, (size_t)k_eff, sizeof(int32_t), cmp_int32_asc);
    if (a_k) *a_k = order[k_eff - 1].mag;
    if (a_k1) *a_k1 = (k_eff < M) ? order[k_eff].mag : 0.0;
    free(order);
}

/* ---------------------------------------------------------------------------------------
 * One chunk of CompressChunks (Algorithm "CompressChunks", Algorithm 1 worker loop):
 *   B     = beta*m + g                                   (momentum update)
 *   Q     = T(B; C)                                      (chunk DCT)
 *   Q_sp  = Top-k(Q)                                     (k_eff records, ascending index)
 *   m_new = B - alpha * T^-1(Q_sp; C^T)                  (momentum subtraction)
 * forced_idx (nullable): use this index set (k_eff ascending indices) instead of the
 * oracle's own top-k -- used by the comparison rule for chunks whose k-th / (k+1)-th
 * magnitudes are too close to pin the set.
 * Outputs (any may be NULL except m_new): Q_out[M], idx_out[k_eff], val_out[k_eff] (fp64
 * coefficient at each index), gap[2] = {a_k, a_k1} of the oracle's OWN order.
 * ------------------------------------------------------------------------------------- */
void oracle_compress_chunk(int s, int rows, int k, double beta, double alpha, const double *C, const double *g,
                           const double *m, const int32_t *forced_idx, double *Q_out,
                           int32_t *idx_out, double *val_out, double *m_new, double *gap)
{
    const int M = rows * s;
    const int k_eff = k < M ? k : M;
    double *B = (double *)malloc(sizeof(double) * (size_t)M);
    double *Q = (double *)malloc(sizeof(double) * (size_t)M);
    double *Qsp = (double *)calloc((size_t)M, sizeof(double));
    double *R = (double *)malloc(sizeof(double) * (size_t)M);
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)k_eff);

    for (int i = 0; i < M; ++i) B[i] = beta * m[i] + g[i];
    oracle_forward(s, rows, C, B, Q);
    double a_k = 0.0, a_k1 = 0.0;
    oracle_topk(M, k, Q, idx, &a_k, &a_k1);
    if (gap) {
        gap[0] = a_k;
        gap[1] = a_k1;
    }
    if (forced_idx) memcpy(idx, forced_idx, sizeof(int32_t) * (size_t)k_eff);
    for (int i = 0; i < k_eff; ++i) Qsp[idx[i]] = Q[idx[i]];
    oracle_inverse(s, rows, C, Qsp, R);
    for (int i = 0; i < M; ++i) m_new[i] = B[i] - alpha * R[i];

    if (Q_out) memcpy(Q_out, Q, sizeof(double) * (size_t)M);
    if (idx_out) memcpy(idx_out, idx, sizeof(int32_t) * (size_t)k_eff);
    if (val_out)
        for (int i = 0; i < k_eff; ++i) val_out[i] = Q[idx[i]];
    free(B);
    free(Q);
    free(Qsp);
    free(R);
    free(idx);
}

/* Batch of independent chunks given as tiles: g, m are [n][M]; outputs [n][...]. */
void oracle_compress_chunks(int64_t n, int s, int rows, int k, double beta, double alpha, const double *g,
                            const double *m, const int32_t *forced_idx, double *Q_out,
                            int32_t *idx_out, double *val_out, double *m_new, double *gap,
                            int n_threads, const double *basis)
{
    const int M = rows * s;
    const int k_eff = k < M ? k : M;
    double *C = (double *)malloc(sizeof(double) * (size_t)s * s);
    chunk_basis(s, basis, C);
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : omp_get_max_threads())
#endif
    for (int64_t c = 0; c < n; ++c) {
        oracle_compress_chunk(s, rows, k, beta, alpha, C, g + c * M, m + c * M,
                              forced_idx ? forced_idx + c * k_eff : NULL,
                              Q_out ? Q_out + c * M : NULL, idx_out ? idx_out + c * k_eff : NULL,
                              val_out ? val_out + c * k_eff : NULL, m_new + c * M,
                              gap ? gap + c * 2 : NULL);
    }
    free(C);
}

/* ---------------------------------------------------------------------------------------
 * Whole tensor, one worker: blocking + oracle_compress_chunk per chunk + un-blocking.
 * ndim 1: n0 ignored (=1), n1 = length; ndim 2: n0 x n1 row-major.  n0 % s == 0 (2-D) and
 * n1 % s == 0 are the caller's responsibility (returns -1 otherwise).
 * m is updated in place.  Chunk order is row-major over the (c0, c1) chunk grid.
 * records: [n_chunks][k_eff] of {int32 idx, float val} -- val is the fp64 coefficient
 * rounded once to fp32.  val64 / gap / forced_idx as in the chunk routine (nullable).
 * ------------------------------------------------------------------------------------- */
int oracle_compress_tensor(int ndim, int64_t n0, int64_t n1, int s, int k, double beta, double alpha, const double *g,
                           double *m, const int32_t *forced_idx, oracle_record *records, double *val64,
                           double *gap, int n_threads, const double *basis)
{
    if (ndim != 1 && ndim != 2) return -1;
    if (ndim == 1) n0 = 1;
    const int rows = (ndim == 2) ? s : 1;
    if (n1 % s != 0 || (ndim == 2 && n0 % s != 0)) return -1;
    const int64_t c0 = (ndim == 2) ? n0 / s : 1, c1 = n1 / s;
    const int M = rows * s;
    const int k_eff = k < M ? k : M;
    double *C = (double *)malloc(sizeof(double) * (size_t)s * s);
    chunk_basis(s, basis, C);
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 4) num_threads(n_threads > 0 ? n_threads : omp_get_max_threads())
#endif
    for (int64_t c = 0; c < c0 * c1; ++c) {
        const int64_t k0 = c / c1, k1 = c % c1;
        double *gt = (double *)malloc(sizeof(double) * (size_t)M);
        double *mt = (double *)malloc(sizeof(double) * (size_t)M);
        double *mn = (double *)malloc(sizeof(double) * (size_t)M);
        double *vals = (double *)malloc(sizeof(double) * (size_t)k_eff);
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)k_eff);
        oracle_block_extract(g, n1, rows, s, k0, k1, gt);
        oracle_block_extract(m, n1, rows, s, k0, k1, mt);
        oracle_compress_chunk(s, rows, k, beta, alpha, C, gt, mt, forced_idx ? forced_idx + c * k_eff : NULL, NULL,
                              idx, vals, mn, gap ? gap + c * 2 : NULL);
        oracle_block_insert(m, n1, rows, s, k0, k1, mn);
        for (int i = 0; i < k_eff; ++i) {
            records[c * k_eff + i].idx = idx[i];
            records[c * k_eff + i].val = (float)vals[i];
            if (val64) val64[c * k_eff + i] = vals[i];
        }
        free(gt);
        free(mt);
        free(mn);
        free(vals);
        free(idx);
    }
    free(C);
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * One chunk of Decompress&Aggregate + the parameter update (Algorithm 1, server side):
 *   S = 0;  for w = 0..W-1 in order:  S[idx] += val  for that worker's k_eff records
 *   agg = 0: S as is (sum);  agg = 1: S / W (mean, AvgAllGather);
 *   agg = 2: S[i] / n[i] with n[i] the number of workers that sent coordinate i, 0/0 = 0
 *            (appendix algorithm "Sparse Top-k Averaging")
 *   R = T^-1(S; C^T)
 *   phi = 0: sg = (R > 0) - (R < 0)  (Signum, sign(0) = 0);  phi = 1: sg = R  (SGD-style, Section 2.1)
 *   x_new = x - lr * (sg + wd * x)                          (decoupled weight decay)
 * recs[w] points at that worker's k_eff records for this chunk (fp32 values as stored).
 * R_out (nullable) receives the reconstructed momentum chunk.
 * ------------------------------------------------------------------------------------- */
void oracle_decode_chunk(int s, int rows, int k_eff, int W, int agg, int phi, const double *C,
                         const oracle_record *const *recs, const double *x, double lr, double wd, double *x_new,
                         double *R_out)
{
    const int M = rows * s;
    double *S = (double *)calloc((size_t)M, sizeof(double));
    int *cnt = (int *)calloc((size_t)M, sizeof(int));
    double *R = (double *)malloc(sizeof(double) * (size_t)M);
    for (int w = 0; w < W; ++w)
        for (int i = 0; i < k_eff; ++i) {
            S[recs[w][i].idx] += (double)recs[w][i].val;
            cnt[recs[w][i].idx] += 1;
        }
    if (agg == 1)
        for (int i = 0; i < M; ++i) S[i] /= (double)W;
    if (agg == 2)
        for (int i = 0; i < M; ++i) S[i] = cnt[i] ? S[i] / (double)cnt[i] : 0.0;
    free(cnt);
    oracle_inverse(s, rows, C, S, R);
    for (int i = 0; i < M; ++i) {
        double sg = (phi == 1) ? R[i] : (double)((R[i] > 0.0) - (R[i] < 0.0));
        x_new[i] = x[i] - lr * (sg + wd * x[i]);
    }
    if (R_out) memcpy(R_out, R, sizeof(double) * (size_t)M);
    free(S);
    free(R);
}

/* Batch of independent chunks: recs is [W][n][k_eff] contiguous; x, x_new, R_out are [n][M]. */
void oracle_decode_chunks(int64_t n, int s, int rows, int k_eff, int W, int agg, int phi, const oracle_record *recs,
                          const double *x, double lr, double wd, double *x_new, double *R_out, int n_threads,
                          const double *basis)
{
    const int M = rows * s;
    double *C = (double *)malloc(sizeof(double) * (size_t)s * s);
    chunk_basis(s, basis, C);
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : omp_get_max_threads())
#endif
    for (int64_t c = 0; c < n; ++c) {
        const oracle_record **rw = (const oracle_record **)malloc(sizeof(void *) * (size_t)W);
        for (int w = 0; w < W; ++w) rw[w] = recs + ((size_t)w * (size_t)n + (size_t)c) * (size_t)k_eff;
        oracle_decode_chunk(s, rows, k_eff, W, agg, phi, C, rw, x + c * M, lr, wd, x_new + c * M,
                            R_out ? R_out + c * M : NULL);
        free(rw);
    }
    free(C);
}

/* Whole tensor: payloads[w] points at worker w's [n_chunks][k_eff] records for THIS tensor.
 * x is updated in place; R_out (nullable) receives the reconstructed global momentum. */
int oracle_decode_tensor(int ndim, int64_t n0, int64_t n1, int s, int k, int W, int agg, int phi,
                         const oracle_record *const *payloads, double *x, double lr, double wd, double *R_out,
                         int n_threads, const double *basis)
{
    if (ndim != 1 && ndim != 2) return -1;
    if (ndim == 1) n0 = 1;
    const int rows = (ndim == 2) ? s : 1;
    if (n1 % s != 0 || (ndim == 2 && n0 % s != 0)) return -1;
    const int64_t c0 = (ndim == 2) ? n0 / s : 1, c1 = n1 / s;
    const int M = rows * s;
    const int k_eff = k < M ? k : M;
    double *C = (double *)malloc(sizeof(double) * (size_t)s * s);
    chunk_basis(s, basis, C);
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 4) num_threads(n_threads > 0 ? n_threads : omp_get_max_threads())
#endif
    for (int64_t c = 0; c < c0 * c1; ++c) {
        const int64_t k0 = c / c1, k1 = c % c1;
        double *xt = (double *)malloc(sizeof(double) * (size_t)M);
        double *xn = (double *)malloc(sizeof(double) * (size_t)M);
        double *Rt = (double *)malloc(sizeof(double) * (size_t)M);
        const oracle_record **rw = (const oracle_record **)malloc(sizeof(void *) * (size_t)W);
        for (int w = 0; w < W; ++w) rw[w] = payloads[w] + (size_t)c * (size_t)k_eff;
        oracle_block_extract(x, n1, rows, s, k0, k1, xt);
        oracle_decode_chunk(s, rows, k_eff, W, agg, phi, C, rw, xt, lr, wd, xn, Rt);
        oracle_block_insert(x, n1, rows, s, k0, k1, xn);
        if (R_out) oracle_block_insert(R_out, n1, rows, s, k0, k1, Rt);
        free(xt);
        free(xn);
        free(Rt);
        free(rw);
    }
    free(C);
    return 0;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
