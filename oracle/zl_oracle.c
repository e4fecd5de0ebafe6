/*
 * TEST INFRASTRUCTURE -- fp64 CPU oracle for the coalesced attention engine.
 *
 * This file is the slow, plain definition that the CUDA path is checked against.  It is
 * never part of the product path: only tests, the smoke check and the benchmark's
 * cpu_baseline / reference arm may build or call it.  It shares no code with the CUDA
 * kernels.
 *
 * What it computes (paper Section II-A: dense bidirectional self-attention of a DiT
 * block; Section IV-D: attention is never mixed across sequences, and context-parallel
 * shards compute exact attention from the K/V chunks they are given):
 *
 *   for one logical problem (query rows I, key rows J, one head):
 *       s_ij  = scale * sum_c q[i][c] * k[j][c]
 *       LSE_i = log sum_j exp(s_ij)           (evaluated as m_i + log sum_j exp(s_ij - m_i))
 *       p_ij  = exp(s_ij - LSE_i)
 *       O_i   = sum_j p_ij * v[j]
 *       |J| = 0  ->  O_i = 0, LSE_i = -inf
 *
 *   merge of partial results (O_t, LSE_t) of the same query rows over disjoint key sets:
 *       LSE = M + log sum_t exp(LSE_t - M),  M = max_t LSE_t
 *       O   = sum_t exp(LSE_t - LSE) * O_t                 (all LSE_t = -inf -> O = 0, LSE = -inf)
 *
 *   analytic gradients for a loss with dL/dO = dO (no gradient flows through LSE):
 *       D_i   = sum_c dO[i][c] * O[i][c]
 *       dP_ij = sum_c dO[i][c] * v[j][c]
 *       dS_ij = p_ij * (dP_ij - D_i)
 *       dQ_i  = scale * sum_j dS_ij * k[j]
 *       dK_j  = scale * sum_i dS_ij * q[i]
 *       dV_j  = sum_i p_ij * dO[i]
 *
 * Every array is one head of fp64 values with a row stride given in elements, so a
 * caller can pass a view of a [rows, H, d] array.  Loops run in index order; the only
 * parallelism is OpenMP over independent output rows.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Query rows are processed in groups of ORC_GROUP rows that share each pass over the keys
 * (so a long key set is streamed from memory once per group instead of once per row); the
 * arithmetic of every row, and the order of its sums, is exactly the one written above. */
#define ORC_GROUP 8

/* Forward for query rows listed in `rows` (NULL: rows 0..n_rows-1).  Output r belongs to
 * query row rows[r]; O has n_rows rows with stride ldo, lse has n_rows entries. */
void orc_attn_fwd(const double* q, long ldq, const double* k, long ldk, const double* v, long ldv,
                  long n_kv, int d, double scale, const long* rows, long n_rows,
                  double* O, long ldo, double* lse) {
    const long n_groups = (n_rows + ORC_GROUP - 1) / ORC_GROUP;
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)ORC_GROUP * (size_t)(n_kv > 0 ? n_kv : 1));
#pragma omp for schedule(dynamic, 1)
        for (long g = 0; g < n_groups; ++g) {
            const long r0 = g * ORC_GROUP;
            const int nr = (int)((n_rows - r0 < ORC_GROUP) ? (n_rows - r0) : ORC_GROUP);
            const double* qi[ORC_GROUP];
            double m[ORC_GROUP], L[ORC_GROUP];
            for (int a = 0; a < nr; ++a) {
                const long i = rows ? rows[r0 + a] : (r0 + a);
                qi[a] = q + i * ldq;
                double* Oi = O + (r0 + a) * ldo;
                for (int c = 0; c < d; ++c) Oi[c] = 0.0;
                m[a] = -INFINITY;
            }
            if (n_kv <= 0) {
                for (int a = 0; a < nr; ++a) lse[r0 + a] = -INFINITY;
                continue;
            }
            for (long j = 0; j < n_kv; ++j) {          /* scores and row maxima */
                const double* kj = k + j * ldk;
                for (int a = 0; a < nr; ++a) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += qi[a][c] * kj[c];
                    const double sj = scale * acc;
                    s[(size_t)a * n_kv + j] = sj;
                    if (sj > m[a]) m[a] = sj;
                }
            }
            for (int a = 0; a < nr; ++a) {             /* log-sum-exp */
                double l = 0.0;
                for (long j = 0; j < n_kv; ++j) l += exp(s[(size_t)a * n_kv + j] - m[a]);
                L[a] = m[a] + log(l);
                lse[r0 + a] = L[a];
            }
            for (long j = 0; j < n_kv; ++j) {          /* O_i = sum_j p_ij v_j */
                const double* vj = v + j * ldv;
                for (int a = 0; a < nr; ++a) {
                    const double p = exp(s[(size_t)a * n_kv + j] - L[a]);
                    double* Oi = O + (r0 + a) * ldo;
                    for (int c = 0; c < d; ++c) Oi[c] += p * vj[c];
                }
            }
        }
        free(s);
    }
}

/* Merge n_parts partial results of the same n_rows query rows.  O_parts[t] has row stride
 * ldp, lse_parts[t] has n_rows entries.  Parts are summed in ascending t. */
void orc_lse_merge(int n_parts, const double* const* O_parts, long ldp,
                   const double* const* lse_parts, long n_rows, int d,
                   double* O, long ldo, double* lse) {
#pragma omp parallel for schedule(static)
    for (long r = 0; r < n_rows; ++r) {
        double* Or = O + r * ldo;
        for (int c = 0; c < d; ++c) Or[c] = 0.0;
        double M = -INFINITY;
        for (int t = 0; t < n_parts; ++t)
            if (lse_parts[t][r] > M) M = lse_parts[t][r];
        if (n_parts == 0 || M == -INFINITY) { lse[r] = -INFINITY; continue; }
        double z = 0.0;
        for (int t = 0; t < n_parts; ++t) z += exp(lse_parts[t][r] - M);
        const double L = M + log(z);
        lse[r] = L;
        for (int t = 0; t < n_parts; ++t) {
            const double w = exp(lse_parts[t][r] - L);
            const double* Ot = O_parts[t] + r * ldp;
            for (int c = 0; c < d; ++c) Or[c] += w * Ot[c];
        }
    }
}

/* D_i = sum_c dO[i][c] * O[i][c] for rows 0..n_q-1. */
void orc_attn_bwd_delta(const double* dO, long lddo, const double* O, long ldo,
                        long n_q, int d, double* D) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n_q; ++i) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += dO[i * lddo + c] * O[i * ldo + c];
        D[i] = acc;
    }
}

/* dQ for the query rows in `rows` (NULL: 0..n_rows-1) against key rows 0..n_kv-1.
 * lse and D are indexed by absolute query row. Output r belongs to rows[r]. */
void orc_attn_bwd_dq(const double* q, long ldq, const double* k, long ldk, const double* v, long ldv,
                     const double* dO, long lddo, const double* lse, const double* D,
                     long n_kv, int d, double scale, const long* rows, long n_rows,
                     double* dQ, long lddq) {
    const long n_groups = (n_rows + ORC_GROUP - 1) / ORC_GROUP;
#pragma omp parallel for schedule(dynamic, 1)
    for (long g = 0; g < n_groups; ++g) {
        const long r0 = g * ORC_GROUP;
        const int nr = (int)((n_rows - r0 < ORC_GROUP) ? (n_rows - r0) : ORC_GROUP);
        long idx[ORC_GROUP];
        for (int a = 0; a < nr; ++a) {
            idx[a] = rows ? rows[r0 + a] : (r0 + a);
            double* dqi = dQ + (r0 + a) * lddq;
            for (int c = 0; c < d; ++c) dqi[c] = 0.0;
        }
        if (n_kv <= 0) continue;
        for (long j = 0; j < n_kv; ++j) {
            const double* kj = k + j * ldk;
            const double* vj = v + j * ldv;
            for (int a = 0; a < nr; ++a) {
                const long i = idx[a];
                const double* qi = q + i * ldq;
                const double* doi = dO + i * lddo;
                double* dqi = dQ + (r0 + a) * lddq;
                double s = 0.0, dp = 0.0;
                for (int c = 0; c < d; ++c) { s += qi[c] * kj[c]; dp += doi[c] * vj[c]; }
                const double p = exp(scale * s - lse[i]);
                const double ds = p * (dp - D[i]);
                for (int c = 0; c < d; ++c) dqi[c] += scale * ds * kj[c];
            }
        }
    }
}

/* dK, dV for the key rows in `cols` (NULL: 0..n_cols-1) against query rows 0..n_q-1.
 * Output r belongs to cols[r].  Rows with lse = -inf contribute nothing. */
void orc_attn_bwd_dkdv(const double* q, long ldq, const double* k, long ldk, const double* v, long ldv,
                       const double* dO, long lddo, const double* lse, const double* D,
                       long n_q, int d, double scale, const long* cols, long n_cols,
                       double* dK, long lddk, double* dV, long lddv) {
#pragma omp parallel for schedule(dynamic, 4)
    for (long r = 0; r < n_cols; ++r) {
        const long j = cols ? cols[r] : r;
        const double* kj = k + j * ldk;
        const double* vj = v + j * ldv;
        double* dkj = dK + r * lddk;
        double* dvj = dV + r * lddv;
        for (int c = 0; c < d; ++c) { dkj[c] = 0.0; dvj[c] = 0.0; }
        for (long i = 0; i < n_q; ++i) {
            const double* qi = q + i * ldq;
            const double* doi = dO + i * lddo;
            double s = 0.0, dp = 0.0;
            for (int c = 0; c < d; ++c) { s += qi[c] * kj[c]; dp += doi[c] * vj[c]; }
            const double p = exp(scale * s - lse[i]);
            const double ds = p * (dp - D[i]);
            for (int c = 0; c < d; ++c) { dvj[c] += p * doi[c]; dkj[c] += scale * ds * qi[c]; }
        }
    }
}
