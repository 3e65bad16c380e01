/*
 * Plain fp64 CPU oracle for exact K-means Lloyd iterations on bf16 inputs.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
 * hot path computes.  It shares no code with the CUDA library and is never on the product path:
 * only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may call it.
 *
 * What it follows: the paper's Section 5, paragraph "Flash-KMeans clean-start workload":
 *   - `assign` computes the squared Euclidean distance from each point to all K centroids and
 *     returns the arg-min;
 *   - `centroid_update` reduces the points of each cluster into per-cluster sums and counts;
 *   - the workload is *exact* K-means, so the textbook definition is the reference result.
 * The paper stops at sums and counts; the division into means and the empty-cluster rule (an
 * empty cluster keeps its previous centroid) are this build's stated reading.
 *
 * Arithmetic: every bf16 input is widened exactly to double.  Distances use direct differences
 * sum_d (x_d - c_d)^2, accumulated left to right in d, so nothing here resembles the
 * ||x||^2 - 2 x.c + ||c||^2 expansion the GPU path uses.  Ties go to the lowest centroid index.
 * There is no blocking, no reordering and no vectorisation pragma; OpenMP only spreads the
 * independent points (assign) or the independent clusters' columns (update) over cores, which
 * does not change any sum's order.
 *
 * Pins (all in tests/test_oracle_pins.py): numpy/scipy brute force on tiny inputs, exact
 * integer-valued cases, K=1 / C=X / 1-D midpoint special cases, permutation and translation
 * invariances, mean / mass-conservation / Huygens identities for update, monotone inertia and
 * fixed point for Lloyd, a hand-worked 2-D example in exact rationals, and a scikit-learn
 * cross-check; oracle_knn: numpy lexsort brute force, exact integer ties, k = 1 against
 * oracle_assign, k >= M.  No function here is "parity unpinned" against the mathematics; the paper
 * itself prints no numeric K-means or KNN result to pin against.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef long long i64;

static inline double bf16_bits_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* fp64 -> fp32 (round to nearest even, the C conversion) -> bf16 (round to nearest even). */
static inline uint16_t f64_to_bf16_bits(double v) {
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* quiet NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

void oracle_bf16_to_f64(const uint16_t* in, i64 n, double* out) {
    for (i64 i = 0; i < n; ++i) out[i] = bf16_bits_to_f64(in[i]);
}

void oracle_f64_to_bf16(const double* in, i64 n, uint16_t* out) {
    for (i64 i = 0; i < n; ++i) out[i] = f64_to_bf16_bits(in[i]);
}

/*
 * Assignment against fp64 centroids.
 *   X      [N,D] bf16 bits, row major
 *   C      [K,D] double, row major
 *   idx    [N]   arg-min_k d(i,k), lowest k on exact ties
 *   dist   [N]   d(i, idx[i])                                   (may be NULL)
 *   second [N]   smallest d(i,k) over k != idx[i]; +inf if K==1 (may be NULL)
 * Returns 0, or -1 on bad arguments.
 */
int oracle_assign_f64c(const uint16_t* X, const double* C, i64 N, int D, int K,
                       int32_t* idx, double* dist, double* second) {
    if (!X || !C || !idx || N < 0 || D < 1 || K < 1) return -1;
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(static)
        for (i64 i = 0; i < N; ++i) {
            for (int d = 0; d < D; ++d) x[d] = bf16_bits_to_f64(X[i * D + d]);
            double best = INFINITY, sec = INFINITY;
            int32_t arg = 0;
            for (int k = 0; k < K; ++k) {
                const double* c = C + (i64)k * D;
                double acc = 0.0;
                for (int d = 0; d < D; ++d) {
                    double t = x[d] - c[d];
                    acc += t * t;
                }
                if (acc < best) {           /* strict: an equal later k never replaces */
                    sec = best;
                    best = acc;
                    arg = k;
                } else if (acc < sec) {
                    sec = acc;
                }
            }
            idx[i] = arg;
            if (dist) dist[i] = best;
            if (second) second[i] = sec;
        }
        free(x);
    }
    return 0;
}

/* Same with bf16 centroids (widened exactly). */
int oracle_assign(const uint16_t* X, const uint16_t* C, i64 N, int D, int K,
                  int32_t* idx, double* dist, double* second) {
    if (!C || D < 1 || K < 1) return -1;
    double* Cd = (double*)malloc(sizeof(double) * (size_t)K * (size_t)D);
    if (!Cd) return -2;
    oracle_bf16_to_f64(C, (i64)K * D, Cd);
    int rc = oracle_assign_f64c(X, Cd, N, D, K, idx, dist, second);
    free(Cd);
    return rc;
}

/* d(i) = sum_d (X[i,d] - C[g[i],d])^2 for a given pairing g; used to grade near-ties. */
int oracle_pair_sqdist(const uint16_t* X, const double* C, i64 N, int D, int K,
                       const int32_t* g, double* out) {
    if (!X || !C || !g || !out) return -1;
    for (i64 i = 0; i < N; ++i) {
        if (g[i] < 0 || g[i] >= K) return -3;
        const double* c = C + (i64)g[i] * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) {
            double t = bf16_bits_to_f64(X[i * D + d]) - c[d];
            acc += t * t;
        }
        out[i] = acc;
    }
    return 0;
}

/*
 * Centroid update.
 *   counts[k] = #{i : idx[i]==k}
 *   sums[k,:] = sum of those rows, added in increasing i
 *   C_new[k,:] = sums[k,:] / counts[k], or C_prev[k,:] when the cluster is empty
 *                (zeros when C_prev is NULL)
 *   sums may be NULL.
 * Returns 0, -1 on bad arguments, -3 if some idx is outside [0,K).
 */
int oracle_update(const uint16_t* X, const int32_t* idx, i64 N, int D, int K,
                  const double* C_prev, double* C_new, i64* counts, double* sums_out) {
    if (!X || !idx || !C_new || !counts || N < 0 || D < 1 || K < 1) return -1;
    double* sums = sums_out ? sums_out : (double*)malloc(sizeof(double) * (size_t)K * (size_t)D);
    if (!sums) return -2;
    memset(sums, 0, sizeof(double) * (size_t)K * (size_t)D);
    memset(counts, 0, sizeof(i64) * (size_t)K);
    int bad = 0;
    for (i64 i = 0; i < N; ++i) {
        if (idx[i] < 0 || idx[i] >= K) { bad = 1; break; }
        counts[idx[i]] += 1;
    }
    if (bad) { if (!sums_out) free(sums); return -3; }
    /* each thread owns a band of columns; every column's sum runs over i in increasing order */
#pragma omp parallel
    {
        int nt = 1, me = 0;
#ifdef _OPENMP
        nt = omp_get_num_threads();
        me = omp_get_thread_num();
#endif
        int d0 = (int)(((i64)D * me) / nt), d1 = (int)(((i64)D * (me + 1)) / nt);
        for (i64 i = 0; i < N; ++i)
            for (int d = d0; d < d1; ++d)
                sums[(i64)idx[i] * D + d] += bf16_bits_to_f64(X[i * D + d]);
    }
    for (int k = 0; k < K; ++k)
        for (int d = 0; d < D; ++d) {
            i64 o = (i64)k * D + d;
            if (counts[k] > 0) C_new[o] = sums[o] / (double)counts[k];
            else C_new[o] = C_prev ? C_prev[o] : 0.0;
        }
    if (!sums_out) free(sums);
    return 0;
}

/*
 * Lloyd iterations: for t in [0,iters): assign against C_t, inertia[t] = sum_i dist_t[i],
 * then update -> C_{t+1}.
 *   round_centroids != 0: C_{t+1} is rounded fp64 -> fp32 -> bf16 before the next assign
 *   (the two kernels exchange bf16 centroids); C_out holds the *unrounded* means of the
 *   last update and C_out_bits their bf16 rounding.
 *   round_centroids == 0: pure fp64 Lloyd (C_out_bits still filled, for convenience).
 * idx/dist/second are those of the LAST assign (against C_{iters-1}); counts of the last update.
 */
int oracle_lloyd(const uint16_t* X, const uint16_t* C0, i64 N, int D, int K, int iters,
                 int round_centroids, double* C_out, uint16_t* C_out_bits, int32_t* idx,
                 double* dist, double* second, i64* counts, double* inertia) {
    if (!X || !C0 || !C_out || !idx || !counts || iters < 0) return -1;
    size_t kd = (size_t)K * (size_t)D;
    double* Ct = (double*)malloc(sizeof(double) * kd);
    double* dloc = dist ? dist : (double*)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1));
    if (!Ct || !dloc) return -2;
    oracle_bf16_to_f64(C0, (i64)kd, Ct);
    memcpy(C_out, Ct, sizeof(double) * kd);
    int rc = 0;
    for (int t = 0; t < iters && rc == 0; ++t) {
        rc = oracle_assign_f64c(X, Ct, N, D, K, idx, dloc, second);
        if (rc) break;
        if (inertia) {
            double s = 0.0;
            for (i64 i = 0; i < N; ++i) s += dloc[i];
            inertia[t] = s;
        }
        rc = oracle_update(X, idx, N, D, K, Ct, C_out, counts, NULL);
        if (rc) break;
        if (round_centroids) {
            for (size_t j = 0; j < kd; ++j) Ct[j] = bf16_bits_to_f64(f64_to_bf16_bits(C_out[j]));
        } else {
            memcpy(Ct, C_out, sizeof(double) * kd);
        }
    }
    if (C_out_bits) oracle_f64_to_bf16(C_out, (i64)kd, C_out_bits);
    free(Ct);
    if (!dist) free(dloc);
    return rc;
}

/*
 * Exact k-nearest-neighbour search (the paper's Section 6 names a "KNN search" family with recall 1.0,
 * i.e. the exact result; the distance is the squared Euclidean one of the K-means workload).
 *   Q    [N,D] bf16 bits: queries          X [M,D] bf16 bits: database rows
 *   idx  [N,k] the k database rows nearest to each query, ascending by (distance, row number):
 *              among equal distances the lower row number comes first
 *   dist [N,k] their squared distances (direct differences, fp64)
 * When M < k the tail of each row is idx = -1, dist = +inf.
 * Plain statement: every distance is computed, and a row enters the sorted list of the k best only if
 * its distance is strictly smaller than the current k-th best (rows come in ascending order, so an equal
 * later row never displaces an earlier one) and is placed behind every entry that is not larger.
 */
int oracle_knn(const uint16_t* Q, const uint16_t* X, i64 N, i64 M, int D, int k, int32_t* idx, double* dist) {
    if (!Q || !X || !idx || !dist || N < 0 || M < 0 || D < 1 || k < 1) return -1;
#pragma omp parallel
    {
        double* q = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(static)
        for (i64 i = 0; i < N; ++i) {
            for (int d = 0; d < D; ++d) q[d] = bf16_bits_to_f64(Q[i * D + d]);
            int32_t* bi = idx + i * k;
            double* bd = dist + i * k;
            int cnt = 0;
            for (int s = 0; s < k; ++s) { bi[s] = -1; bd[s] = INFINITY; }
            for (i64 j = 0; j < M; ++j) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) {
                    double t = q[d] - bf16_bits_to_f64(X[j * D + d]);
                    acc += t * t;
                }
                if (cnt == k && !(acc < bd[k - 1])) continue;
                int pos = cnt < k ? cnt : k - 1;          /* slot that opens up (the last one is dropped when full) */
                while (pos > 0 && bd[pos - 1] > acc) {    /* entries strictly larger move down one place */
                    bd[pos] = bd[pos - 1];
                    bi[pos] = bi[pos - 1];
                    --pos;
                }
                bd[pos] = acc;
                bi[pos] = (int32_t)j;
                if (cnt < k) ++cnt;
            }
        }
        free(q);
    }
    return 0;
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
