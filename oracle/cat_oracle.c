/*
 * CAT oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, obviously-correct CPU statement of Cluster-based Affine
 * Transformation (CAT): K-Means fitting over the low-bit (LQ) output rows,
 * the closed-form per-cluster affine parameters (gamma, beta), and CAT
 * inference (nearest centroid + per-cluster affine correction).
 *
 * Everything is written from the paper:
 *   - Section 3.1 (cluster means, variance, covariance; Eq. "gamma-beta";
 *     the alpha-blended correction),
 *   - Algorithm 1 "CAT Fitting"  (empty cluster => gamma=1, beta=0; variance
 *     floor 1e-8; gamma = Mean[(Q-muQ)(F-muF)] / max(Var(Q),1e-8);
 *     beta = muF - gamma*muQ),
 *   - Algorithm 2 "CAT Inferencing" (affine_corrected = q*gamma + beta;
 *     blended = q + alpha*(affine_corrected - q)),
 *   - Section 4 Setup ("We use K-Means as the clustering algorithm").
 *
 * Inputs and stored results are fp32; every sum, distance, mean and division
 * is carried in fp64.  No blocking, no algebraic rearrangement: distances are
 * the direct form sum_j (y_j - c_j)^2, moments are the two-pass centred
 * definitions.  Row sums run in ascending row order so results do not depend
 * on the thread count (threads split rows for assignment, columns for sums).
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code with the CUDA library.
 *
 * Readings where the paper is silent (each is also exercised by a test):
 *   init = first K rows; exactly `iters` assign+update rounds; squared
 *   Euclidean distance; ties go to the lowest cluster index; a cluster that
 *   loses all rows keeps its centroid; a final assignment against the final
 *   centroids feeds gamma/beta; population (1/n) variance and covariance.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Squared Euclidean distance in fp64, direct form. */
static double sqdist(const float *y, const float *c, int32_t D)
{
    double s = 0.0;
    for (int32_t j = 0; j < D; ++j) {
        double d = (double)y[j] - (double)c[j];
        s += d * d;
    }
    return s;
}

/*
 * Nearest-centroid assignment (the "predict" of the cluster model, Alg. 2
 * step 2).  Scans k ascending and replaces only on strict '<', so the lowest
 * index wins a tie.  best/second (may be NULL) receive the smallest and the
 * second-smallest squared distance; second = +inf when K == 1.
 */
void oracle_assign(const float *Yq, int64_t N, int32_t D, int32_t K,
                   const float *C, int32_t *labels, double *best, double *second)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        const float *y = Yq + i * (int64_t)D;
        double b = INFINITY, s = INFINITY;
        int32_t bk = 0;
        for (int32_t k = 0; k < K; ++k) {
            double d = sqdist(y, C + (int64_t)k * D, D);
            if (d < b) { s = b; b = d; bk = k; }
            else if (d < s) { s = d; }
        }
        labels[i] = bk;
        if (best) best[i] = b;
        if (second) second[i] = s;
    }
}

/*
 * Per-cluster column sums of M (N x D) in fp64, rows added in ascending
 * order.  sums is K x D, counts is K.
 */
static void cluster_sums(const float *M, const int32_t *labels, int64_t N, int32_t D,
                         int32_t K, double *sums, int64_t *counts)
{
    memset(sums, 0, sizeof(double) * (size_t)K * (size_t)D);
    memset(counts, 0, sizeof(int64_t) * (size_t)K);
    for (int64_t i = 0; i < N; ++i) counts[labels[i]]++;
#pragma omp parallel
    {
        int nt = 1, t = 0;
#ifdef _OPENMP
        nt = omp_get_num_threads();
        t = omp_get_thread_num();
#endif
        int32_t j0 = (int32_t)(((int64_t)D * t) / nt);
        int32_t j1 = (int32_t)(((int64_t)D * (t + 1)) / nt);
        for (int64_t i = 0; i < N; ++i) {
            const float *m = M + i * (int64_t)D;
            double *s = sums + (int64_t)labels[i] * D;
            for (int32_t j = j0; j < j1; ++j) s[j] += (double)m[j];
        }
    }
}

/*
 * Centroid update of one Lloyd round: c_k <- mean of the rows labelled k,
 * rounded to fp32; a cluster with no rows keeps its centroid.
 * counts (K, may be NULL) receives the cluster sizes.
 */
void oracle_update_centroids(const float *Yq, const int32_t *labels, int64_t N, int32_t D,
                             int32_t K, float *C, int64_t *counts_out)
{
    double *sums = (double *)malloc(sizeof(double) * (size_t)K * (size_t)D);
    int64_t *counts = (int64_t *)malloc(sizeof(int64_t) * (size_t)K);
    cluster_sums(Yq, labels, N, D, K, sums, counts);
    for (int32_t k = 0; k < K; ++k) {
        if (counts[k] == 0) continue;
        for (int32_t j = 0; j < D; ++j)
            C[(int64_t)k * D + j] = (float)(sums[(int64_t)k * D + j] / (double)counts[k]);
    }
    if (counts_out) memcpy(counts_out, counts, sizeof(int64_t) * (size_t)K);
    free(sums);
    free(counts);
}

/*
 * Closed-form affine parameters for given labels (Section 3.1; Algorithm 1,
 * the loop over cluster ids).  Per cluster k and column j, over the rows of
 * the cluster:
 *   muQ = mean(q), muF = mean(f)
 *   var = mean((q-muQ)^2), floored at 1e-8
 *   cov = mean((q-muQ)(f-muF))
 *   gamma = cov/var, beta = muF - gamma*muQ
 * Empty cluster: gamma = 1, beta = 0.
 */
void oracle_solve_gamma_beta(const float *Yq, const float *Yfp, const int32_t *labels,
                             int64_t N, int32_t D, int32_t K, float *gamma, float *beta)
{
    size_t KD = (size_t)K * (size_t)D;
    double *sq = (double *)malloc(sizeof(double) * KD);
    double *sf = (double *)malloc(sizeof(double) * KD);
    double *var = (double *)calloc(KD, sizeof(double));
    double *cov = (double *)calloc(KD, sizeof(double));
    int64_t *counts = (int64_t *)malloc(sizeof(int64_t) * (size_t)K);
    int64_t *counts2 = (int64_t *)malloc(sizeof(int64_t) * (size_t)K);
    cluster_sums(Yq, labels, N, D, K, sq, counts);
    cluster_sums(Yfp, labels, N, D, K, sf, counts2);
    /* sq, sf become the means */
    for (int32_t k = 0; k < K; ++k) {
        if (counts[k] == 0) continue;
        for (int32_t j = 0; j < D; ++j) {
            sq[(int64_t)k * D + j] /= (double)counts[k];
            sf[(int64_t)k * D + j] /= (double)counts[k];
        }
    }
    /* second pass: centred second moments, rows in ascending order */
#pragma omp parallel
    {
        int nt = 1, t = 0;
#ifdef _OPENMP
        nt = omp_get_num_threads();
        t = omp_get_thread_num();
#endif
        int32_t j0 = (int32_t)(((int64_t)D * t) / nt);
        int32_t j1 = (int32_t)(((int64_t)D * (t + 1)) / nt);
        for (int64_t i = 0; i < N; ++i) {
            int64_t o = (int64_t)labels[i] * D;
            const float *q = Yq + i * (int64_t)D;
            const float *f = Yfp + i * (int64_t)D;
            for (int32_t j = j0; j < j1; ++j) {
                double dq = (double)q[j] - sq[o + j];
                double df = (double)f[j] - sf[o + j];
                var[o + j] += dq * dq;
                cov[o + j] += dq * df;
            }
        }
    }
    for (int32_t k = 0; k < K; ++k) {
        for (int32_t j = 0; j < D; ++j) {
            int64_t o = (int64_t)k * D + j;
            if (counts[k] == 0) {
                gamma[o] = 1.0f;
                beta[o] = 0.0f;
                continue;
            }
            double v = var[o] / (double)counts[k];
            double c = cov[o] / (double)counts[k];
            if (v < 1e-8) v = 1e-8;
            double g = c / v;
            double b = sf[o] - g * sq[o];
            gamma[o] = (float)g;
            beta[o] = (float)b;
        }
    }
    free(sq); free(sf); free(var); free(cov); free(counts); free(counts2);
}

/*
 * CAT fitting without PCA (Algorithm 1 with the cluster model fitted on the
 * rows themselves).
 *   init      : K x D starting centroids, or NULL for the first K rows of Yq.
 *   C         : K x D out, final centroids.
 *   gamma,beta: K x D out.
 *   labels    : N out, final assignment against the final centroids.
 *   J         : iters+1 out (may be NULL): J[t] = sum_i best_i of round t's
 *               assignment (against the centroids entering round t);
 *               J[iters] belongs to the final assignment.
 *   near      : iters+1 out (may be NULL): rows with second-best <= near_rel*second
 *               in that assignment (near-ties; exact ties included).
 *   counts    : K out (may be NULL): final cluster sizes.
 * Returns 0, or 1 on bad arguments.
 */
int oracle_fit(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K,
               int32_t iters, const float *init, double near_rel,
               float *C, float *gamma, float *beta, int32_t *labels,
               double *J, int64_t *near, int64_t *counts)
{
    if (N < K || K < 1 || D < 1 || iters < 0) return 1;
    memcpy(C, init ? init : Yq, sizeof(float) * (size_t)K * (size_t)D);
    double *best = (double *)malloc(sizeof(double) * (size_t)N);
    double *second = (double *)malloc(sizeof(double) * (size_t)N);
    for (int32_t t = 0; t <= iters; ++t) {
        oracle_assign(Yq, N, D, K, C, labels, best, second);
        double obj = 0.0;
        int64_t nn = 0;
        for (int64_t i = 0; i < N; ++i) {
            obj += best[i];
            if (K > 1 && (second[i] - best[i]) <= near_rel * second[i]) nn++;
        }
        if (J) J[t] = obj;
        if (near) near[t] = nn;
        if (t == iters) break;
        oracle_update_centroids(Yq, labels, N, D, K, C, NULL);
    }
    free(best);
    free(second);
    oracle_solve_gamma_beta(Yq, Yfp, labels, N, D, K, gamma, beta);
    if (counts) {
        memset(counts, 0, sizeof(int64_t) * (size_t)K);
        for (int64_t i = 0; i < N; ++i) counts[labels[i]]++;
    }
    return 0;
}

/*
 * CAT inference (Algorithm 2 without PCA):
 *   l = nearest centroid of row i
 *   affine = q*gamma_l + beta_l            (one rounding to fp32 when alpha==1)
 *   out    = q + alpha*(affine - q)        (Alg. 2 blend; alpha==1 => affine)
 * With alpha == 1 the result is float(gamma*q + beta) evaluated in fp64,
 * i.e. a single rounding of the exact value (the fp64 product of two fp32
 * numbers is exact; the sum is rounded once to fp64, then to fp32).
 */
void oracle_apply(const float *Yq, int64_t N, int32_t D, int32_t K,
                  const float *C, const float *gamma, const float *beta, double alpha,
                  float *out, int32_t *labels, double *best, double *second)
{
    oracle_assign(Yq, N, D, K, C, labels, best, second);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        const float *q = Yq + i * (int64_t)D;
        const float *g = gamma + (int64_t)labels[i] * D;
        const float *b = beta + (int64_t)labels[i] * D;
        float *o = out + i * (int64_t)D;
        for (int32_t j = 0; j < D; ++j) {
            double a = (double)q[j] * (double)g[j] + (double)b[j];
            if (alpha == 1.0) o[j] = (float)a;
            else o[j] = (float)((double)q[j] + alpha * (a - (double)q[j]));
        }
    }
}

/* Affine correction for given labels (no assignment). */
void oracle_affine_with_labels(const float *Yq, const int32_t *labels, int64_t N, int32_t D,
                               const float *gamma, const float *beta, double alpha, float *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        const float *q = Yq + i * (int64_t)D;
        const float *g = gamma + (int64_t)labels[i] * D;
        const float *b = beta + (int64_t)labels[i] * D;
        float *o = out + i * (int64_t)D;
        for (int32_t j = 0; j < D; ++j) {
            double a = (double)q[j] * (double)g[j] + (double)b[j];
            if (alpha == 1.0) o[j] = (float)a;
            else o[j] = (float)((double)q[j] + alpha * (a - (double)q[j]));
        }
    }
}
