/*
 * cat.h -- C ABI of the B200 (sm_100a) CAT library.
 *
 * CAT (Cluster-based Affine Transformation) corrects the outputs of a low-bit
 * quantised (LQ) model towards those of its full-precision (FP) counterpart:
 * the LQ output rows are clustered with K-Means, each cluster k gets an
 * element-wise affine map (gamma_k, beta_k) fitted in closed form against the
 * FP outputs, and at inference a row is assigned to its nearest centroid and
 * corrected with that cluster's map.
 *
 * Conventions for every entry point unless stated otherwise
 *   - All data pointers are DEVICE pointers owned by the caller; matrices are
 *     fp32, row-major, contiguous (leading dimension D); base addresses must
 *     be 16-byte aligned.  Labels are 0-based int32.
 *   - `workspace` is caller-provided device scratch of at least the size the
 *     matching *_workspace_bytes query returns (256-byte aligned).  The
 *     library allocates and frees nothing.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls only enqueue work: they return after launching, never synchronise,
 *     and are re-entrant for distinct workspaces (the two
 *     process-wide kernel selectors at the end of this header aside).
 *   - Return value: CAT_OK or an error code; on error nothing was enqueued
 *     (argument errors) or outputs are undefined (CAT_ERR_CUDA).  The library
 *     never throws, aborts or traps.
 *   - Inputs must be finite.  Non-finite values give unspecified labels but
 *     never an out-of-range label or an invalid memory access.
 *   - Limits: 1 <= K <= CAT_MAX_K, K <= N < 2^31 (cat_fit and the step-level sums:
 *     N < 2^30), 1 <= D <= CAT_MAX_D.  D % 4 != 0 is supported through scalar loads (slower).
 */
#ifndef CAT_H_
#define CAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int cat_status_t;

enum {
    CAT_OK = 0,
    CAT_ERR_NULL = 1,        /* a required pointer is NULL */
    CAT_ERR_SHAPE = 2,       /* N < K, K < 1, D < 1, iters < 0, alpha outside [0,1] */
    CAT_ERR_ALIGN = 3,       /* a base pointer is not 16-byte aligned */
    CAT_ERR_WORKSPACE = 4,   /* workspace NULL or smaller than the query says */
    CAT_ERR_CUDA = 5,        /* a CUDA runtime call failed: see cat_last_cuda_error() */
    CAT_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait gave up (reported by cat_device_status) */
    CAT_ERR_UNSUPPORTED = 7  /* K > CAT_MAX_K, D > CAT_MAX_D or N >= 2^31 */
};

#define CAT_MAX_K 512
#define CAT_MAX_D 16384

/* Diagnostics of one cat_fit_from call, written to device memory.  The first four words are
 * always filled.  The per-assignment records cost an extra pass over Yq after every assignment
 * (the `iters` assignments of the Lloyd rounds and the final one, Algorithm 1 with K-Means as
 * the cluster model), so a fit that asks for them is slower than one that passes diag = NULL.
 * Assignment t is recorded at index t for t < CAT_DIAG_MAX_ROUNDS - 1; the final assignment is
 * always recorded, at index min(iters, CAT_DIAG_MAX_ROUNDS - 1). */
#define CAT_DIAG_MAX_ROUNDS 64
typedef struct cat_fit_diag {
    int64_t refined_rows_total;   /* rows whose label needed the exact fp64 pass, summed over all assignments */
    int64_t refined_rows_final;   /* same, final assignment only */
    int64_t empty_clusters_final; /* clusters with no rows in the final assignment */
    int64_t device_status;        /* CAT_OK or CAT_ERR_DEVICE_TIMEOUT */
    int64_t assignments_recorded; /* min(iters + 1, CAT_DIAG_MAX_ROUNDS) */
    int64_t undecided_rows[CAT_DIAG_MAX_ROUNDS]; /* rows the fast scores could not decide (sent to the exact pass) */
    int64_t near_tie_rows[CAT_DIAG_MAX_ROUNDS];  /* rows whose two nearest centroids are within 1e-6 relative of each
                                                    other in squared distance (fp64 direct form) */
    double objective[CAT_DIAG_MAX_ROUNDS];       /* sum_i ||Yq_i - c_label(i)||^2 against the centroids the assignment
                                                    used, fp64; the order of the additions is not fixed, so the last
                                                    bits vary from run to run */
} cat_fit_diag_t;

/* ---- the two calls of the hot path ------------------------------------ */

/*
 * CAT fitting (Algorithm 1 "CAT Fitting" with the cluster model fitted on the
 * rows themselves; Section 3.1 for the closed form; Section 4 Setup: K-Means).
 *
 *   1. centroids <- init_centroids, or the first K rows of Yq when NULL
 *   2. `iters` Lloyd rounds: label_i = argmin_k ||Yq_i - c_k||^2 (lowest k on
 *      ties); c_k <- mean of its rows (a cluster with no rows keeps c_k)
 *   3. final assignment against the final centroids -> labels_out
 *   4. per cluster k and column j over the rows of the cluster:
 *        muQ, muF = means of Yq, Yfp;  var = mean (q-muQ)^2;  cov = mean (q-muQ)(f-muF)
 *        gamma = cov / max(var, 1e-8);  beta = muF - gamma*muQ
 *      empty cluster: gamma = 1, beta = 0.
 *
 * Yq, Yfp       [N, D] in.   centroids_out, gamma_out, beta_out  [K, D] out.
 * labels_out    [N] out, may be NULL.
 * init_centroids [K, D] in, may be NULL; must not alias centroids_out.
 * diag          device pointer to one cat_fit_diag_t, may be NULL.
 * Labels are decided in fp64 whenever the fast scores cannot separate the two
 * nearest centroids; sums and moments are accumulated in fp64.  In the Lloyd
 * rounds the per-cluster sums are carried from round to round and updated with
 * the rows whose label changed (the same sums up to fp64 rounding).
 * The workspace holds, besides tables of a few N and K*D words, an fp16 copy
 * of Yq (N*D*2 bytes) that the tensor-core assignment reads in every round.
 */
size_t cat_fit_workspace_bytes(int64_t N, int32_t D, int32_t K);

cat_status_t cat_fit(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K,
                     int32_t iters, float *centroids_out, float *gamma_out, float *beta_out,
                     int32_t *labels_out, void *workspace, size_t workspace_bytes, void *stream);

cat_status_t cat_fit_from(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K,
                          int32_t iters, const float *init_centroids,
                          float *centroids_out, float *gamma_out, float *beta_out,
                          int32_t *labels_out, cat_fit_diag_t *diag,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * CAT inference (Algorithm 2 "CAT Inferencing" without PCA, alpha = 1):
 *   label_i = argmin_k ||Yq_i - c_k||^2 ;  Y_out_i = gamma_label * Yq_i + beta_label
 * evaluated as one fused multiply-add per element (a single rounding).
 *
 * Yq [N, D] in; centroids, gamma, beta [K, D] in; Y_out [N, D] out (must not
 * overlap Yq); labels_out [N] out, may be NULL.  N >= 1 (N < K is allowed).
 */
size_t cat_apply_workspace_bytes(int64_t N, int32_t D, int32_t K);

cat_status_t cat_apply(const float *Yq, int64_t N, int32_t D, int32_t K,
                       const float *centroids, const float *gamma, const float *beta,
                       float *Y_out, int32_t *labels_out,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * The alpha-blended correction of Section 3.1 / Algorithm 2:
 *   Y_out_i = Yq_i + alpha * ((gamma_l * Yq_i + beta_l) - Yq_i),  0 <= alpha <= 1.
 * Evaluated as fma(1 + alpha*(gamma-1), y, alpha*beta) with the two
 * coefficients formed in fp64 per element.  alpha = 1 is exactly cat_apply.
 */
cat_status_t cat_apply_blend(const float *Yq, int64_t N, int32_t D, int32_t K,
                             const float *centroids, const float *gamma, const float *beta,
                             float alpha, float *Y_out, int32_t *labels_out,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * cat_apply with a bf16 result: Y_out_bf16 [N, D] receives bf16(gamma_l * Yq_i + beta_l), the fp32
 * fused multiply-add of cat_apply rounded to nearest even (Algorithm 2 with alpha = 1; Section 3.1
 * notes that the correction suits low-precision deployment, without fixing a format).  The labels
 * are exact as in cat_apply.  Halves the bytes written.  For shapes the 64-row-tile kernel takes
 * (K >= the tensor-core threshold, K <= 256, D >= 128, D % 8 == 0, N > 64) assignment and correction
 * are fused; other shapes run the assignment, then one pass that reads the rows again.
 * Workspace: cat_apply_workspace_bytes(N, D, K).
 */
cat_status_t cat_apply_bf16(const float *Yq, int64_t N, int32_t D, int32_t K,
                            const float *centroids, const float *gamma, const float *beta,
                            void *Y_out_bf16, int32_t *labels_out,
                            void *workspace, size_t workspace_bytes, void *stream);

/* ---- step-level entry points (the same kernels cat_fit chains; used for
 *      row-sharded multi-GPU fitting and for step-wise checks) ------------ */

/* Nearest-centroid labels only (the cluster model's "predict", Alg. 2 step 2).
 * Workspace: cat_apply_workspace_bytes(N, D, K). */
cat_status_t cat_assign(const float *Yq, int64_t N, int32_t D, int32_t K,
                        const float *centroids, int32_t *labels_out,
                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * cat_assign that also hands out what its fast pass saw, so that the label decision can be
 * audited from outside (Alg. 2 step 2; the decision rule is the library's own: a row's label is
 * taken from fast scores t_k = ||c_k||^2 - 2 y.c_k when the two smallest are more than 2e apart,
 * e being a bound on the error of a fast score, and from fp64 direct-form distances otherwise).
 * Every array of `scores` has N entries and may be NULL:
 *   best, second  the two smallest fast scores of the row.  On the tensor-core path a score
 *                 carries the index of its centroid in the low 8 bits of its fp32 pattern.
 *   bound         e for this row: |fast score - exact score| <= e for every centroid (the
 *                 tensor-core bound includes the index packing).
 *   label         the centroid of `best`, i.e. the label before the exact pass.
 * labels_out receives the final labels as cat_assign gives them.
 * flags: CAT_ASSIGN_FP16_OPERANDS runs the tensor-core contraction on an fp16 copy of the rows
 * (per-row power-of-two scale) and of the centroids, as cat_fit does for its Lloyd rounds; it
 * needs D % 8 == 0 and K <= 256 (CAT_ERR_UNSUPPORTED otherwise) and a workspace of
 * cat_fit_workspace_bytes(N, D, K); the centroids must not exceed the largest magnitude of Yq.
 * Without flags the workspace is cat_apply_workspace_bytes(N, D, K).
 */
typedef struct cat_fast_scores {
    float *best;
    float *second;
    float *bound;
    int32_t *label;
} cat_fast_scores_t;
#define CAT_ASSIGN_FP16_OPERANDS 1

cat_status_t cat_assign_scores(const float *Yq, int64_t N, int32_t D, int32_t K,
                               const float *centroids, int32_t *labels_out,
                               const cat_fast_scores_t *scores, int32_t flags,
                               void *workspace, size_t workspace_bytes, void *stream);

/*
 * cat_assign without any workspace: the same labels as cat_assign, for callers that
 * cannot allocate device memory.  (The paper has no counterpart: this is a packaging
 * variant of the assignment step, not a step of the method.)
 *
 * Who needs it: code that runs where a device allocation is impossible or unwelcome --
 * a serving loop that must never hit the allocator (cudaMalloc may synchronise the whole
 * device), a plug-in that only ever receives its input and output buffers from a host
 * framework that owns all device memory, or a process whose memory budget was fixed at
 * start-up.  Such callers cannot provide the scratch cat_assign asks for, so this entry
 * point keeps its own: a fixed array inside the library image, about 1 MiB per GPU that
 * loads the library, held until the process exits.
 *
 *   - Limits: N <= CAT_NOALLOC_MAX_ROWS, K <= CAT_MAX_K, D <= CAT_MAX_D; anything larger
 *     returns CAT_ERR_UNSUPPORTED ("size beyond the supported limits") and enqueues nothing.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current); make that first call outside any
 *     stream capture.  Later calls only launch kernels on `stream`.
 *   - All calls on one device share the one array.  Calls that may overlap on the GPU
 *     (different streams without ordering between them, or different host threads) race on
 *     it and give wrong labels; order them on one stream or with events.  The array keeps
 *     the previous call's contents; the call itself clears what has to start at zero.
 */
#define CAT_NOALLOC_MAX_ROWS 262144
cat_status_t cat_assign_noalloc(const float *Yq, int64_t N, int32_t D, int32_t K,
                                const float *centroids, int32_t *labels_out, void *stream);

/*
 * Row-sharded fitting (one shard of the rows per GPU).  K-Means (Section 4 Setup; Algorithm 1, the
 * cluster model's fit) needs the rows only through per-cluster sums, so a Lloyd round splits into a
 * local half -- assign this shard's rows, form what the round changed in the per-cluster sums -- and
 * an update every rank repeats on the all-reduced changes.  The local half runs the same kernels as
 * cat_fit (fp16 copy of the shard, exact pass for undecided rows, sums over the rows whose label
 * changed), and the library issues no collective: the caller all-reduces between the calls.
 *
 *   cat_fit_shard_begin   once per fit: fp16 copy and norms of this shard's rows in the workspace;
 *                         amax_out (device, 1 float) = largest magnitude of the shard.  The caller
 *                         takes the maximum over all shards.
 *   cat_fit_shard_round   round = 0, 1, 2, ... in order, on the same workspace: labels of the shard
 *                         against `centroids`; delta_sums [K, D] double and delta_counts [K] int64
 *                         receive, per cluster, (rows that entered) - (rows that left) since the
 *                         previous round of this workspace (round 0: every row enters).  amax
 *                         (device, 1 float) is the maximum over all shards from cat_fit_shard_begin.
 *                         labels_out [N] may be NULL.  The caller sums the deltas over all shards.
 *   cat_fit_shard_update  sums += delta_sums, counts += delta_counts, c_k = sums_k / counts_k where
 *                         counts_k > 0 (a cluster with no rows keeps c_k); sums_inout / counts_inout
 *                         are the caller's running totals, zero before round 0.
 *
 * With one shard the three calls reproduce cat_fit's Lloyd rounds bit for bit.  A further round call
 * with the final centroids gives the final labels; the closed form then follows from
 * cat_cluster_sums, cat_centred_moments and cat_solve_gamma_beta on all-reduced sums.
 * Workspace: cat_fit_workspace_bytes(N, D, K) of the shard; N >= 1 (a shard may hold fewer than K rows).
 */
cat_status_t cat_fit_shard_begin(const float *Yq, int64_t N, int32_t D, int32_t K, float *amax_out,
                                 void *workspace, size_t workspace_bytes, void *stream);
cat_status_t cat_fit_shard_round(const float *Yq, int64_t N, int32_t D, int32_t K, int32_t round,
                                 const float *centroids, const float *amax, double *delta_sums,
                                 int64_t *delta_counts, int32_t *labels_out,
                                 void *workspace, size_t workspace_bytes, void *stream);
cat_status_t cat_fit_shard_update(const double *delta_sums, const int64_t *delta_counts, int32_t D,
                                  int32_t K, double *sums_inout, int64_t *counts_inout,
                                  float *centroids_inout, void *stream);

/* Per-cluster column sums of Y (fp64) and cluster sizes for given labels (the sums behind the
 * cluster means of the K-Means update, Section 4 Setup, and behind mu_LQ,k / mu_FP,k of Section 3.1):
 * sums_out [K, D] double, counts_out [K] int64.  Labels must lie in [0, K).
 * Rows are added in a fixed order: results are reproducible run to run.
 * Workspace: cat_fit_workspace_bytes(N, D, K). */
cat_status_t cat_cluster_sums(const float *Y, const int32_t *labels, int64_t N, int32_t D,
                              int32_t K, double *sums_out, int64_t *counts_out,
                              void *workspace, size_t workspace_bytes, void *stream);

/* The centroid update of a K-Means round (Section 4 Setup: K-Means is the cluster model):
 * c_k <- float(sums_k / counts_k) where counts_k > 0, else unchanged. */
cat_status_t cat_centroids_from_sums(const double *sums, const int64_t *counts, int32_t D,
                                     int32_t K, float *centroids_inout, void *stream);

/* Centred second moments for given labels and cluster means (fp64), the numerators of
 * sigma^2_LQ,k and cov_LQ,FP,k of Section 3.1 (Algorithm 1, the Var and Mean of its loop body):
 *   var_out[k,j] = sum_{i in k} (q_ij - meanQ[k,j])^2
 *   cov_out[k,j] = sum_{i in k} (q_ij - meanQ[k,j]) (f_ij - meanF[k,j])
 * (sums, not yet divided by the cluster size).  Workspace as for cat_fit. */
cat_status_t cat_centred_moments(const float *Yq, const float *Yfp, const int32_t *labels,
                                 int64_t N, int32_t D, int32_t K,
                                 const double *meanQ, const double *meanF,
                                 double *var_out, double *cov_out,
                                 void *workspace, size_t workspace_bytes, void *stream);

/* gamma/beta from cluster sums and centred moment sums (Algorithm 1 steps
 * after the means): n = counts[k]; n == 0 -> (1, 0); else
 * gamma = (cov/n) / max(var/n, 1e-8), beta = sumF/n - gamma*sumQ/n. */
cat_status_t cat_solve_gamma_beta(const double *sumQ, const double *sumF,
                                  const double *var_sum, const double *cov_sum,
                                  const int64_t *counts, int32_t D, int32_t K,
                                  float *gamma_out, float *beta_out, void *stream);

/* ---- PCA front-end ------------------------------------------------------ */

/*
 * Section 3.1 clusters the LQ outputs after reducing them with PCA ("PCA is only used to obtain
 * clusters": gamma and beta stay in the original D-dimensional space).  Algorithm 1 step 1 fits
 * the projection on the LQ outputs of the fit set, Algorithm 2 step 1 applies it at inference.
 *
 * cat_pca_fit: column means of Yq [N, D] -> mean_out [D]; covariance of the centred rows in fp64
 * (1 / (N - 1)); its eigen-decomposition by one-sided Jacobi rotations in fp64 on the device; the p
 * directions of largest variance -> components_out [p, D] (rows, unit length, decreasing variance;
 * the sign of a row is fixed so that its entry of largest magnitude is positive); their variances
 * -> eigenvalues_out [p] double, may be NULL.  Deterministic.  N >= 2, 1 <= p <= D,
 * D <= CAT_PCA_MAX_D, p <= CAT_PCA_MAX_P.  Directions whose variances coincide are determined
 * only up to a rotation among themselves.
 * cat_pca_project: Z_out [N, p] = (Y - mean) components^T, fp64 accumulation, fp32 result.
 * cat_affine_with_labels: Y_out_i = gamma_l * Yq_i + beta_l for given cluster ids l = labels[i]
 * (Algorithm 2, the loop over the samples with alpha = 1); a label outside [0, K) copies the row.
 */
#define CAT_PCA_MAX_D 4096
#define CAT_PCA_MAX_P 512
size_t cat_pca_workspace_bytes(int64_t N, int32_t D, int32_t p);
cat_status_t cat_pca_fit(const float *Yq, int64_t N, int32_t D, int32_t p, float *mean_out,
                         float *components_out, double *eigenvalues_out,
                         void *workspace, size_t workspace_bytes, void *stream);
cat_status_t cat_pca_project(const float *Y, int64_t N, int32_t D, int32_t p, const float *mean,
                             const float *components, float *Z_out, void *stream);
cat_status_t cat_affine_with_labels(const float *Yq, int64_t N, int32_t D, int32_t K,
                                    const int32_t *labels, const float *gamma, const float *beta,
                                    float *Y_out, void *stream);

/*
 * Algorithm 1 as printed: PCA on Yq, K-Means on the reduced rows (first K reduced rows as the
 * start, `iters` Lloyd rounds, a final assignment), then per cluster the closed-form gamma / beta
 * from the original Yq, Yfp.  centroids_out is [K, p]; gamma_out, beta_out are [K, D].
 * Algorithm 2 as printed (alpha = 1): project, nearest centroid in the reduced space, affine
 * correction in the original space.
 */
size_t cat_fit_pca_workspace_bytes(int64_t N, int32_t D, int32_t K, int32_t p);
cat_status_t cat_fit_pca(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K,
                         int32_t iters, int32_t p, float *mean_out, float *components_out,
                         float *centroids_out, float *gamma_out, float *beta_out, int32_t *labels_out,
                         void *workspace, size_t workspace_bytes, void *stream);
size_t cat_apply_pca_workspace_bytes(int64_t N, int32_t D, int32_t K, int32_t p);
cat_status_t cat_apply_pca(const float *Yq, int64_t N, int32_t D, int32_t K, int32_t p,
                           const float *mean, const float *components, const float *centroids,
                           const float *gamma, const float *beta, float *Y_out, int32_t *labels_out,
                           void *workspace, size_t workspace_bytes, void *stream);

/* ---- host-buffer entry points (end-to-end use) ------------------------- */

/*
 * cat_apply with HOST inputs and outputs.  Yq_host / Y_out_host [N, D] and
 * labels_out_host [N] (may be NULL) are host pointers, ideally page-locked so
 * that copies overlap compute; centroids/gamma/beta [K, D] are host pointers
 * too.  Rows are streamed through device staging buffers carved from
 * `workspace` (device memory, size from cat_apply_host_workspace_bytes) in
 * chunks, overlapping H2D copy, the fused kernel and D2H copy.  The call
 * BLOCKS until all results are on the host.
 */
size_t cat_apply_host_workspace_bytes(int64_t N, int32_t D, int32_t K);

cat_status_t cat_apply_host(const float *Yq_host, int64_t N, int32_t D, int32_t K,
                            const float *centroids_host, const float *gamma_host,
                            const float *beta_host, float *Y_out_host, int32_t *labels_out_host,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * cat_fit with HOST inputs and outputs: copies Yq/Yfp to device buffers carved
 * from `workspace` (size from cat_fit_host_workspace_bytes), runs cat_fit and
 * copies centroids, gamma, beta and (if not NULL) labels back.  BLOCKS until
 * done.
 */
size_t cat_fit_host_workspace_bytes(int64_t N, int32_t D, int32_t K);

cat_status_t cat_fit_host(const float *Yq_host, const float *Yfp_host, int64_t N, int32_t D,
                          int32_t K, int32_t iters, float *centroids_out_host,
                          float *gamma_out_host, float *beta_out_host, int32_t *labels_out_host,
                          void *workspace, size_t workspace_bytes, void *stream);

/* ---- misc --------------------------------------------------------------- */

/* Reads back counters kept in a workspace by the calls that used it last: waits for
 * `stream`, then copies to the HOST pointers (each may be NULL) the number of rows
 * whose label needed the exact fp64 pass in the latest assignment, the running
 * total since the last cat_fit started on that workspace, and the device status
 * word (CAT_OK or CAT_ERR_DEVICE_TIMEOUT). */
cat_status_t cat_workspace_report(const void *workspace, void *stream, int64_t *refined_last_host,
                                  int64_t *refined_total_host, int32_t *device_status_host);

/* Self-test of the failure path of the device-side waits.  The tensor-core kernels wait on
 * barriers with a time limit; a wait that runs out records CAT_ERR_DEVICE_TIMEOUT in the
 * workspace's control block and the kernel returns instead of hanging.  This call enqueues one
 * warp that waits limit_ms (clamped to 1 .. 1000) on a barrier nothing completes; afterwards
 * cat_workspace_report on the same workspace gives device_status = CAT_ERR_DEVICE_TIMEOUT.
 * Any workspace of at least 256 bytes will do; its counters are reset. */
cat_status_t cat_selftest_wait_timeout(void *workspace, size_t workspace_bytes, int32_t limit_ms, void *stream);

/* Kernel selection for the distance contraction.  With K >= min_k (and D % 4 == 0,
 * K <= 256) the scores are formed on the tensor cores (tcgen05, TF32 or fp16 operands, fp32
 * accumulation); below it on the fp32 pipes.  Either way undecided rows are settled in
 * fp64, so the labels are the same.  Default 8: measured at K = 8, 16 and 32 (rows of 1000
 * columns) a Lloyd round takes half the time on the tensor path and so does inference, except
 * where low-precision scores leave most rows undecided (unimodal data, K = 32: there the fp32
 * pipes are a quarter faster for inference).
 * This and cat_set_apply_column_split are PROCESS-WIDE tuning and test hooks: they change
 * which kernel every later call of every thread launches (never the results), and they are
 * not meant to be flipped while other threads are inside the library. */
void cat_set_tensor_core_min_k(int32_t min_k);
int32_t cat_get_tensor_core_min_k(void);

/* Small problems (D one of 32, 64, 128; K <= 128, and K * D <= 4096 for fitting; at least 128
 * rows; K >= the tensor-core threshold above) have persistent single-launch kernels: scores on the
 * tensor cores, undecided rows settled in fp64 inside the kernel, and for fitting the per-cluster
 * sums kept on chip and combined across the grid in a fixed order, all rounds in one launch.
 * mask bit 0: the whole of cat_apply (Algorithm 2) runs that way.  mask bit 1: so do the K-Means
 * rounds and the final assignment of cat_fit / cat_fit_from (Algorithm 1, step 2; calls without
 * per-round diagnostics).  Default 3: both are the faster form where they apply.  Clearing a bit
 * sends these shapes down the general multi-launch path instead: same labels (rows on a bisector
 * apart, when a centroid differs in its last bit); sums that agree to fp64 rounding.  A PROCESS-WIDE
 * tuning and test hook like the one above. */
void cat_set_small_problem_kernels(int32_t mask);
int32_t cat_get_small_problem_kernels(void);

/* 1 if the tensor-core kernels can run in this process (the driver hands out the tensor-map
 * encoder they need), 0 if not.  When it is 0 every call takes the fp32-pipe kernels, which
 * give the same results about ten times slower for large K; callers that depend on the speed
 * should check this once. */
int32_t cat_tensor_path_available(void);

/* Form of the fused inference kernel on the tensor-core path.  All forms compute the same thing
 * (bit-identical outputs):
 *   1   TF32 row tiles: a CTA pair shares 256 rows, each CTA all D columns of its 128;
 *   2,4 column split: the CTAs of a cluster share 128 rows, each staging D / cs columns, partial
 *       scores summed through distributed shared memory (needs D a multiple of 32 cs, K rounded
 *       up to 32 cs at most 256, N > 128);
 *   64  64-row tiles on fp16 operands converted inside the kernel (needs D >= 128, D % 8 == 0);
 *   0   chosen from the shape (default).
 * A form that the shape does not allow falls back to form 1.  Other values count as 0.
 * Process-wide, see above. */
void cat_set_apply_column_split(int32_t cs);
int32_t cat_get_apply_column_split(void);

const char *cat_status_string(cat_status_t status);
int cat_last_cuda_error(void);           /* cudaError_t of the last failing runtime call on this thread */
const char *cat_version(void);
int64_t cat_kernel_launches(void);       /* kernels launched by this library in this process so far */

#ifdef __cplusplus
}
#endif
#endif /* CAT_H_ */
