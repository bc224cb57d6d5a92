// Internal declarations shared by the translation units of libcat.so.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "cat.h"

namespace cat {

// ---------------------------------------------------------------- launch bookkeeping
extern thread_local int g_last_cuda_error;
void count_launch(int n = 1);

inline bool cuda_ok(cudaError_t e)
{
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return false;
    }
    return true;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Programmatic dependent launch for the chains of short kernels (a Lloyd round is seven of them):
// a kernel launched with launch_pdl may be scheduled while the previous kernel of its stream is
// still running, which hides its launch latency.  Such a kernel calls pdl_enter() before anything
// else: it lets its own dependents be scheduled early, then waits until the previous grid has
// completed and its writes are visible -- so the kernels still run in stream order.  Both
// instructions do nothing in a kernel that was launched the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_enter()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args &&...args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

// ---------------------------------------------------------------- workspace layouts
// Optional outputs of the fast pass (device pointers, each may be null): see cat_fast_scores_t.
struct FastOut {
    float *best = nullptr;
    float *second = nullptr;
    float *bound = nullptr;
    int32_t *label = nullptr;
};

// Control block at the start of every workspace (device memory).
struct Control {
    int32_t refine_count;        // rows queued for the exact fp64 pass by the current assignment
    int32_t device_status;       // CAT_OK or CAT_ERR_DEVICE_TIMEOUT
    int64_t refined_total;       // running total over assignments
    int64_t refined_last;        // rows of the latest finished assignment that took an exact pass
    int32_t cand_count;          // rows queued with a short candidate list by the current assignment
    uint32_t grid_bar;           // arrival counter of the grid-wide barrier of the persistent small-problem kernel
    int64_t pad[4];
};

// Geometry of the sort-based segmented sums for NE entries over KK keys (full mode: N rows,
// K labels; delta mode: 2N virtual entries, 2K keys): identical in the workspace query and
// at launch time.
struct SegGeom {
    int nblk;       // 1024-entry blocks of the sort
    int seg_rows;   // largest rows per segment (multiple of 128); a sort may choose shorter segments
    int max_segs;   // upper bound on the number of segments: ceil(NE / seg_rows) + KK
};
SegGeom seg_geometry(int64_t NE, int D, int KK);

struct AssignWs {          // what assign/apply need
    Control *ctl;
    float *cnorm;          // [K] squared centroid norms, fp32
    int32_t *refine_rows;  // [N]
    int32_t *labels;       // [N] (used when the caller passes no labels_out)
    float *gamma_b;        // [K*D] blended gamma (alpha != 1)
    float *beta_b;         // [K*D]
    float *ynorm2;         // [N] squared row norms (tensor-core labels-only path)
    int32_t *cand_rows;    // [N] rows queued with candidates
    uint64_t *cand_list;   // [N] their candidates, 4 x 16 bit
    void *ch;              // [K*D] fp16 copy of the centroids (inference on fp16 operands)
    float *hscale;         // [4] scale of that copy: {s_c, -2 / s_c, 2^-25 / s_c, -}
    size_t bytes;
};
AssignWs carve_assign(void *base, int64_t N, int D, int K);

struct FitWs {
    AssignWs a;
    // sized for delta mode (2N virtual entries, 2K keys)
    uint32_t *blk_hist;    // [nblk][2K] key histogram / offsets of the sort
    uint32_t *key_total;   // [2K] entries per key
    int32_t *cluster_start; // [2K+1] first position of each key in `order`
    int32_t *seg_start;    // [2K+2] first segment of each key, total, segment length of the current sort
    int32_t *order;        // [2N] row indices sorted by key (stable)
    int32_t *labels_prev;  // [N] labels of the previous Lloyd round
    double *segpart;       // [max_segs][2][D] per-segment partial sums
    void *yh;              // [N*D] fp16 copy of Yq (tensor-core fits with D % 8 == 0)
    void *ch;              // [K*D] fp16 copy of the centroids
    float *hscale;         // [4 + N] scale of the fp16 centroids, then the inverse row scales
    double *sumQ, *sumF, *var, *cov;   // [K*D] each
    double *meanQ, *meanF;             // [K*D] each
    int64_t *counts;       // [K]
    double *small_part;    // [SMALL_MAX_GRID][K*D] per-CTA sums of the persistent small-problem kernel (or null)
    int32_t *small_counts; // [SMALL_MAX_GRID][K+1]
    size_t bytes;
};
FitWs carve_fit(void *base, int64_t N, int D, int K);

// ---------------------------------------------------------------- kernel launchers (cat_kernels.cu)
// All return a cudaError_t from the launch; none synchronises.

// cnorm[k] = ||c_k||^2 (fp64 accumulate, rounded up to fp32); also resets ctl->refine_count,
// and with reset_all the status word and the counters (start of a top-level call).
cudaError_t launch_centroid_norms(const float *C, int D, int K, float *cnorm, Control *ctl,
                                  cudaStream_t s, bool reset_all = false);

// Fast fp32 scores + certainty test; optional fused affine epilogue.
cudaError_t launch_assign(const float *Y, int64_t N, int D, int K, const float *C,
                          const float *cnorm, int32_t *labels, int32_t *refine_rows, Control *ctl,
                          const float *gamma, const float *beta, float *out, cudaStream_t s,
                          const FastOut *fast = nullptr);

// Exact fp64 direct-form labels for the queued rows; optional affine output.
cudaError_t launch_refine(const float *Y, int64_t N, int D, int K, const float *C,
                          int32_t *labels, const int32_t *refine_rows, Control *ctl,
                          const float *gamma, const float *beta, float *out, cudaStream_t s);

// Persistent single-launch kernels for small problems (D in {32, 64, 128}, K <= 128): a run of
// Lloyd rounds with the per-cluster sums in registers and a grid-wide combine, and inference.
constexpr int SMALL_MAX_GRID = 160;   // CTAs the partial-sum planes are sized for
bool small_fit_supported(int64_t N, int D, int K);
bool small_apply_supported(int64_t N, int D, int K);
size_t small_part_doubles(int D, int K);
size_t small_part_counts(int K);
cudaError_t launch_small_fit(const float *Y, int64_t N, int D, int K, float *C, int passes, bool update_last,
                             int32_t *labels, double *part, int32_t *part_counts, double *sums, int64_t *counts,
                             Control *ctl, unsigned int *bar_count, cudaStream_t s);
cudaError_t launch_small_apply(const float *Y, int64_t N, int D, int K, const float *C, const float *gamma,
                               const float *beta, float *out, int32_t *labels, Control *ctl, cudaStream_t s);

// Tensor-core (tcgen05, TF32) variant of launch_assign; ynorm2 is needed when out == nullptr.
bool tc_supported(int64_t N, int D, int K);
// Form of the fused inference kernel on the tensor path: 0 = chosen by shape, 1 = TF32 row tiles
// (128 rows per CTA), 2 / 4 = column split over that many CTAs where it applies, 64 = 64-row tiles
// on fp16 operands made on the fly where that applies.
void set_apply_column_split(int cs);
int get_apply_column_split();
int choose_apply_form(int64_t N, int D, int K);   // 1, 2, 4 or 64 for this shape under the current setting
// 64-row-tile inference kernel on fp16 operands (cat_apply64.cu).  Ch = fp16(C * scale[0]) and
// scale = {s_c, -2 / s_c, 2^-25 / s_c, -} come from launch_absmax + launch_half_scale + launch_to_half.
bool apply_h64_supported(int64_t N, int D, int K);
cudaError_t launch_absmax(const float *src, size_t n, float *scale, cudaStream_t s);   // scale[0] <- bits of max |src|
cudaError_t launch_half_scale(float *scale, cudaStream_t s);                           // bits of the maximum -> the three scale words
cudaError_t launch_apply_h64(const float *Y, int64_t N, int D, int K, const void *Ch, const float *scale,
                             const float *cnorm, int32_t *labels, int32_t *refine_rows, int32_t *cand_rows,
                             uint64_t *cand_list, Control *ctl, const float *gamma, const float *beta, float *out,
                             cudaStream_t s, bool out_bf16 = false);   // out_bf16: `out` is a [N, D] bf16 matrix
// out_bf16[row] = bf16(gamma_l * y + beta_l), l = labels[row]: for all rows (rows == nullptr, n_rows = N) or
// for the listed rows (two lists, lengths read from ctl: the exact-pass queues).
cudaError_t launch_affine_bf16(const float *Y, int64_t N, int D, int K, const int32_t *labels, const float *gamma,
                               const float *beta, void *out_bf16, const int32_t *refine_rows, const int32_t *cand_rows,
                               const Control *ctl, cudaStream_t s);
cudaError_t launch_row_norms(const float *Y, int64_t N, int D, float *out, cudaStream_t s);
// With Yh / Ch / scale (labels only): the fp16 copies of the rows and centroids are the MMA operands.
cudaError_t launch_assign_tc(const float *Y, int64_t N, int D, int K, const float *C, const float *cnorm,
                             const float *ynorm2, int32_t *labels, int32_t *refine_rows,
                             int32_t *cand_rows, uint64_t *cand_list, Control *ctl,
                             const float *gamma, const float *beta, float *out, cudaStream_t s,
                             const void *Yh = nullptr, const void *Ch = nullptr, const float *scale = nullptr,
                             const FastOut *fast = nullptr);

// One warp waits (at most limit_ms, clamped to 1 .. 1000) on a barrier that is never completed.
cudaError_t launch_wait_selftest(Control *ctl, int limit_ms, cudaStream_t s);

// fp16 copy of a matrix for repeated assignments, made in one sweep: squared row norms, per-row
// power-of-two scales, Yh[i] = fp16(Y[i] * scale_i), and scale[4 + N] = {centroid scale s_c from the
// largest magnitude, -2 / s_c, 2^-25 / s_c, unused, then 1 / scale_i for every row}.  Needs D % 8 == 0.
bool tc_half_supported(int64_t N, int D, int K);
// finish_scale = false leaves the bits of the largest magnitude in scale[0] (launch_half_scale turns them
// into the three scale words later, e.g. once the maximum over several shards is known).
cudaError_t launch_half_shadow(const float *Y, int64_t N, int D, float *ynorm2, float *scale, void *Yh,
                               cudaStream_t s, bool finish_scale = true);
// dst = fp16(src * scale[0]) for n elements (n % 4 == 0)
cudaError_t launch_to_half(const float *src, size_t n, const float *scale, void *dst, cudaStream_t s);

// Exact fp64 decision among the listed candidates of each queued row; optional affine output.
cudaError_t launch_refine_both(const float *Y, int64_t N, int D, int K, const float *C, int32_t *labels,
                               const int32_t *cand_rows, const uint64_t *cand_list, const int32_t *refine_rows,
                               Control *ctl, const float *gamma, const float *beta, float *out, cudaStream_t s);

// Stable sort of the row indices by key.  prev == NULL (full mode): key = label, counts[k] = size of
// cluster k.  prev != NULL (delta mode): entries only for rows with labels[i] != prev[i], under keys
// labels[i] and K + prev[i]; counts[k] += (rows that entered k) - (rows that left k).  Tables have one
// entry per key (+1).  Labels outside [0, K) are left out.
cudaError_t launch_label_sort(const int32_t *labels, const int32_t *prev, int64_t N, int K, const SegGeom &g,
                              uint32_t *blk_hist, uint32_t *key_total, int64_t *counts, int32_t *cluster_start,
                              int32_t *seg_start, int32_t *order, cudaStream_t s);

// Per-segment partial sums over KK keys.  mode 0: column sums of Yq (plane 0); mode 1: of Yq and Yf
// (planes 0, 1); mode 2 (full mode only): centred moments sum (q-muQ)^2 (plane 0) and
// sum (q-muQ)(f-muF) (plane 1); mode 3 (full mode only, three planes per segment): sum (q-muQ)^2,
// sum (q-muQ)(f-muQ), sum f.
cudaError_t launch_segment_sums(int mode, const float *Yq, const float *Yf, const int32_t *order,
                                const int32_t *cluster_start, const int32_t *seg_start, const double *meanQ,
                                const double *meanF, int D, int KK, const SegGeom &g, double *part,
                                cudaStream_t s);

// Adds each cluster's segment partials in order into out0 (and out1 if not NULL); in delta mode
// out0[k] += (partials of key k) - (partials of key K + k).  With C also writes the centroid
// float(out0 / n_k) for clusters with n_k > 0.
cudaError_t launch_segment_combine(const double *part, const int32_t *seg_start, const int64_t *counts, int D,
                                   int K, bool delta, double *out0, double *out1, float *C, cudaStream_t s);

// Sums of the three planes of mode 3 per cluster: out0 = sum (q-muQ)^2, out1 = sum (q-muQ)(f-muQ), out2 = sum f.
cudaError_t launch_segment_combine3(const double *part, const int32_t *seg_start, int D, int K, double *out0,
                                    double *out1, double *out2, cudaStream_t s);

// Delta-mode centroid update fused with what the next assignment needs: running sums, centroids,
// their squared norms, (with Ch) their fp16 copy, and the reset of the exact-pass queues.
cudaError_t launch_centroid_update(const double *part, const int32_t *seg_start, const int64_t *counts, int D,
                                   int K, double *sums, float *C, float *cnorm, const float *scale, void *Ch,
                                   Control *ctl, cudaStream_t s);

cudaError_t launch_centroids_from_sums(const double *sums, const int64_t *counts, int D, int K,
                                       float *C, cudaStream_t s);
// sums += delta_sums, counts += delta_counts, C = float(sums / counts) where counts > 0
cudaError_t launch_shard_update(const double *delta_sums, const int64_t *delta_counts, int D, int K, double *sums,
                                int64_t *counts, float *C, cudaStream_t s);
cudaError_t launch_means_from_sums(const double *sums, const int64_t *counts, int D, int K,
                                   double *mean, cudaStream_t s);
cudaError_t launch_solve(const double *sumQ, const double *sumF, const double *var,
                         const double *cov, const int64_t *counts, int D, int K, float *gamma,
                         float *beta, cudaStream_t s);
cudaError_t launch_blend_params(const float *gamma, const float *beta, float alpha, int64_t KD,
                                float *gamma_b, float *beta_b, cudaStream_t s);
cudaError_t launch_fit_diag(const Control *ctl, const int64_t *counts, int K, cat_fit_diag_t *diag,
                            cudaStream_t s);
// Record of one assignment in diag (slot): objective against C for the given labels, rows that were
// queued for the exact pass (the queues of the workspace as the exact pass left them), and how many
// of those have their two nearest centroids within 1e-6 relative.  An extra pass over Y.
cudaError_t launch_fit_diag_round(const float *Y, int64_t N, int D, int K, const float *C, const int32_t *labels,
                                  const int32_t *refine_rows, const int32_t *cand_rows, const Control *ctl,
                                  cat_fit_diag_t *diag, int slot, int recorded, cudaStream_t s);
cudaError_t launch_reset_control(Control *ctl, cudaStream_t s);

}  // namespace cat
