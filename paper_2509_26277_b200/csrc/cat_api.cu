// C ABI of libcat.so: argument checks, workspace carving and the launch sequences of
// cat_fit / cat_apply and the step-level entry points declared in cat.h.
#include "cat_internal.cuh"

#include <atomic>

namespace cat {

thread_local int g_last_cuda_error = 0;
static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---------------------------------------------------------------- workspace carving
struct Carver {
    unsigned char *base;
    size_t off = 0;
    explicit Carver(void *b) : base(reinterpret_cast<unsigned char *>(b)) {}
    template <class T>
    T *take(size_t count)
    {
        off = align_up(off, 256);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
};

static void carve_assign_into(Carver &c, AssignWs &w, int64_t N, int D, int K)
{
    w.ctl = c.take<Control>(1);
    w.cnorm = c.take<float>((size_t)K);
    w.refine_rows = c.take<int32_t>((size_t)N);
    w.labels = c.take<int32_t>((size_t)N);
    w.gamma_b = c.take<float>((size_t)K * D);
    w.beta_b = c.take<float>((size_t)K * D);
    w.ynorm2 = c.take<float>((size_t)N);
    w.cand_rows = c.take<int32_t>((size_t)N);
    w.cand_list = c.take<uint64_t>((size_t)N);
    w.ch = c.take<uint16_t>((size_t)K * D);
    w.hscale = c.take<float>(4);
}

AssignWs carve_assign(void *base, int64_t N, int D, int K)
{
    Carver c(base);
    AssignWs w{};
    carve_assign_into(c, w, N, D, K);
    w.bytes = align_up(c.off, 256);
    return w;
}

FitWs carve_fit(void *base, int64_t N, int D, int K)
{
    Carver c(base);
    FitWs w{};
    carve_assign_into(c, w.a, N, D, K);
    SegGeom g = seg_geometry(2 * N, D, 2 * K);   // delta mode is the larger of the two
    size_t KD = (size_t)K * D;
    w.blk_hist = c.take<uint32_t>((size_t)g.nblk * 2 * K);
    w.key_total = c.take<uint32_t>((size_t)2 * K);
    w.cluster_start = c.take<int32_t>((size_t)2 * K + 1);
    w.seg_start = c.take<int32_t>((size_t)2 * K + 2);
    w.order = c.take<int32_t>((size_t)2 * N);
    w.labels_prev = c.take<int32_t>((size_t)N);
    {
        // two planes per segment in delta mode, three in the single-sweep final pass (full mode)
        const SegGeom gf = seg_geometry(N, D, K);
        const size_t a = (size_t)g.max_segs * 2, b = (size_t)gf.max_segs * 3;
        w.segpart = c.take<double>((a > b ? a : b) * D);
    }
    w.yh = c.take<uint16_t>((size_t)N * D);
    w.ch = c.take<uint16_t>(KD);
    w.hscale = c.take<float>(4 + (size_t)N);
    w.sumQ = c.take<double>(KD);
    w.sumF = c.take<double>(KD);
    w.var = c.take<double>(KD);
    w.cov = c.take<double>(KD);
    w.meanQ = c.take<double>(KD);
    w.meanF = c.take<double>(KD);
    w.counts = c.take<int64_t>((size_t)K);
    if (small_fit_supported(N, D, K)) {
        // per-CTA partial sums and sizes of the persistent small-problem kernel
        w.small_part = c.take<double>(small_part_doubles(D, K));
        w.small_counts = c.take<int32_t>(small_part_counts(K));
    }
    w.bytes = align_up(c.off, 256);
    return w;
}

// ---------------------------------------------------------------- validation
static cat_status_t check_shape(int64_t N, int32_t D, int32_t K, bool need_n_ge_k)
{
    if (K < 1 || D < 1 || N < 1) return CAT_ERR_SHAPE;
    if (need_n_ge_k && N < K) return CAT_ERR_SHAPE;
    if (K > CAT_MAX_K || D > CAT_MAX_D || N >= ((int64_t)1 << 31)) return CAT_ERR_UNSUPPORTED;
    return CAT_OK;
}

#define CAT_CUDA(expr)                                  \
    do {                                                \
        if (!cuda_ok((expr))) return CAT_ERR_CUDA;      \
    } while (0)

static std::atomic<int> g_tc_min_k{8};
static std::atomic<int> g_small_kernels{3};   // bit 0: inference, bit 1: the K-Means rounds of a fit

static bool use_tensor_path(int64_t N, int D, int K)
{
    return K >= g_tc_min_k.load(std::memory_order_relaxed) && tc_supported(N, D, K);
}

// the persistent single-launch kernels take the small shapes they support, unless switched off
static bool use_small_fit(int64_t N, int D, int K)
{
    return (g_small_kernels.load(std::memory_order_relaxed) & 2) && use_tensor_path(N, D, K) && small_fit_supported(N, D, K);
}
static bool use_small_apply(int64_t N, int D, int K)
{
    return (g_small_kernels.load(std::memory_order_relaxed) & 1) && use_tensor_path(N, D, K) && small_apply_supported(N, D, K);
}

// norms -> fast assignment (tensor cores for large K, fp32 pipes otherwise) -> exact pass for
// undecided rows.  row_norms_ready: w.ynorm2 already holds this Y's squared row norms.
static cat_status_t run_assign(const float *Y, int64_t N, int D, int K, const float *C,
                               int32_t *labels, const AssignWs &w, const float *gamma,
                               const float *beta, float *out, cudaStream_t s,
                               bool row_norms_ready = false, bool top_level = true,
                               const void *Yh = nullptr, void *Ch = nullptr, const float *hscale = nullptr,
                               bool centroids_ready = false, const FastOut *fast = nullptr)
{
    if (out && labels && top_level && !fast && use_small_apply(N, D, K)) {
        // small problems: everything in one persistent launch (exact decisions included)
        CAT_CUDA(launch_reset_control(w.ctl, s));
        CAT_CUDA(launch_small_apply(Y, N, D, K, C, gamma, beta, out, labels, w.ctl, s));
        return CAT_OK;
    }
    // centroids_ready: the centroid update that produced C has already left its norms, its fp16
    // copy and empty exact-pass queues in the workspace
    if (!centroids_ready) CAT_CUDA(launch_centroid_norms(C, D, K, w.cnorm, w.ctl, s, top_level));
    if (out && use_tensor_path(N, D, K) && choose_apply_form(N, D, K) == 64) {
        // inference on 64-row tiles: fp16 copy of the centroids (scaled by a power of two from
        // their largest magnitude), rows converted inside the kernel
        CAT_CUDA(launch_absmax(C, (size_t)K * D, w.hscale, s));
        CAT_CUDA(launch_half_scale(w.hscale, s));
        CAT_CUDA(launch_to_half(C, (size_t)K * D, w.hscale, w.ch, s));
        CAT_CUDA(launch_apply_h64(Y, N, D, K, w.ch, w.hscale, w.cnorm, labels, w.refine_rows, w.cand_rows, w.cand_list,
                                  w.ctl, gamma, beta, out, s));
        CAT_CUDA(launch_refine_both(Y, N, D, K, C, labels, w.cand_rows, w.cand_list, w.refine_rows, w.ctl, gamma,
                                    beta, out, s));
    } else if (use_tensor_path(N, D, K)) {
        if (!out && !row_norms_ready) CAT_CUDA(launch_row_norms(Y, N, D, w.ynorm2, s));
        if (Yh && !centroids_ready) CAT_CUDA(launch_to_half(C, (size_t)K * D, hscale, Ch, s));
        CAT_CUDA(launch_assign_tc(Y, N, D, K, C, w.cnorm, w.ynorm2, labels, w.refine_rows, w.cand_rows,
                                  w.cand_list, w.ctl, gamma, beta, out, s, Yh, Ch, hscale, fast));
        CAT_CUDA(launch_refine_both(Y, N, D, K, C, labels, w.cand_rows, w.cand_list, w.refine_rows, w.ctl, gamma,
                                    beta, out, s));
    } else {
        CAT_CUDA(launch_assign(Y, N, D, K, C, w.cnorm, labels, w.refine_rows, w.ctl, gamma, beta, out, s, fast));
        if (K > 1) CAT_CUDA(launch_refine(Y, N, D, K, C, labels, w.refine_rows, w.ctl, gamma, beta, out, s));
    }
    return CAT_OK;
}

// sort the rows by label (full mode): counts, cluster/segment tables and `order` in the workspace
static cat_status_t run_sort(const int32_t *labels, int64_t N, int D, int K, const FitWs &w,
                             int64_t *counts, cudaStream_t s)
{
    SegGeom g = seg_geometry(N, D, K);
    CAT_CUDA(launch_label_sort(labels, nullptr, N, K, g, w.blk_hist, w.key_total, counts, w.cluster_start,
                               w.seg_start, w.order, s));
    return CAT_OK;
}

// per-cluster column sums of M for the sorted rows; optionally the centroid update
static cat_status_t run_sums(const float *M, int64_t N, int D, int K, const FitWs &w, const int64_t *counts,
                             double *sums, float *C, cudaStream_t s)
{
    SegGeom g = seg_geometry(N, D, K);
    CAT_CUDA(launch_segment_sums(0, M, nullptr, w.order, w.cluster_start, w.seg_start, nullptr, nullptr, D, K,
                                 g, w.segpart, s));
    CAT_CUDA(launch_segment_combine(w.segpart, w.seg_start, counts, D, K, false, sums, nullptr, C, s));
    return CAT_OK;
}

// One centroid update of a Lloyd round from the rows whose label changed: the running sums
// and sizes in the workspace (sumQ, counts) move by what entered and left each cluster, then
// c_k = sumQ_k / n_k.  `prev` = all -1 makes every row an entry (the first round).
static cat_status_t run_delta_update(const float *Yq, const int32_t *labels, const int32_t *prev, int64_t N, int D,
                                     int K, const FitWs &w, float *C, bool half, cudaStream_t s)
{
    SegGeom g = seg_geometry(2 * N, D, 2 * K);
    CAT_CUDA(launch_label_sort(labels, prev, N, K, g, w.blk_hist, w.key_total, w.counts, w.cluster_start,
                               w.seg_start, w.order, s));
    CAT_CUDA(launch_segment_sums(0, Yq, nullptr, w.order, w.cluster_start, w.seg_start, nullptr, nullptr, D,
                                 2 * K, g, w.segpart, s));
    CAT_CUDA(launch_centroid_update(w.segpart, w.seg_start, w.counts, D, K, w.sumQ, C, w.a.cnorm, w.hscale,
                                    half ? w.ch : nullptr, w.a.ctl, s));
    return CAT_OK;
}

static cat_status_t run_centred(const float *Yq, const float *Yfp, int64_t N, int D, int K, const FitWs &w,
                                const double *meanQ, const double *meanF, double *var, double *cov,
                                cudaStream_t s)
{
    SegGeom g = seg_geometry(N, D, K);
    CAT_CUDA(launch_segment_sums(2, Yq, Yfp, w.order, w.cluster_start, w.seg_start, meanQ, meanF, D, K, g,
                                 w.segpart, s));
    CAT_CUDA(launch_segment_combine(w.segpart, w.seg_start, nullptr, D, K, false, var, cov, nullptr, s));
    return CAT_OK;
}

}  // namespace cat

using namespace cat;

extern "C" {

size_t cat_apply_workspace_bytes(int64_t N, int32_t D, int32_t K)
{
    if (check_shape(N, D, K, false) != CAT_OK) return 0;
    return carve_assign(nullptr, N, D, K).bytes;
}

size_t cat_fit_workspace_bytes(int64_t N, int32_t D, int32_t K)
{
    if (check_shape(N, D, K, false) != CAT_OK || N >= ((int64_t)1 << 30)) return 0;
    return carve_fit(nullptr, N, D, K).bytes;
}

cat_status_t cat_apply_blend(const float *Yq, int64_t N, int32_t D, int32_t K,
                             const float *centroids, const float *gamma, const float *beta,
                             float alpha, float *Y_out, int32_t *labels_out, void *workspace,
                             size_t workspace_bytes, void *stream)
{
    if (!Yq || !centroids || !gamma || !beta || !Y_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (!(alpha >= 0.f && alpha <= 1.f)) return CAT_ERR_SHAPE;
    if (!aligned16(Yq) || !aligned16(centroids) || !aligned16(gamma) || !aligned16(beta) ||
        !aligned16(Y_out) || (labels_out && !aligned16(labels_out)))
        return CAT_ERR_ALIGN;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_apply_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    AssignWs w = carve_assign(workspace, N, D, K);
    int32_t *labels = labels_out ? labels_out : w.labels;
    const float *g = gamma, *b = beta;
    if (alpha != 1.f) {
        CAT_CUDA(launch_blend_params(gamma, beta, alpha, (int64_t)K * D, w.gamma_b, w.beta_b, s));
        g = w.gamma_b;
        b = w.beta_b;
    }
    return run_assign(Yq, N, D, K, centroids, labels, w, g, b, Y_out, s);
}

cat_status_t cat_apply(const float *Yq, int64_t N, int32_t D, int32_t K, const float *centroids,
                       const float *gamma, const float *beta, float *Y_out, int32_t *labels_out,
                       void *workspace, size_t workspace_bytes, void *stream)
{
    return cat_apply_blend(Yq, N, D, K, centroids, gamma, beta, 1.f, Y_out, labels_out, workspace,
                           workspace_bytes, stream);
}

cat_status_t cat_apply_bf16(const float *Yq, int64_t N, int32_t D, int32_t K, const float *centroids,
                            const float *gamma, const float *beta, void *Y_out_bf16, int32_t *labels_out,
                            void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq || !centroids || !gamma || !beta || !Y_out_bf16) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (!aligned16(Yq) || !aligned16(centroids) || !aligned16(gamma) || !aligned16(beta) || !aligned16(Y_out_bf16) ||
        (labels_out && !aligned16(labels_out)))
        return CAT_ERR_ALIGN;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_apply_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    AssignWs w = carve_assign(workspace, N, D, K);
    int32_t *labels = labels_out ? labels_out : w.labels;
    if (use_tensor_path(N, D, K) && apply_h64_supported(N, D, K)) {
        // fused: the 64-row-tile kernel writes bf16 with the fast labels; the exact pass settles the
        // undecided rows' labels, and those rows are written once more
        CAT_CUDA(launch_centroid_norms(centroids, D, K, w.cnorm, w.ctl, s, true));
        CAT_CUDA(launch_absmax(centroids, (size_t)K * D, w.hscale, s));
        CAT_CUDA(launch_half_scale(w.hscale, s));
        CAT_CUDA(launch_to_half(centroids, (size_t)K * D, w.hscale, w.ch, s));
        CAT_CUDA(launch_apply_h64(Yq, N, D, K, w.ch, w.hscale, w.cnorm, labels, w.refine_rows, w.cand_rows, w.cand_list, w.ctl,
                                  gamma, beta, reinterpret_cast<float *>(Y_out_bf16), s, true));
        CAT_CUDA(launch_refine_both(Yq, N, D, K, centroids, labels, w.cand_rows, w.cand_list, w.refine_rows, w.ctl, nullptr,
                                    nullptr, nullptr, s));
        CAT_CUDA(launch_affine_bf16(Yq, N, D, K, labels, gamma, beta, Y_out_bf16, w.refine_rows, w.cand_rows, w.ctl, s));
        return CAT_OK;
    }
    st = run_assign(Yq, N, D, K, centroids, labels, w, nullptr, nullptr, nullptr, s);
    if (st != CAT_OK) return st;
    CAT_CUDA(launch_affine_bf16(Yq, N, D, K, labels, gamma, beta, Y_out_bf16, nullptr, nullptr, nullptr, s));
    return CAT_OK;
}

cat_status_t cat_assign(const float *Yq, int64_t N, int32_t D, int32_t K, const float *centroids,
                        int32_t *labels_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq || !centroids || !labels_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (!aligned16(Yq) || !aligned16(centroids) || !aligned16(labels_out)) return CAT_ERR_ALIGN;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_apply_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    AssignWs w = carve_assign(workspace, N, D, K);
    return run_assign(Yq, N, D, K, centroids, labels_out, w, nullptr, nullptr, nullptr,
                      reinterpret_cast<cudaStream_t>(stream));
}

cat_status_t cat_assign_scores(const float *Yq, int64_t N, int32_t D, int32_t K, const float *centroids,
                               int32_t *labels_out, const cat_fast_scores_t *scores, int32_t flags,
                               void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq || !centroids || !labels_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (flags & ~CAT_ASSIGN_FP16_OPERANDS) return CAT_ERR_SHAPE;
    if (!aligned16(Yq) || !aligned16(centroids) || !aligned16(labels_out)) return CAT_ERR_ALIGN;
    FastOut fast;
    if (scores) {
        fast.best = scores->best;
        fast.second = scores->second;
        fast.bound = scores->bound;
        fast.label = scores->label;
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (flags & CAT_ASSIGN_FP16_OPERANDS) {
        if (!tc_half_supported(N, D, K) || N >= ((int64_t)1 << 30)) return CAT_ERR_UNSUPPORTED;
        if (!workspace || !aligned16(workspace) || workspace_bytes < cat_fit_workspace_bytes(N, D, K))
            return CAT_ERR_WORKSPACE;
        FitWs w = carve_fit(workspace, N, D, K);
        CAT_CUDA(launch_centroid_norms(centroids, D, K, w.a.cnorm, w.a.ctl, s, true));
        CAT_CUDA(launch_half_shadow(Yq, N, D, w.a.ynorm2, w.hscale, w.yh, s));
        CAT_CUDA(launch_to_half(centroids, (size_t)K * D, w.hscale, w.ch, s));
        CAT_CUDA(launch_assign_tc(Yq, N, D, K, centroids, w.a.cnorm, w.a.ynorm2, labels_out, w.a.refine_rows,
                                  w.a.cand_rows, w.a.cand_list, w.a.ctl, nullptr, nullptr, nullptr, s, w.yh, w.ch,
                                  w.hscale, &fast));
        CAT_CUDA(launch_refine_both(Yq, N, D, K, centroids, labels_out, w.a.cand_rows, w.a.cand_list, w.a.refine_rows,
                                    w.a.ctl, nullptr, nullptr, nullptr, s));
        return CAT_OK;
    }
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_apply_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    AssignWs w = carve_assign(workspace, N, D, K);
    return run_assign(Yq, N, D, K, centroids, labels_out, w, nullptr, nullptr, nullptr, s, false, true, nullptr, nullptr,
                      nullptr, false, &fast);
}

cat_status_t cat_fit_from(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K,
                          int32_t iters, const float *init_centroids, float *centroids_out,
                          float *gamma_out, float *beta_out, int32_t *labels_out,
                          cat_fit_diag_t *diag, void *workspace, size_t workspace_bytes,
                          void *stream)
{
    if (!Yq || !Yfp || !centroids_out || !gamma_out || !beta_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, true);
    if (st != CAT_OK) return st;
    if (iters < 0) return CAT_ERR_SHAPE;
    if (N >= ((int64_t)1 << 30)) return CAT_ERR_UNSUPPORTED;   // a round may sort 2N entries with 32-bit positions
    if (!aligned16(Yq) || !aligned16(Yfp) || !aligned16(centroids_out) || !aligned16(gamma_out) ||
        !aligned16(beta_out) || (labels_out && !aligned16(labels_out)) ||
        (init_centroids && !aligned16(init_centroids)) || (diag && !aligned16(diag)))
        return CAT_ERR_ALIGN;
    if (init_centroids == centroids_out) return CAT_ERR_SHAPE;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_fit_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    FitWs w = carve_fit(workspace, N, D, K);
    const size_t KD = (size_t)K * D;
    double *meanQ = w.meanQ;
    int32_t *labels = labels_out ? labels_out : w.a.labels;
    float *C = centroids_out;

    CAT_CUDA(launch_reset_control(w.a.ctl, s));
    CAT_CUDA(cudaMemcpyAsync(C, init_centroids ? init_centroids : Yq, KD * sizeof(float),
                             cudaMemcpyDeviceToDevice, s));

    // Small problems without per-round diagnostics: every round, the final assignment and the
    // per-cluster sums and sizes that follow its labels come from one persistent launch.
    const bool small = !diag && use_small_fit(N, D, K);
    if (small) {
        unsigned int bar_count = 0;   // (the control block was reset above)
        CAT_CUDA(launch_small_fit(Yq, N, D, K, C, iters + 1, false, labels, w.small_part, w.small_counts, w.sumQ,
                                  w.counts, w.a.ctl, &bar_count, s));
    }

    const bool tc = use_tensor_path(N, D, K);
    // Yq is fixed over the fit: its row norms, and where the shape allows an fp16 copy for the
    // tensor cores, are made once
    // (only with the default start: centroids that are rows or means of rows cannot exceed the
    // largest magnitude of Yq, which sets the fp16 scale; caller-provided ones could overflow it)
    const bool half = tc && !init_centroids && tc_half_supported(N, D, K);
    const void *Yh = half ? w.yh : nullptr;
    if (small) {
    } else if (half) CAT_CUDA(launch_half_shadow(Yq, N, D, w.a.ynorm2, w.hscale, w.yh, s));
    else if (tc) CAT_CUDA(launch_row_norms(Yq, N, D, w.a.ynorm2, s));

    // Lloyd rounds.  Two label buffers alternate so that a round sees the previous round's
    // labels and the final assignment lands in `labels`; the running per-cluster sums and
    // sizes start at zero with "no previous label" (-1) for every row.
    const int diag_recorded = iters + 1 < CAT_DIAG_MAX_ROUNDS ? iters + 1 : CAT_DIAG_MAX_ROUNDS;
    int32_t *lab[2] = {labels, w.labels_prev};
    if (!small) {
    CAT_CUDA(cudaMemsetAsync(lab[(iters & 1) ^ 1], 0xFF, (size_t)N * sizeof(int32_t), s));
    CAT_CUDA(cudaMemsetAsync(w.sumQ, 0, KD * sizeof(double), s));
    CAT_CUDA(cudaMemsetAsync(w.counts, 0, (size_t)K * sizeof(int64_t), s));
    for (int t = 0; t < iters; ++t) {
        int32_t *cur = lab[(iters - t) & 1], *prev = lab[((iters - t) & 1) ^ 1];
        st = run_assign(Yq, N, D, K, C, cur, w.a, nullptr, nullptr, nullptr, s, tc, false, Yh, w.ch, w.hscale,
                        t > 0);
        if (st != CAT_OK) return st;
        if (diag && t < CAT_DIAG_MAX_ROUNDS - 1)
            CAT_CUDA(launch_fit_diag_round(Yq, N, D, K, C, cur, w.a.refine_rows, w.a.cand_rows, w.a.ctl, diag, t,
                                           diag_recorded, s));
        st = run_delta_update(Yq, cur, prev, N, D, K, w, C, half, s);
        if (st != CAT_OK) return st;
    }

    // final assignment, then the closed form
    st = run_assign(Yq, N, D, K, C, labels, w.a, nullptr, nullptr, nullptr, s, tc, false, Yh, w.ch, w.hscale,
                    iters > 0);
    if (st != CAT_OK) return st;
    if (diag)
        CAT_CUDA(launch_fit_diag_round(Yq, N, D, K, C, labels, w.a.refine_rows, w.a.cand_rows, w.a.ctl, diag,
                                       diag_recorded - 1, diag_recorded, s));
    // The running sums follow the final labels too (without touching the centroids), which gives
    // the cluster means of Yq before the one sweep over Yq and Yfp that forms the centred moments
    // and the sums of Yfp.
    {
        SegGeom gd = seg_geometry(2 * N, D, 2 * K);
        CAT_CUDA(launch_label_sort(labels, lab[1], N, K, gd, w.blk_hist, w.key_total, w.counts, w.cluster_start,
                                   w.seg_start, w.order, s));
        CAT_CUDA(launch_segment_sums(0, Yq, nullptr, w.order, w.cluster_start, w.seg_start, nullptr, nullptr, D,
                                     2 * K, gd, w.segpart, s));
        CAT_CUDA(launch_segment_combine(w.segpart, w.seg_start, w.counts, D, K, true, w.sumQ, nullptr, nullptr, s));
    }
    }   // !small
    CAT_CUDA(launch_means_from_sums(w.sumQ, w.counts, D, K, meanQ, s));
    st = run_sort(labels, N, D, K, w, w.counts, s);
    if (st != CAT_OK) return st;
    {
        SegGeom g = seg_geometry(N, D, K);
        CAT_CUDA(launch_segment_sums(3, Yq, Yfp, w.order, w.cluster_start, w.seg_start, meanQ, nullptr, D, K, g,
                                     w.segpart, s));
        CAT_CUDA(launch_segment_combine3(w.segpart, w.seg_start, D, K, w.var, w.cov, w.sumF, s));
    }
    CAT_CUDA(launch_solve(w.sumQ, w.sumF, w.var, w.cov, w.counts, D, K, gamma_out, beta_out, s));
    if (diag) CAT_CUDA(launch_fit_diag(w.a.ctl, w.counts, K, diag, s));
    return CAT_OK;
}

cat_status_t cat_fit(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K,
                     int32_t iters, float *centroids_out, float *gamma_out, float *beta_out,
                     int32_t *labels_out, void *workspace, size_t workspace_bytes, void *stream)
{
    return cat_fit_from(Yq, Yfp, N, D, K, iters, nullptr, centroids_out, gamma_out, beta_out,
                        labels_out, nullptr, workspace, workspace_bytes, stream);
}

// ---- row-sharded fitting: the local half of a Lloyd round and the replicated update

cat_status_t cat_fit_shard_begin(const float *Yq, int64_t N, int32_t D, int32_t K, float *amax_out,
                                 void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq || !amax_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (N >= ((int64_t)1 << 30)) return CAT_ERR_UNSUPPORTED;
    if (!aligned16(Yq)) return CAT_ERR_ALIGN;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_fit_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    FitWs w = carve_fit(workspace, N, D, K);
    CAT_CUDA(launch_reset_control(w.a.ctl, s));
    CAT_CUDA(cudaMemsetAsync(w.hscale, 0, 4 * sizeof(float), s));
    const bool tc = use_tensor_path(N, D, K);
    if (tc && tc_half_supported(N, D, K))
        CAT_CUDA(launch_half_shadow(Yq, N, D, w.a.ynorm2, w.hscale, w.yh, s, false));
    else if (tc)
        CAT_CUDA(launch_row_norms(Yq, N, D, w.a.ynorm2, s));
    // (the bit pattern of a non-negative float is the float itself)
    CAT_CUDA(cudaMemcpyAsync(amax_out, w.hscale, sizeof(float), cudaMemcpyDeviceToDevice, s));
    // round 0 sees "no previous label" for every row
    CAT_CUDA(cudaMemsetAsync(w.labels_prev, 0xFF, (size_t)N * sizeof(int32_t), s));
    return CAT_OK;
}

cat_status_t cat_fit_shard_round(const float *Yq, int64_t N, int32_t D, int32_t K, int32_t round,
                                 const float *centroids, const float *amax, double *delta_sums,
                                 int64_t *delta_counts, int32_t *labels_out, void *workspace,
                                 size_t workspace_bytes, void *stream)
{
    if (!Yq || !centroids || !amax || !delta_sums || !delta_counts) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (round < 0) return CAT_ERR_SHAPE;
    if (N >= ((int64_t)1 << 30)) return CAT_ERR_UNSUPPORTED;
    if (!aligned16(Yq) || !aligned16(centroids) || !aligned16(delta_sums) || !aligned16(delta_counts) ||
        (labels_out && !aligned16(labels_out)))
        return CAT_ERR_ALIGN;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_fit_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    FitWs w = carve_fit(workspace, N, D, K);
    const bool tc = use_tensor_path(N, D, K);
    const bool half = tc && tc_half_supported(N, D, K);
    // the two label buffers of the workspace alternate; round 0 reads the all -1 buffer cat_fit_shard_begin left
    int32_t *cur = (round & 1) ? w.labels_prev : w.a.labels;
    int32_t *prev = (round & 1) ? w.a.labels : w.labels_prev;
    if (half) {
        CAT_CUDA(cudaMemcpyAsync(w.hscale, amax, sizeof(float), cudaMemcpyDeviceToDevice, s));
        CAT_CUDA(launch_half_scale(w.hscale, s));
    }
    st = run_assign(Yq, N, D, K, centroids, cur, w.a, nullptr, nullptr, nullptr, s, tc, false, half ? w.yh : nullptr,
                    w.ch, w.hscale, false);
    if (st != CAT_OK) return st;
    const size_t KD = (size_t)K * D;
    CAT_CUDA(cudaMemsetAsync(delta_sums, 0, KD * sizeof(double), s));
    CAT_CUDA(cudaMemsetAsync(delta_counts, 0, (size_t)K * sizeof(int64_t), s));
    SegGeom g = seg_geometry(2 * N, D, 2 * K);
    CAT_CUDA(launch_label_sort(cur, prev, N, K, g, w.blk_hist, w.key_total, delta_counts, w.cluster_start,
                               w.seg_start, w.order, s));
    CAT_CUDA(launch_segment_sums(0, Yq, nullptr, w.order, w.cluster_start, w.seg_start, nullptr, nullptr, D, 2 * K, g,
                                 w.segpart, s));
    CAT_CUDA(launch_segment_combine(w.segpart, w.seg_start, nullptr, D, K, true, delta_sums, nullptr, nullptr, s));
    if (labels_out)
        CAT_CUDA(cudaMemcpyAsync(labels_out, cur, (size_t)N * sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
    return CAT_OK;
}

cat_status_t cat_fit_shard_update(const double *delta_sums, const int64_t *delta_counts, int32_t D, int32_t K,
                                  double *sums_inout, int64_t *counts_inout, float *centroids_inout, void *stream)
{
    if (!delta_sums || !delta_counts || !sums_inout || !counts_inout || !centroids_inout) return CAT_ERR_NULL;
    cat_status_t st = check_shape(K, D, K, false);
    if (st != CAT_OK) return st;
    CAT_CUDA(launch_shard_update(delta_sums, delta_counts, D, K, sums_inout, counts_inout, centroids_inout,
                                 reinterpret_cast<cudaStream_t>(stream)));
    return CAT_OK;
}

cat_status_t cat_cluster_sums(const float *Y, const int32_t *labels, int64_t N, int32_t D,
                              int32_t K, double *sums_out, int64_t *counts_out, void *workspace,
                              size_t workspace_bytes, void *stream)
{
    if (!Y || !labels || !sums_out || !counts_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (!aligned16(Y) || !aligned16(labels) || !aligned16(sums_out) || !aligned16(counts_out))
        return CAT_ERR_ALIGN;
    if (N >= ((int64_t)1 << 30)) return CAT_ERR_UNSUPPORTED;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_fit_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    FitWs w = carve_fit(workspace, N, D, K);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    st = run_sort(labels, N, D, K, w, counts_out, s);
    if (st != CAT_OK) return st;
    return run_sums(Y, N, D, K, w, counts_out, sums_out, nullptr, s);
}

cat_status_t cat_centroids_from_sums(const double *sums, const int64_t *counts, int32_t D,
                                     int32_t K, float *centroids_inout, void *stream)
{
    if (!sums || !counts || !centroids_inout) return CAT_ERR_NULL;
    cat_status_t st = check_shape(K, D, K, false);
    if (st != CAT_OK) return st;
    CAT_CUDA(launch_centroids_from_sums(sums, counts, D, K, centroids_inout,
                                        reinterpret_cast<cudaStream_t>(stream)));
    return CAT_OK;
}

cat_status_t cat_centred_moments(const float *Yq, const float *Yfp, const int32_t *labels,
                                 int64_t N, int32_t D, int32_t K, const double *meanQ,
                                 const double *meanF, double *var_out, double *cov_out,
                                 void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq || !Yfp || !labels || !meanQ || !meanF || !var_out || !cov_out) return CAT_ERR_NULL;
    cat_status_t st = check_shape(N, D, K, false);
    if (st != CAT_OK) return st;
    if (!aligned16(Yq) || !aligned16(Yfp) || !aligned16(labels) || !aligned16(meanQ) ||
        !aligned16(meanF) || !aligned16(var_out) || !aligned16(cov_out))
        return CAT_ERR_ALIGN;
    if (N >= ((int64_t)1 << 30)) return CAT_ERR_UNSUPPORTED;
    if (!workspace || !aligned16(workspace) || workspace_bytes < cat_fit_workspace_bytes(N, D, K))
        return CAT_ERR_WORKSPACE;
    FitWs w = carve_fit(workspace, N, D, K);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    st = run_sort(labels, N, D, K, w, w.counts, s);
    if (st != CAT_OK) return st;
    return run_centred(Yq, Yfp, N, D, K, w, meanQ, meanF, var_out, cov_out, s);
}

cat_status_t cat_solve_gamma_beta(const double *sumQ, const double *sumF, const double *var_sum,
                                  const double *cov_sum, const int64_t *counts, int32_t D,
                                  int32_t K, float *gamma_out, float *beta_out, void *stream)
{
    if (!sumQ || !sumF || !var_sum || !cov_sum || !counts || !gamma_out || !beta_out)
        return CAT_ERR_NULL;
    cat_status_t st = check_shape(K, D, K, false);
    if (st != CAT_OK) return st;
    CAT_CUDA(launch_solve(sumQ, sumF, var_sum, cov_sum, counts, D, K, gamma_out, beta_out,
                          reinterpret_cast<cudaStream_t>(stream)));
    return CAT_OK;
}

cat_status_t cat_workspace_report(const void *workspace, void *stream, int64_t *refined_last_host,
                                  int64_t *refined_total_host, int32_t *device_status_host)
{
    if (!workspace) return CAT_ERR_NULL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    Control h{};
    CAT_CUDA(cudaMemcpyAsync(&h, workspace, sizeof(Control), cudaMemcpyDeviceToHost, s));
    CAT_CUDA(cudaStreamSynchronize(s));
    if (refined_last_host) *refined_last_host = h.refined_last;
    if (refined_total_host) *refined_total_host = h.refined_total;
    if (device_status_host) *device_status_host = h.device_status;
    return CAT_OK;
}

cat_status_t cat_selftest_wait_timeout(void *workspace, size_t workspace_bytes, int32_t limit_ms, void *stream)
{
    if (!workspace) return CAT_ERR_NULL;
    if (!aligned16(workspace) || workspace_bytes < sizeof(Control)) return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    CAT_CUDA(launch_reset_control(reinterpret_cast<Control *>(workspace), s));
    CAT_CUDA(launch_wait_selftest(reinterpret_cast<Control *>(workspace), limit_ms, s));
    return CAT_OK;
}

void cat_set_tensor_core_min_k(int32_t min_k)
{
    g_tc_min_k.store(min_k < 1 ? 1 : min_k, std::memory_order_relaxed);
}

int32_t cat_get_tensor_core_min_k(void) { return g_tc_min_k.load(std::memory_order_relaxed); }

void cat_set_small_problem_kernels(int32_t mask) { g_small_kernels.store(mask & 3, std::memory_order_relaxed); }
int32_t cat_get_small_problem_kernels(void) { return g_small_kernels.load(std::memory_order_relaxed); }

int32_t cat_tensor_path_available(void) { return tc_supported(1, 4, 1) ? 1 : 0; }

void cat_set_apply_column_split(int32_t cs) { set_apply_column_split((int)cs); }

int32_t cat_get_apply_column_split(void) { return (int32_t)get_apply_column_split(); }

const char *cat_status_string(cat_status_t status)
{
    switch (status) {
    case CAT_OK: return "ok";
    case CAT_ERR_NULL: return "a required pointer is NULL";
    case CAT_ERR_SHAPE: return "bad shape or parameter (need N >= K >= 1, D >= 1, iters >= 0, 0 <= alpha <= 1)";
    case CAT_ERR_ALIGN: return "a base pointer is not 16-byte aligned";
    case CAT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CAT_ERR_CUDA: return "a CUDA runtime call failed (see cat_last_cuda_error)";
    case CAT_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
    case CAT_ERR_UNSUPPORTED: return "size beyond the supported limits (CAT_MAX_K, CAT_MAX_D, N < 2^31)";
    default: return "unknown status";
    }
}

int cat_last_cuda_error(void) { return g_last_cuda_error; }
const char *cat_version(void) { return "cat-b200 0.1 (sm_100a)"; }
int64_t cat_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
