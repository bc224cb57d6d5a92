// Host-buffer entry points: cat_apply_host streams rows through device staging buffers
// (H2D copy, fused kernel and D2H copy of consecutive chunks overlap on three streams);
// cat_fit_host copies the fit set in, runs cat_fit and copies the model back.
#include "cat_internal.cuh"

#include <mutex>

namespace cat {

constexpr int H_SLOTS = 3;
constexpr size_t H_CHUNK_BYTES = (size_t)64 << 20;  // per staging buffer

static int64_t host_chunk_rows(int64_t N, int D)
{
    int64_t rows = (int64_t)(H_CHUNK_BYTES / ((size_t)D * sizeof(float)));
    rows = rows / 128 * 128;
    if (rows < 128) rows = 128;
    if (rows > N) rows = N;
    return rows;
}

struct ApplyHostWs {
    float *C, *gamma, *beta;
    float *in[H_SLOTS];
    float *out[H_SLOTS];
    int32_t *labels[H_SLOTS];
    void *assign_ws;
    size_t assign_bytes;
    size_t bytes;
};

static ApplyHostWs carve_apply_host(void *base, int64_t N, int D, int K)
{
    unsigned char *b = reinterpret_cast<unsigned char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) -> void * {
        off = align_up(off, 256);
        void *p = b ? b + off : nullptr;
        off += bytes;
        return p;
    };
    ApplyHostWs w{};
    const int64_t rows = host_chunk_rows(N, D);
    const size_t KD = (size_t)K * D * sizeof(float);
    w.C = (float *)take(KD);
    w.gamma = (float *)take(KD);
    w.beta = (float *)take(KD);
    for (int i = 0; i < H_SLOTS; ++i) {
        w.in[i] = (float *)take((size_t)rows * D * sizeof(float));
        w.out[i] = (float *)take((size_t)rows * D * sizeof(float));
        w.labels[i] = (int32_t *)take((size_t)rows * sizeof(int32_t));
    }
    w.assign_bytes = cat_apply_workspace_bytes(rows, D, K);
    w.assign_ws = take(w.assign_bytes);
    w.bytes = align_up(off, 256);
    return w;
}

// Side streams and events, created once per device and kept for the life of the process.
struct HostPipe {
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t in_ready[H_SLOTS], done[H_SLOTS], out_free[H_SLOTS], start = nullptr;
};
static HostPipe g_pipes[64];
static std::mutex g_pipes_mu;   // first use on a device may come from several host threads at once

static cudaError_t get_pipe(HostPipe **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    HostPipe &p = g_pipes[dev];
    std::lock_guard<std::mutex> lock(g_pipes_mu);
    if (!p.ready) {
        if ((e = cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking)) != cudaSuccess) return e;
        if ((e = cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking)) != cudaSuccess) return e;
        for (int i = 0; i < H_SLOTS; ++i) {
            if ((e = cudaEventCreateWithFlags(&p.in_ready[i], cudaEventDisableTiming)) != cudaSuccess) return e;
            if ((e = cudaEventCreateWithFlags(&p.done[i], cudaEventDisableTiming)) != cudaSuccess) return e;
            if ((e = cudaEventCreateWithFlags(&p.out_free[i], cudaEventDisableTiming)) != cudaSuccess) return e;
        }
        if ((e = cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming)) != cudaSuccess) return e;
        p.ready = true;
    }
    *out = &p;
    return cudaSuccess;
}

}  // namespace cat

using namespace cat;

#define CAT_CUDA(expr)                                  \
    do {                                                \
        if (!cuda_ok((expr))) return CAT_ERR_CUDA;      \
    } while (0)

extern "C" {

size_t cat_apply_host_workspace_bytes(int64_t N, int32_t D, int32_t K)
{
    if (cat_apply_workspace_bytes(N, D, K) == 0) return 0;
    return carve_apply_host(nullptr, N, D, K).bytes;
}

cat_status_t cat_apply_host(const float *Yq_host, int64_t N, int32_t D, int32_t K,
                            const float *centroids_host, const float *gamma_host,
                            const float *beta_host, float *Y_out_host, int32_t *labels_out_host,
                            void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq_host || !centroids_host || !gamma_host || !beta_host || !Y_out_host) return CAT_ERR_NULL;
    if (K < 1 || D < 1 || N < 1) return CAT_ERR_SHAPE;
    if (K > CAT_MAX_K || D > CAT_MAX_D || N >= ((int64_t)1 << 31)) return CAT_ERR_UNSUPPORTED;
    size_t need = cat_apply_host_workspace_bytes(N, D, K);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return CAT_ERR_WORKSPACE;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    HostPipe *pp = nullptr;
    CAT_CUDA(get_pipe(&pp));
    HostPipe &p = *pp;
    ApplyHostWs w = carve_apply_host(workspace, N, D, K);
    const int64_t rows = host_chunk_rows(N, D);
    const size_t KD = (size_t)K * D * sizeof(float);

    // parameters go in on the compute stream; the side streams start after `start`
    CAT_CUDA(cudaMemcpyAsync(w.C, centroids_host, KD, cudaMemcpyHostToDevice, s));
    CAT_CUDA(cudaMemcpyAsync(w.gamma, gamma_host, KD, cudaMemcpyHostToDevice, s));
    CAT_CUDA(cudaMemcpyAsync(w.beta, beta_host, KD, cudaMemcpyHostToDevice, s));
    CAT_CUDA(cudaEventRecord(p.start, s));
    CAT_CUDA(cudaStreamWaitEvent(p.h2d, p.start, 0));
    CAT_CUDA(cudaStreamWaitEvent(p.d2h, p.start, 0));

    const int64_t nchunks = (N + rows - 1) / rows;
    cat_status_t st = CAT_OK;
    for (int64_t c = 0; c < nchunks && st == CAT_OK; ++c) {
        const int slot = (int)(c % H_SLOTS);
        const int64_t r0 = c * rows;
        const int64_t n = (N - r0 < rows) ? (N - r0) : rows;
        const size_t bytes = (size_t)n * D * sizeof(float);
        // in[slot] is free once the kernel of chunk c - H_SLOTS has finished
        if (c >= H_SLOTS) CAT_CUDA(cudaStreamWaitEvent(p.h2d, p.done[slot], 0));
        CAT_CUDA(cudaMemcpyAsync(w.in[slot], Yq_host + (size_t)r0 * D, bytes, cudaMemcpyHostToDevice, p.h2d));
        CAT_CUDA(cudaEventRecord(p.in_ready[slot], p.h2d));
        // out[slot] is free once chunk c - H_SLOTS has been copied out
        CAT_CUDA(cudaStreamWaitEvent(s, p.in_ready[slot], 0));
        if (c >= H_SLOTS) CAT_CUDA(cudaStreamWaitEvent(s, p.out_free[slot], 0));
        st = cat_apply(w.in[slot], n, D, K, w.C, w.gamma, w.beta, w.out[slot], w.labels[slot],
                       w.assign_ws, w.assign_bytes, s);
        if (st != CAT_OK) break;
        CAT_CUDA(cudaEventRecord(p.done[slot], s));
        CAT_CUDA(cudaStreamWaitEvent(p.d2h, p.done[slot], 0));
        CAT_CUDA(cudaMemcpyAsync(Y_out_host + (size_t)r0 * D, w.out[slot], bytes, cudaMemcpyDeviceToHost, p.d2h));
        if (labels_out_host)
            CAT_CUDA(cudaMemcpyAsync(labels_out_host + r0, w.labels[slot], (size_t)n * sizeof(int32_t),
                                     cudaMemcpyDeviceToHost, p.d2h));
        CAT_CUDA(cudaEventRecord(p.out_free[slot], p.d2h));
    }
    // drain everything before returning, also on error
    cudaError_t e1 = cudaStreamSynchronize(p.h2d);
    cudaError_t e2 = cudaStreamSynchronize(s);
    cudaError_t e3 = cudaStreamSynchronize(p.d2h);
    if (st != CAT_OK) return st;
    CAT_CUDA(e1);
    CAT_CUDA(e2);
    CAT_CUDA(e3);
    return CAT_OK;
}

size_t cat_fit_host_workspace_bytes(int64_t N, int32_t D, int32_t K)
{
    size_t f = cat_fit_workspace_bytes(N, D, K);
    if (f == 0) return 0;
    size_t ND = align_up((size_t)N * D * sizeof(float), 256);
    size_t KD = align_up((size_t)K * D * sizeof(float), 256);
    return 2 * ND + 3 * KD + align_up((size_t)N * sizeof(int32_t), 256) + f;
}

cat_status_t cat_fit_host(const float *Yq_host, const float *Yfp_host, int64_t N, int32_t D,
                          int32_t K, int32_t iters, float *centroids_out_host,
                          float *gamma_out_host, float *beta_out_host, int32_t *labels_out_host,
                          void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Yq_host || !Yfp_host || !centroids_out_host || !gamma_out_host || !beta_out_host)
        return CAT_ERR_NULL;
    if (K < 1 || D < 1 || N < K || iters < 0) return CAT_ERR_SHAPE;
    size_t need = cat_fit_host_workspace_bytes(N, D, K);
    if (need == 0) return CAT_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    unsigned char *b = reinterpret_cast<unsigned char *>(workspace);
    const size_t ND = align_up((size_t)N * D * sizeof(float), 256);
    const size_t KD = align_up((size_t)K * D * sizeof(float), 256);
    float *Yq = (float *)b;             b += ND;
    float *Yfp = (float *)b;            b += ND;
    float *C = (float *)b;              b += KD;
    float *G = (float *)b;              b += KD;
    float *B = (float *)b;              b += KD;
    int32_t *labels = (int32_t *)b;     b += align_up((size_t)N * sizeof(int32_t), 256);
    const size_t fbytes = cat_fit_workspace_bytes(N, D, K);

    HostPipe *pp = nullptr;
    CAT_CUDA(get_pipe(&pp));
    // the two input copies run on different streams so that they can share the link
    CAT_CUDA(cudaEventRecord(pp->start, s));
    CAT_CUDA(cudaStreamWaitEvent(pp->h2d, pp->start, 0));
    CAT_CUDA(cudaMemcpyAsync(Yq, Yq_host, (size_t)N * D * sizeof(float), cudaMemcpyHostToDevice, s));
    CAT_CUDA(cudaMemcpyAsync(Yfp, Yfp_host, (size_t)N * D * sizeof(float), cudaMemcpyHostToDevice, pp->h2d));
    CAT_CUDA(cudaEventRecord(pp->in_ready[0], pp->h2d));
    CAT_CUDA(cudaStreamWaitEvent(s, pp->in_ready[0], 0));
    cat_status_t st = cat_fit(Yq, Yfp, N, D, K, iters, C, G, B, labels, b, fbytes, s);
    if (st != CAT_OK) {
        cudaStreamSynchronize(s);
        return st;
    }
    const size_t kd = (size_t)K * D * sizeof(float);
    CAT_CUDA(cudaMemcpyAsync(centroids_out_host, C, kd, cudaMemcpyDeviceToHost, s));
    CAT_CUDA(cudaMemcpyAsync(gamma_out_host, G, kd, cudaMemcpyDeviceToHost, s));
    CAT_CUDA(cudaMemcpyAsync(beta_out_host, B, kd, cudaMemcpyDeviceToHost, s));
    if (labels_out_host)
        CAT_CUDA(cudaMemcpyAsync(labels_out_host, labels, (size_t)N * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CAT_CUDA(cudaStreamSynchronize(s));
    return CAT_OK;
}

}  // extern "C"
