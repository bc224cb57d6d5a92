// cat_assign_noalloc: nearest-centroid labels for callers that may not allocate device
// memory.  The scratch that cat_assign takes from a caller-provided workspace (the control
// block, the squared centroid norms and the queue of rows that need the exact pass) lives
// here in one file-scope device array of fixed size, so the call needs nothing but its
// inputs and outputs.  The array is part of the loaded library image: every GPU that loads
// the library holds it (about 1 MiB) until the process exits.
#include "cat_internal.cuh"

#include <mutex>

namespace {

constexpr size_t kCtlBytes = 256;                                        // cat::Control, padded
constexpr size_t kNormBytes = (size_t)CAT_MAX_K * sizeof(float);         // 2 KiB
constexpr size_t kQueueBytes = (size_t)CAT_NOALLOC_MAX_ROWS * sizeof(int32_t);  // 1 MiB
constexpr size_t kScratchBytes = kCtlBytes + kNormBytes + kQueueBytes;
static_assert(sizeof(cat::Control) <= kCtlBytes, "control block must fit its slot");
static_assert(kNormBytes % 256 == 0, "queue must stay 256-byte aligned");

// In host code this name is only a handle for cudaGetSymbolAddress, never an address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices] = {};  // device address of the array, per device

// Looks up (once per device, with that device current) where the array lives on the device.
cudaError_t scratch_address(unsigned char **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = p;
    }
    *out = reinterpret_cast<unsigned char *>(g_scratch_addr[dev]);
    return cudaSuccess;
}

}  // namespace

extern "C" cat_status_t cat_assign_noalloc(const float *Yq, int64_t N, int32_t D, int32_t K,
                                           const float *centroids, int32_t *labels_out,
                                           void *stream)
{
    using namespace cat;
    if (!Yq || !centroids || !labels_out) return CAT_ERR_NULL;
    if (K < 1 || D < 1 || N < 1) return CAT_ERR_SHAPE;
    if (N > CAT_NOALLOC_MAX_ROWS || K > CAT_MAX_K || D > CAT_MAX_D) return CAT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(Yq) | reinterpret_cast<uintptr_t>(centroids) |
         reinterpret_cast<uintptr_t>(labels_out)) & 15u)
        return CAT_ERR_ALIGN;

    unsigned char *base = nullptr;
    if (!cuda_ok(scratch_address(&base))) return CAT_ERR_CUDA;
    Control *ctl = reinterpret_cast<Control *>(base);
    float *cnorm = reinterpret_cast<float *>(base + kCtlBytes);
    int32_t *queue = reinterpret_cast<int32_t *>(base + kCtlBytes + kNormBytes);

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left.  The only word that must start at
    // zero is the queue length, which the norms kernel clears before the assignment runs;
    // norms and queue entries are rewritten before they are read.
    if (!cuda_ok(launch_centroid_norms(centroids, D, K, cnorm, ctl, s))) return CAT_ERR_CUDA;
    if (!cuda_ok(launch_assign(Yq, N, D, K, centroids, cnorm, labels_out, queue, ctl, nullptr,
                               nullptr, nullptr, s)))
        return CAT_ERR_CUDA;
    if (K > 1 && !cuda_ok(launch_refine(Yq, N, D, K, centroids, labels_out, queue, ctl, nullptr,
                                        nullptr, nullptr, s)))
        return CAT_ERR_CUDA;
    return CAT_OK;
}
