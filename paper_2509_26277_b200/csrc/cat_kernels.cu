// CUDA kernels of the CAT hot path (sm_100a), general fp32 path.
//
//   centroid_norms_kernel   ||c_k||^2 for the expanded-form scores
//   assign_kernel           nearest-centroid scores on the fp32 pipes + certainty test
//                           (+ fused per-cluster affine epilogue for inference)
//   refine_kernel           exact fp64 direct-form decision for the rows the fast
//                           scores cannot separate
//   small element-wise kernels for centroid update, means and the gamma/beta solve
//
// Label decision rule.  The K-Means assignment step needs argmin_k ||y - c_k||^2
// (lowest k on ties).  The fast pass evaluates t_k = ||c_k||^2 - 2 y.c_k in fp32,
// whose error is bounded by
//     e <= u * ((2D + 4) * ||y|| * cmax + 4 * cmax^2),  u = 2^-24, cmax = max_k ||c_k||
// (D-term FMA chain, rounding of the stored norm, the final FMA).  If the two smallest
// scores are further apart than 2e the fast argmin is the exact argmin.  Otherwise the
// row is queued and decided by direct-form fp64 distances, scanning k upwards with a
// strict '<' -- the same arithmetic a straightforward double-precision K-Means uses.
#include "cat_internal.cuh"

#include <math_constants.h>

namespace cat {

constexpr int kMaxDevices = 64;

// ======================================================================================
// small helpers
// ======================================================================================

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src, int src_bytes)
{
    unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem_src),
                 "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ======================================================================================
// centroid norms
// ======================================================================================

__global__ void centroid_norms_kernel(const float *__restrict__ C, int D, int K,
                                      float *__restrict__ cnorm, Control *ctl, int reset_all)
{
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctl->refine_count = 0;
        ctl->cand_count = 0;
        if (reset_all) {
            ctl->device_status = CAT_OK;
            ctl->refined_total = 0;
            ctl->refined_last = 0;
        }
    }
    if (warp >= K) return;
    const float *c = C + (size_t)warp * D;
    double s = 0.0;
    for (int j = lane; j < D; j += 32) {
        double v = (double)c[j];
        s += v * v;
    }
    s = warp_sum(s);
    // round up so that the stored norm never under-states the true one
    if (lane == 0) cnorm[warp] = __double2float_ru(s);
}

cudaError_t launch_centroid_norms(const float *C, int D, int K, float *cnorm, Control *ctl,
                                  cudaStream_t s, bool reset_all)
{
    int threads = 128;
    int blocks = (K * 32 + threads - 1) / threads;
    centroid_norms_kernel<<<blocks, threads, 0, s>>>(C, D, K, cnorm, ctl, reset_all ? 1 : 0);
    count_launch();
    return cudaGetLastError();
}

// ======================================================================================
// assignment (fast fp32 scores)
// ======================================================================================

constexpr int A_BM = 128;       // rows per CTA
constexpr int A_BK = 16;        // D-slab per pipeline stage
constexpr int A_LD = A_BK + 4;  // padded row stride in floats (5 x 16 B: conflict-free 128-bit reads)
constexpr int A_STAGES = 3;
constexpr int A_THREADS = 128;

struct AssignParams {
    const float *Y;
    const float *C;
    const float *cnorm;
    int32_t *labels;
    int32_t *refine_rows;
    Control *ctl;
    const float *gamma;
    const float *beta;
    float *out;
    int64_t N;
    int D;
    int K;
    FastOut fast;
};

template <int BN>
struct AssignSmem {
    float a[A_STAGES][A_BM * A_LD];
    float b[A_STAGES][BN * A_LD];
    float red[4];
    float best[A_BM];
    float second[A_BM];
    int idx[A_BM];
    int lab[A_BM];
};

template <int BN, bool VEC4>
__device__ __forceinline__ void assign_load_tile(AssignSmem<BN> &sm, int stage, const AssignParams &p,
                                                 int64_t row0, int chunk, int k0, int tid)
{
    float *As = sm.a[stage];
    float *Bs = sm.b[stage];
    if (VEC4) {
#pragma unroll
        for (int q = 0; q < (A_BM * A_BK / 4) / A_THREADS; ++q) {
            int e = tid + q * A_THREADS;
            int r = e >> 2, c4 = e & 3;
            int col = k0 + c4 * 4;
            int64_t row = row0 + r;
            bool ok = (row < p.N) && (col < p.D);
            const float *src = ok ? (p.Y + (size_t)row * p.D + col) : p.Y;
            cp_async16(As + r * A_LD + c4 * 4, src, ok ? 16 : 0);
        }
        for (int e = tid; e < BN * A_BK / 4; e += A_THREADS) {
            int n = e >> 2, c4 = e & 3;
            int col = k0 + c4 * 4;
            int k = chunk * BN + n;
            bool ok = (k < p.K) && (col < p.D);
            const float *src = ok ? (p.C + (size_t)k * p.D + col) : p.C;
            cp_async16(Bs + n * A_LD + c4 * 4, src, ok ? 16 : 0);
        }
    } else {
        for (int e = tid; e < A_BM * A_BK; e += A_THREADS) {
            int r = e / A_BK, c = e % A_BK;
            int col = k0 + c;
            int64_t row = row0 + r;
            As[r * A_LD + c] = (row < p.N && col < p.D) ? p.Y[(size_t)row * p.D + col] : 0.f;
        }
        for (int e = tid; e < BN * A_BK; e += A_THREADS) {
            int n = e / A_BK, c = e % A_BK;
            int col = k0 + c;
            int k = chunk * BN + n;
            Bs[n * A_LD + c] = (k < p.K && col < p.D) ? p.C[(size_t)k * p.D + col] : 0.f;
        }
    }
}

// BN centroids per chunk, 8 per thread; TX = BN/8 threads share a row; each thread owns
// TM = TX rows (row = ty + TY*i) so that a CTA always covers 128 rows.
template <int BN, bool VEC4, bool AFFINE>
__global__ void __launch_bounds__(A_THREADS) assign_kernel(AssignParams p)
{
    constexpr int TX = BN / 8;
    constexpr int TY = A_THREADS / TX;
    constexpr int TM = A_BM / TY;
    static_assert(TM == TX, "tile shape");

    extern __shared__ __align__(16) unsigned char smem_raw[];
    AssignSmem<BN> &sm = *reinterpret_cast<AssignSmem<BN> *>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % TX;
    const int ty = tid / TX;
    const int64_t row0 = (int64_t)blockIdx.x * A_BM;

    // cmax^2 = max_k ||c_k||^2
    {
        float m = 0.f;
        for (int k = tid; k < p.K; k += A_THREADS) m = fmaxf(m, p.cnorm[k]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if ((tid & 31) == 0) sm.red[tid >> 5] = m;
    }

    const int ktiles = (p.D + A_BK - 1) / A_BK;
    const int nchunks = (p.K + BN - 1) / BN;
    const int T = ktiles * nchunks;

    for (int s = 0; s < A_STAGES - 1; ++s) {
        if (s < T) assign_load_tile<BN, VEC4>(sm, s, p, row0, s / ktiles, (s % ktiles) * A_BK, tid);
        cp_async_commit();
    }

    float acc[TM][8];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    float rb1[TM], rb2[TM];
    int ridx[TM];
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        rb1[i] = CUDART_INF_F;
        rb2[i] = CUDART_INF_F;
        ridx[i] = 0;
    }
    float ysq = 0.f;  // ||y_row||^2 of row `tid`, accumulated during the first chunk

    int chunk = 0, kt = 0;
    for (int t = 0; t < T; ++t) {
        cp_async_wait<A_STAGES - 2>();
        __syncthreads();
        {
            int tn = t + A_STAGES - 1;
            if (tn < T)
                assign_load_tile<BN, VEC4>(sm, tn % A_STAGES, p, row0, tn / ktiles,
                                           (tn % ktiles) * A_BK, tid);
            cp_async_commit();
        }
        const float *As = sm.a[t % A_STAGES];
        const float *Bs = sm.b[t % A_STAGES];

        if (chunk == 0) {
#pragma unroll
            for (int kk = 0; kk < A_BK; kk += 4) {
                float4 v = *reinterpret_cast<const float4 *>(As + tid * A_LD + kk);
                ysq = fmaf(v.x, v.x, ysq);
                ysq = fmaf(v.y, v.y, ysq);
                ysq = fmaf(v.z, v.z, ysq);
                ysq = fmaf(v.w, v.w, ysq);
            }
        }

#pragma unroll
        for (int kk = 0; kk < A_BK; kk += 4) {
            float4 a[TM];
#pragma unroll
            for (int i = 0; i < TM; ++i)
                a[i] = *reinterpret_cast<const float4 *>(As + (ty + TY * i) * A_LD + kk);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float4 b = *reinterpret_cast<const float4 *>(Bs + (tx + TX * j) * A_LD + kk);
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    acc[i][j] = fmaf(a[i].x, b.x, acc[i][j]);
                    acc[i][j] = fmaf(a[i].y, b.y, acc[i][j]);
                    acc[i][j] = fmaf(a[i].z, b.z, acc[i][j]);
                    acc[i][j] = fmaf(a[i].w, b.w, acc[i][j]);
                }
            }
        }

        if (++kt == ktiles) {
            // scores of this chunk of centroids: t = ||c||^2 - 2 y.c
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                int n = chunk * BN + tx + TX * j;
                float cn = (n < p.K) ? p.cnorm[n] : CUDART_INF_F;
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    float sc = (n < p.K) ? fmaf(-2.f, acc[i][j], cn) : CUDART_INF_F;
                    if (sc < rb1[i]) {
                        rb2[i] = rb1[i];
                        rb1[i] = sc;
                        ridx[i] = n;
                    } else if (sc < rb2[i]) {
                        rb2[i] = sc;
                    }
                    acc[i][j] = 0.f;
                }
            }
            kt = 0;
            ++chunk;
        }
    }
    cp_async_wait<0>();

    // merge the TX threads that share a row
#pragma unroll
    for (int i = 0; i < TM; ++i) {
#pragma unroll
        for (int o = 1; o < TX; o <<= 1) {
            float ob1 = __shfl_xor_sync(0xffffffffu, rb1[i], o);
            float ob2 = __shfl_xor_sync(0xffffffffu, rb2[i], o);
            int oidx = __shfl_xor_sync(0xffffffffu, ridx[i], o);
            bool take = (ob1 < rb1[i]) || (ob1 == rb1[i] && oidx < ridx[i]);
            float hi = take ? rb1[i] : ob1;  // the larger of the two bests
            rb2[i] = fminf(fminf(rb2[i], ob2), hi);
            if (take) {
                rb1[i] = ob1;
                ridx[i] = oidx;
            }
        }
        if (tx == 0) {
            int r = ty + TY * i;
            sm.best[r] = rb1[i];
            sm.second[r] = rb2[i];
            sm.idx[r] = ridx[i];
        }
    }
    __syncthreads();

    {
        const float cmax2 = fmaxf(fmaxf(sm.red[0], sm.red[1]), fmaxf(sm.red[2], sm.red[3]));
        const int64_t row = row0 + tid;
        int lab = -1;
        if (row < p.N) {
            const float u = 5.9604645e-8f;  // 2^-24
            float e = 1.0625f * u *
                      ((2.f * (float)p.D + 4.f) * sqrtf(ysq) * sqrtf(cmax2) + 4.f * cmax2);
            float gap = sm.second[tid] - sm.best[tid];
            int k = sm.idx[tid];
            bool certain = (p.K == 1) || (gap > 2.f * e);
            p.labels[row] = k;
            if (p.fast.best) p.fast.best[row] = sm.best[tid];
            if (p.fast.second) p.fast.second[row] = sm.second[tid];
            if (p.fast.bound) p.fast.bound[row] = e;
            if (p.fast.label) p.fast.label[row] = k;
            if (certain) {
                lab = k;
            } else {
                int slot = atomicAdd(&p.ctl->refine_count, 1);
                p.refine_rows[slot] = (int32_t)row;
            }
        }
        sm.lab[tid] = lab;
    }

    if (AFFINE) {
        __syncthreads();
        if (VEC4) {
            const int D4 = p.D >> 2;
            const float4 *Y4 = reinterpret_cast<const float4 *>(p.Y);
            const float4 *G4 = reinterpret_cast<const float4 *>(p.gamma);
            const float4 *B4 = reinterpret_cast<const float4 *>(p.beta);
            float4 *O4 = reinterpret_cast<float4 *>(p.out);
            for (int r = 0; r < A_BM; r += 4) {
                for (int c = tid; c < D4; c += A_THREADS) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        int l = sm.lab[r + q];
                        if (l < 0) continue;
                        size_t o = (size_t)(row0 + r + q) * D4 + c;
                        float4 y = __ldcs(Y4 + o);
                        float4 g = __ldg(G4 + (size_t)l * D4 + c);
                        float4 b = __ldg(B4 + (size_t)l * D4 + c);
                        float4 v;
                        v.x = fmaf(g.x, y.x, b.x);
                        v.y = fmaf(g.y, y.y, b.y);
                        v.z = fmaf(g.z, y.z, b.z);
                        v.w = fmaf(g.w, y.w, b.w);
                        __stcs(O4 + o, v);
                    }
                }
            }
        } else {
            for (int r = 0; r < A_BM; ++r) {
                int l = sm.lab[r];
                if (l < 0) continue;
                size_t o = (size_t)(row0 + r) * p.D;
                for (int c = tid; c < p.D; c += A_THREADS)
                    p.out[o + c] = fmaf(p.gamma[(size_t)l * p.D + c], p.Y[o + c],
                                        p.beta[(size_t)l * p.D + c]);
            }
        }
    }
}

template <int BN, bool VEC4, bool AFFINE>
static cudaError_t launch_assign_t(const AssignParams &p, cudaStream_t s)
{
    auto kern = assign_kernel<BN, VEC4, AFFINE>;
    size_t smem = sizeof(AssignSmem<BN>);
    static bool configured[kMaxDevices] = {};  // the attribute is kept per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = -1;
    if (dev < 0 || !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0) configured[dev] = true;
    }
    unsigned blocks = (unsigned)((p.N + A_BM - 1) / A_BM);
    kern<<<blocks, A_THREADS, smem, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

template <bool VEC4, bool AFFINE>
static cudaError_t launch_assign_bn(const AssignParams &p, cudaStream_t s)
{
    if (p.K <= 8) return launch_assign_t<8, VEC4, AFFINE>(p, s);
    if (p.K <= 16) return launch_assign_t<16, VEC4, AFFINE>(p, s);
    if (p.K <= 32) return launch_assign_t<32, VEC4, AFFINE>(p, s);
    return launch_assign_t<64, VEC4, AFFINE>(p, s);
}

cudaError_t launch_assign(const float *Y, int64_t N, int D, int K, const float *C,
                          const float *cnorm, int32_t *labels, int32_t *refine_rows, Control *ctl,
                          const float *gamma, const float *beta, float *out, cudaStream_t s,
                          const FastOut *fast)
{
    AssignParams p{Y, C, cnorm, labels, refine_rows, ctl, gamma, beta, out, N, D, K, fast ? *fast : FastOut{}};
    const bool vec = (D % 4 == 0);
    const bool affine = (out != nullptr);
    if (vec) return affine ? launch_assign_bn<true, true>(p, s) : launch_assign_bn<true, false>(p, s);
    return affine ? launch_assign_bn<false, true>(p, s) : launch_assign_bn<false, false>(p, s);
}

// ======================================================================================
// exact decision for queued rows
// ======================================================================================

constexpr int R_THREADS = 256;
constexpr int R_WARPS = R_THREADS / 32;

// One CTA per queued row: warp w evaluates centroids w, w + 8, ... in direct form with fp64
// accumulation; the CTA then takes the smallest distance, lowest index on equality.
// The same decision for RG queued rows per CTA at a time (rows of at most RG_MAX_D columns): the
// rows sit in shared memory as fp64, so a centroid element is fetched and converted once for RG
// rows and a row element is converted once for all K centroids -- the scan is bound by those
// conversions and by the fp64 pipe, not by memory.  Warp w takes centroids w, w + 8, ... for all
// rows of the group; lowest index on equality, as in the single-row form.
constexpr int RG = 4;
constexpr int RG_MAX_D = 1024;

template <bool AFFINE>
__device__ __forceinline__ void refine_body_grouped(const float *__restrict__ Y, int64_t N, int D, int K,
                                                    const float *__restrict__ C, int32_t *labels,
                                                    const int32_t *__restrict__ refine_rows, Control *ctl,
                                                    const float *gamma, const float *beta, float *out,
                                                    double *ys /* [RG][D] shared */)
{
    __shared__ double g_best[R_WARPS][RG];
    __shared__ int g_idx[R_WARPS][RG];
    __shared__ int g_label[RG];
    __shared__ int64_t g_row[RG];
    int count = ctl->refine_count;
    if ((int64_t)count > N) count = (int)N;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctl->refined_total += count;
        ctl->refined_last = count + ctl->cand_count;
    }
    const int lane = threadIdx.x & 31;
    const int w = threadIdx.x >> 5;
    for (int base = blockIdx.x * RG; base < count; base += gridDim.x * RG) {
        const int nr = (count - base < RG) ? (count - base) : RG;
        if (threadIdx.x < RG) {
            int64_t row = (threadIdx.x < nr) ? (int64_t)refine_rows[base + threadIdx.x] : -1;
            if (row >= N) row = -1;
            g_row[threadIdx.x] = row;
        }
        __syncthreads();
        for (int r = 0; r < RG; ++r) {
            const int64_t row = g_row[r];
            for (int j = threadIdx.x; j < D; j += R_THREADS)
                ys[r * D + j] = (row >= 0) ? (double)Y[(size_t)row * D + j] : 0.0;
        }
        __syncthreads();
        double best[RG];
        int bk[RG];
#pragma unroll
        for (int r = 0; r < RG; ++r) {
            best[r] = CUDART_INF;
            bk[r] = K;
        }
        for (int k = w; k < K; k += R_WARPS) {
            const float *c = C + (size_t)k * D;
            double s[RG];
#pragma unroll
            for (int r = 0; r < RG; ++r) s[r] = 0.0;
            for (int j = lane; j < D; j += 32) {
                const double cv = (double)c[j];
#pragma unroll
                for (int r = 0; r < RG; ++r) {
                    const double d = ys[r * D + j] - cv;
                    s[r] = fma(d, d, s[r]);
                }
            }
#pragma unroll
            for (int r = 0; r < RG; ++r) {
                const double v = warp_sum(s[r]);
                if (v < best[r]) {
                    best[r] = v;
                    bk[r] = k;
                }
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < RG; ++r) {
                g_best[w][r] = best[r];
                g_idx[w][r] = bk[r];
            }
        }
        __syncthreads();
        if (threadIdx.x < RG) {
            const int r = threadIdx.x;
            double b = g_best[0][r];
            int k = g_idx[0][r];
#pragma unroll
            for (int q = 1; q < R_WARPS; ++q) {
                if (g_best[q][r] < b || (g_best[q][r] == b && g_idx[q][r] < k)) {
                    b = g_best[q][r];
                    k = g_idx[q][r];
                }
            }
            if (k >= K) k = 0;  // only when every distance is NaN
            if (g_row[r] >= 0) labels[g_row[r]] = k;
            g_label[r] = k;
        }
        __syncthreads();
        if (AFFINE) {
            for (int r = 0; r < RG; ++r) {
                const int64_t row = g_row[r];
                if (row < 0) continue;
                const float *y = Y + (size_t)row * D;
                const float *g = gamma + (size_t)g_label[r] * D;
                const float *bb = beta + (size_t)g_label[r] * D;
                float *o = out + (size_t)row * D;
                for (int j = threadIdx.x; j < D; j += R_THREADS) o[j] = fmaf(g[j], y[j], bb[j]);
            }
        }
        __syncthreads();
    }
}

template <bool AFFINE>
__device__ __forceinline__ void refine_body(const float *__restrict__ Y, int64_t N, int D, int K,
                                            const float *__restrict__ C, int32_t *labels,
                                            const int32_t *__restrict__ refine_rows, Control *ctl,
                                            const float *gamma, const float *beta, float *out)
{
    __shared__ double s_best[R_WARPS];
    __shared__ int s_idx[R_WARPS];
    __shared__ int s_label;
    int count = ctl->refine_count;
    if ((int64_t)count > N) count = (int)N;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // the candidate pass (if any) ran before this kernel and has already added its rows
        ctl->refined_total += count;
        ctl->refined_last = count + ctl->cand_count;
    }
    const int lane = threadIdx.x & 31;
    const int w = threadIdx.x >> 5;
    for (int it = blockIdx.x; it < count; it += gridDim.x) {
        int64_t row = refine_rows[it];
        if (row < 0 || row >= N) continue;  // uniform across the CTA
        const float *y = Y + (size_t)row * D;
        double best = CUDART_INF;
        int bk = K;  // "none": loses every comparison below
        for (int k = w; k < K; k += R_WARPS) {
            const float *c = C + (size_t)k * D;
            double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
            int j = lane;
            for (; j + 96 < D; j += 128) {
                double d0 = (double)y[j] - (double)c[j];
                double d1 = (double)y[j + 32] - (double)c[j + 32];
                double d2 = (double)y[j + 64] - (double)c[j + 64];
                double d3 = (double)y[j + 96] - (double)c[j + 96];
                s0 = fma(d0, d0, s0);
                s1 = fma(d1, d1, s1);
                s2 = fma(d2, d2, s2);
                s3 = fma(d3, d3, s3);
            }
            for (; j < D; j += 32) {
                double d0 = (double)y[j] - (double)c[j];
                s0 = fma(d0, d0, s0);
            }
            double s = warp_sum((s0 + s1) + (s2 + s3));
            if (s < best) {
                best = s;
                bk = k;
            }
        }
        if (lane == 0) {
            s_best[w] = best;
            s_idx[w] = bk;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            double b = s_best[0];
            int k = s_idx[0];
#pragma unroll
            for (int q = 1; q < R_WARPS; ++q) {
                if (s_best[q] < b || (s_best[q] == b && s_idx[q] < k)) {
                    b = s_best[q];
                    k = s_idx[q];
                }
            }
            if (k >= K) k = 0;  // only when every distance is NaN
            labels[row] = k;
            s_label = k;
        }
        __syncthreads();
        if (AFFINE) {
            const int l = s_label;
            const float *g = gamma + (size_t)l * D;
            const float *bb = beta + (size_t)l * D;
            float *o = out + (size_t)row * D;
            for (int j = threadIdx.x; j < D; j += R_THREADS) o[j] = fmaf(g[j], y[j], bb[j]);
        }
        __syncthreads();
    }
}

template <bool AFFINE>
__global__ void __launch_bounds__(R_THREADS) refine_kernel(const float *__restrict__ Y, int64_t N,
                                                           int D, int K, const float *__restrict__ C,
                                                           int32_t *labels,
                                                           const int32_t *__restrict__ refine_rows,
                                                           Control *ctl, const float *gamma,
                                                           const float *beta, float *out)
{
    extern __shared__ double refine_rows_f64[];
    if (D <= RG_MAX_D) refine_body_grouped<AFFINE>(Y, N, D, K, C, labels, refine_rows, ctl, gamma, beta, out, refine_rows_f64);
    else refine_body<AFFINE>(Y, N, D, K, C, labels, refine_rows, ctl, gamma, beta, out);
}

// dynamic shared memory of the full-K exact pass: RG rows as fp64 where the grouped form applies
static size_t refine_smem_bytes(int D) { return D <= RG_MAX_D ? (size_t)RG * D * sizeof(double) : 0; }

cudaError_t launch_refine(const float *Y, int64_t N, int D, int K, const float *C,
                          int32_t *labels, const int32_t *refine_rows, Control *ctl,
                          const float *gamma, const float *beta, float *out, cudaStream_t s)
{
    int blocks = (int)(N < 1184 ? N : 1184);
    if (out)
        refine_kernel<true><<<blocks, R_THREADS, refine_smem_bytes(D), s>>>(Y, N, D, K, C, labels, refine_rows, ctl,
                                                         gamma, beta, out);
    else
        refine_kernel<false><<<blocks, R_THREADS, refine_smem_bytes(D), s>>>(Y, N, D, K, C, labels, refine_rows, ctl,
                                                          gamma, beta, out);
    count_launch();
    return cudaGetLastError();
}

// Exact decision among at most four listed candidates: one warp per queued row, the
// candidates' fp64 direct-form distances formed together (the row is read once).
constexpr int RC_THREADS = 256;

template <bool AFFINE>
__device__ __forceinline__ void refine_candidates_body(
    const float *__restrict__ Y, int64_t N, int D, int K, const float *__restrict__ C, int32_t *labels,
    const int32_t *__restrict__ cand_rows, const uint64_t *__restrict__ cand_list, Control *ctl,
    const float *gamma, const float *beta, float *out, bool fast_output_valid)
{
    int count = ctl->cand_count;
    if ((int64_t)count > N) count = (int)N;
    if (blockIdx.x == 0 && threadIdx.x == 0) ctl->refined_total += count;
    const int lane = threadIdx.x & 31;
    const bool vec4 = (D & 3) == 0 && ((reinterpret_cast<uintptr_t>(Y) | reinterpret_cast<uintptr_t>(C)) & 15u) == 0 &&
                      (!AFFINE || ((reinterpret_cast<uintptr_t>(gamma) | reinterpret_cast<uintptr_t>(beta) |
                                    reinterpret_cast<uintptr_t>(out)) & 15u) == 0);
    const int gw = blockIdx.x * (RC_THREADS / 32) + (threadIdx.x >> 5);
    const int nw = gridDim.x * (RC_THREADS / 32);
    // A warp walks its rows one after the other, and each row is a chain of dependent loads (queue
    // entry -> row and centroids -> label): the queue entry of the warp's next row is fetched while
    // this row is worked on, and the row's fast label is requested together with its data.
    int64_t next_row = (gw < count) ? (int64_t)cand_rows[gw] : -1;
    uint64_t next_packed = (gw < count) ? cand_list[gw] : 0;
    for (int it = gw; it < count; it += nw) {
        const int64_t row = next_row;
        const uint64_t packed = next_packed;
        if (it + nw < count) {
            next_row = cand_rows[it + nw];
            next_packed = cand_list[it + nw];
        }
        if (row < 0 || row >= N) continue;
        const int fast = labels[row];
        int cand[4];
        const float *cp[4];
        int ncand = 0;   // the list is filled from the front: unused slots are at the end
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int k = (int)((packed >> (16 * q)) & 0xFFFFu);
            cand[q] = (k < K) ? k : -1;
            cp[q] = C + (size_t)(k < K ? k : 0) * D;
            if (k < K) ncand = q + 1;
        }
        const float *y = Y + (size_t)row * D;
        double s[4] = {0.0, 0.0, 0.0, 0.0};
        if (vec4) {
            // rows and centroids as 128-bit loads (D a multiple of 4, bases 16-byte aligned)
            const float4 *y4 = reinterpret_cast<const float4 *>(y);
            const int D4 = D >> 2;
            if (ncand <= 2) {
                const float4 *c0 = reinterpret_cast<const float4 *>(cp[0]);
                const float4 *c1 = reinterpret_cast<const float4 *>(cp[1]);
                // (unrolled so that the loads of several steps are in flight together: one warp walks
                // its row alone, and a step that waited for its own loads cost a memory latency each)
#pragma unroll 8
                for (int j = lane; j < D4; j += 32) {
                    const float4 yv = y4[j], a = c0[j], b = c1[j];
                    double d;
                    d = (double)yv.x - (double)a.x; s[0] = fma(d, d, s[0]);
                    d = (double)yv.y - (double)a.y; s[0] = fma(d, d, s[0]);
                    d = (double)yv.z - (double)a.z; s[0] = fma(d, d, s[0]);
                    d = (double)yv.w - (double)a.w; s[0] = fma(d, d, s[0]);
                    d = (double)yv.x - (double)b.x; s[1] = fma(d, d, s[1]);
                    d = (double)yv.y - (double)b.y; s[1] = fma(d, d, s[1]);
                    d = (double)yv.z - (double)b.z; s[1] = fma(d, d, s[1]);
                    d = (double)yv.w - (double)b.w; s[1] = fma(d, d, s[1]);
                }
            } else {
#pragma unroll 4
                for (int j = lane; j < D4; j += 32) {
                    const float4 yv = y4[j];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 c = reinterpret_cast<const float4 *>(cp[q])[j];
                        double d;
                        d = (double)yv.x - (double)c.x; s[q] = fma(d, d, s[q]);
                        d = (double)yv.y - (double)c.y; s[q] = fma(d, d, s[q]);
                        d = (double)yv.z - (double)c.z; s[q] = fma(d, d, s[q]);
                        d = (double)yv.w - (double)c.w; s[q] = fma(d, d, s[q]);
                    }
                }
            }
        } else if (ncand <= 2) {
            // the common case: only the two nearest are in question
            for (int j = lane; j < D; j += 32) {
                const double yv = (double)y[j];
                const double d0 = yv - (double)cp[0][j];
                const double d1 = yv - (double)cp[1][j];
                s[0] = fma(d0, d0, s[0]);
                s[1] = fma(d1, d1, s[1]);
            }
        } else {
            for (int j = lane; j < D; j += 32) {
                const double yv = (double)y[j];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const double d = yv - (double)cp[q][j];
                    s[q] = fma(d, d, s[q]);
                }
            }
        }
        double best = CUDART_INF;
        int bk = K;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const double v = warp_sum(s[q]);
            if (cand[q] >= 0 && (v < best || (v == best && cand[q] < bk))) {
                best = v;
                bk = cand[q];
            }
        }
        if (bk >= K) bk = (cand[0] >= 0) ? cand[0] : 0;   // only when every distance is NaN
        // The fast pass has already written this row's output with the label it left in
        // labels[row] (read above); the row is rewritten only when the exact label differs.
        __syncwarp();
        if (lane == 0) labels[row] = bk;
        if (AFFINE && (bk != fast || !fast_output_valid)) {
            const float *g = gamma + (size_t)bk * D;
            const float *bb = beta + (size_t)bk * D;
            float *o = out + (size_t)row * D;
            if (vec4) {
                for (int j = lane; j < (D >> 2); j += 32) {
                    const float4 yv = reinterpret_cast<const float4 *>(y)[j];
                    const float4 gv = reinterpret_cast<const float4 *>(g)[j];
                    const float4 bv = reinterpret_cast<const float4 *>(bb)[j];
                    reinterpret_cast<float4 *>(o)[j] = make_float4(fmaf(gv.x, yv.x, bv.x), fmaf(gv.y, yv.y, bv.y),
                                                                   fmaf(gv.z, yv.z, bv.z), fmaf(gv.w, yv.w, bv.w));
                }
            } else {
                for (int j = lane; j < D; j += 32) o[j] = fmaf(g[j], y[j], bb[j]);
            }
        }
    }
}

// Both exact passes in one launch: the rows queued with their candidates (a warp each), then the
// rows queued for a scan of all K (a CTA each).  A row is in one queue only.
static_assert(RC_THREADS == R_THREADS, "the fused exact pass runs both bodies with one block size");
template <bool AFFINE>
__global__ void __launch_bounds__(R_THREADS) refine_both_kernel(
    const float *__restrict__ Y, int64_t N, int D, int K, const float *__restrict__ C, int32_t *labels,
    const int32_t *__restrict__ cand_rows, const uint64_t *__restrict__ cand_list,
    const int32_t *__restrict__ refine_rows, Control *ctl, const float *gamma, const float *beta, float *out)
{
    pdl_enter();
    refine_candidates_body<AFFINE>(Y, N, D, K, C, labels, cand_rows, cand_list, ctl, gamma, beta, out, AFFINE);
    __syncthreads();   // (block 0's thread 0 updates the counters in both bodies, in this order)
    extern __shared__ double refine_rows_f64[];
    if (D <= RG_MAX_D) refine_body_grouped<AFFINE>(Y, N, D, K, C, labels, refine_rows, ctl, gamma, beta, out, refine_rows_f64);
    else refine_body<AFFINE>(Y, N, D, K, C, labels, refine_rows, ctl, gamma, beta, out);
}

cudaError_t launch_refine_both(const float *Y, int64_t N, int D, int K, const float *C, int32_t *labels,
                               const int32_t *cand_rows, const uint64_t *cand_list, const int32_t *refine_rows,
                               Control *ctl, const float *gamma, const float *beta, float *out, cudaStream_t s)
{
    int64_t want = (N + (RC_THREADS / 32) - 1) / (RC_THREADS / 32);
    int blocks = (int)(want < 1184 ? want : 1184);
    if (out)
        launch_pdl(refine_both_kernel<true>, dim3(blocks), dim3(R_THREADS), refine_smem_bytes(D), s, Y, N, D, K, C, labels,
                   cand_rows, cand_list, refine_rows, ctl, gamma, beta, out);
    else
        launch_pdl(refine_both_kernel<false>, dim3(blocks), dim3(R_THREADS), refine_smem_bytes(D), s, Y, N, D, K, C, labels,
                   cand_rows, cand_list, refine_rows, ctl, gamma, beta, out);
    count_launch();
    return cudaGetLastError();
}

// ======================================================================================
// element-wise kernels
// ======================================================================================

__global__ void centroids_from_sums_kernel(const double *__restrict__ sums,
                                           const int64_t *__restrict__ counts, int D, size_t KD,
                                           float *__restrict__ C)
{
    size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    int64_t n = counts[e / D];
    if (n > 0) C[e] = (float)(sums[e] / (double)n);
}

cudaError_t launch_centroids_from_sums(const double *sums, const int64_t *counts, int D, int K,
                                       float *C, cudaStream_t s)
{
    size_t KD = (size_t)K * D;
    int threads = 256;
    unsigned blocks = (unsigned)((KD + threads - 1) / threads);
    centroids_from_sums_kernel<<<blocks, threads, 0, s>>>(sums, counts, D, KD, C);
    count_launch();
    return cudaGetLastError();
}

// one block per cluster: the cluster's size first (by thread 0, before anyone reads it), then its columns
__global__ void shard_update_kernel(const double *__restrict__ dsums, const int64_t *__restrict__ dcounts, int D,
                                    double *__restrict__ sums, int64_t *__restrict__ counts, float *__restrict__ C)
{
    __shared__ long long n_s;
    const int k = blockIdx.x;
    if (threadIdx.x == 0) {
        const long long n = (long long)counts[k] + (long long)dcounts[k];
        counts[k] = n;
        n_s = n;
    }
    __syncthreads();
    const long long n = n_s;
    for (int j = threadIdx.x; j < D; j += blockDim.x) {
        const size_t e = (size_t)k * D + j;
        const double a = sums[e] + dsums[e];
        sums[e] = a;
        if (n > 0) C[e] = (float)(a / (double)n);
    }
}

cudaError_t launch_shard_update(const double *delta_sums, const int64_t *delta_counts, int D, int K, double *sums,
                                int64_t *counts, float *C, cudaStream_t s)
{
    shard_update_kernel<<<K, 256, 0, s>>>(delta_sums, delta_counts, D, sums, counts, C);
    count_launch();
    return cudaGetLastError();
}

__global__ void means_from_sums_kernel(const double *__restrict__ sums,
                                       const int64_t *__restrict__ counts, int D, size_t KD,
                                       double *__restrict__ mean)
{
    size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    int64_t n = counts[e / D];
    mean[e] = (n > 0) ? sums[e] / (double)n : 0.0;
}

cudaError_t launch_means_from_sums(const double *sums, const int64_t *counts, int D, int K,
                                   double *mean, cudaStream_t s)
{
    size_t KD = (size_t)K * D;
    int threads = 256;
    unsigned blocks = (unsigned)((KD + threads - 1) / threads);
    means_from_sums_kernel<<<blocks, threads, 0, s>>>(sums, counts, D, KD, mean);
    count_launch();
    return cudaGetLastError();
}

// gamma = (cov/n) / max(var/n, 1e-8), beta = muF - gamma*muQ; empty cluster -> (1, 0).
__global__ void solve_kernel(const double *__restrict__ sumQ, const double *__restrict__ sumF,
                             const double *__restrict__ var, const double *__restrict__ cov,
                             const int64_t *__restrict__ counts, int D, size_t KD,
                             float *__restrict__ gamma, float *__restrict__ beta)
{
    size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    int64_t n = counts[e / D];
    if (n <= 0) {
        gamma[e] = 1.f;
        beta[e] = 0.f;
        return;
    }
    double dn = (double)n;
    double v = var[e] / dn;
    double c = cov[e] / dn;
    if (v < 1e-8) v = 1e-8;
    double g = c / v;
    double b = sumF[e] / dn - g * (sumQ[e] / dn);
    gamma[e] = (float)g;
    beta[e] = (float)b;
}

cudaError_t launch_solve(const double *sumQ, const double *sumF, const double *var,
                         const double *cov, const int64_t *counts, int D, int K, float *gamma,
                         float *beta, cudaStream_t s)
{
    size_t KD = (size_t)K * D;
    int threads = 256;
    unsigned blocks = (unsigned)((KD + threads - 1) / threads);
    solve_kernel<<<blocks, threads, 0, s>>>(sumQ, sumF, var, cov, counts, D, KD, gamma, beta);
    count_launch();
    return cudaGetLastError();
}

// gamma' = 1 + alpha (gamma - 1), beta' = alpha beta  (so that gamma' y + beta' is the blend)
__global__ void blend_params_kernel(const float *__restrict__ gamma, const float *__restrict__ beta,
                                    double alpha, size_t KD, float *__restrict__ gb,
                                    float *__restrict__ bb)
{
    size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    gb[e] = (float)(1.0 + alpha * ((double)gamma[e] - 1.0));
    bb[e] = (float)(alpha * (double)beta[e]);
}

cudaError_t launch_blend_params(const float *gamma, const float *beta, float alpha, int64_t KD,
                                float *gamma_b, float *beta_b, cudaStream_t s)
{
    int threads = 256;
    unsigned blocks = (unsigned)((KD + threads - 1) / threads);
    blend_params_kernel<<<blocks, threads, 0, s>>>(gamma, beta, (double)alpha, (size_t)KD, gamma_b,
                                                   beta_b);
    count_launch();
    return cudaGetLastError();
}

__global__ void fit_diag_kernel(const Control *ctl, const int64_t *counts, int K,
                                cat_fit_diag_t *diag)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int64_t empty = 0;
    for (int k = 0; k < K; ++k) empty += (counts[k] == 0);
    diag->refined_rows_total = ctl->refined_total;
    diag->refined_rows_final = ctl->refined_last;
    diag->empty_clusters_final = empty;
    diag->device_status = ctl->device_status;
}

cudaError_t launch_fit_diag(const Control *ctl, const int64_t *counts, int K, cat_fit_diag_t *diag,
                            cudaStream_t s)
{
    fit_diag_kernel<<<1, 32, 0, s>>>(ctl, counts, K, diag);
    count_launch();
    return cudaGetLastError();
}

// ---- per-assignment diagnostics (only when the caller asks for them)

// objective += sum over rows of ||y - c_label||^2 (fp64, one warp per row, one atomic per block)
__global__ void __launch_bounds__(256) diag_objective_kernel(const float *__restrict__ Y, int64_t N, int D,
                                                             const float *__restrict__ C,
                                                             const int32_t *__restrict__ labels, double *objective)
{
    __shared__ double part[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    double acc = 0.0;
    for (int64_t row = (int64_t)blockIdx.x * 8 + w; row < N; row += (int64_t)gridDim.x * 8) {
        const float *y = Y + (size_t)row * D;
        const float *c = C + (size_t)labels[row] * D;
        double s = 0.0;
        for (int j = lane; j < D; j += 32) {
            const double d = (double)y[j] - (double)c[j];
            s = fma(d, d, s);
        }
        acc += warp_sum(s);
    }
    if (lane == 0) part[w] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int q = 0; q < 8; ++q) t += part[q];
        atomicAdd(objective, t);
    }
}

// Rows of the two exact-pass queues whose two nearest centroids are within 1e-6 relative of each
// other in squared distance (fp64 direct form over all K): one warp per queued row.
__global__ void __launch_bounds__(256) diag_near_kernel(const float *__restrict__ Y, int64_t N, int D, int K,
                                                        const float *__restrict__ C,
                                                        const int32_t *__restrict__ refine_rows,
                                                        const int32_t *__restrict__ cand_rows, const Control *ctl,
                                                        long long *near_out)
{
    const int lane = threadIdx.x & 31;
    int nref = ctl->refine_count, ncand = ctl->cand_count;
    if ((int64_t)nref > N) nref = (int)N;
    if ((int64_t)ncand > N) ncand = (int)N;
    const int total = nref + ncand;
    int found = 0;
    for (int q = blockIdx.x * 8 + (threadIdx.x >> 5); q < total; q += gridDim.x * 8) {
        const int64_t row = q < nref ? refine_rows[q] : cand_rows[q - nref];
        if (row < 0 || row >= N) continue;
        const float *y = Y + (size_t)row * D;
        double best = CUDART_INF, second = CUDART_INF;
        for (int k = 0; k < K; ++k) {
            const float *c = C + (size_t)k * D;
            double s = 0.0;
            for (int j = lane; j < D; j += 32) {
                const double d = (double)y[j] - (double)c[j];
                s = fma(d, d, s);
            }
            s = warp_sum(s);
            if (s < best) {
                second = best;
                best = s;
            } else if (s < second) {
                second = s;
            }
        }
        if (K > 1 && (second - best) <= 1e-6 * second) ++found;
    }
    if (lane == 0 && found) atomicAdd(reinterpret_cast<unsigned long long *>(near_out), (unsigned long long)found);
}

__global__ void diag_round_begin_kernel(const Control *ctl, int64_t N, cat_fit_diag_t *diag, int slot, int recorded)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int64_t q = (int64_t)ctl->refine_count + (int64_t)ctl->cand_count;
    diag->undecided_rows[slot] = q < N ? q : N;
    diag->near_tie_rows[slot] = 0;
    diag->objective[slot] = 0.0;
    diag->assignments_recorded = recorded;
}

cudaError_t launch_fit_diag_round(const float *Y, int64_t N, int D, int K, const float *C, const int32_t *labels,
                                  const int32_t *refine_rows, const int32_t *cand_rows, const Control *ctl,
                                  cat_fit_diag_t *diag, int slot, int recorded, cudaStream_t s)
{
    diag_round_begin_kernel<<<1, 32, 0, s>>>(ctl, N, diag, slot, recorded);
    int64_t blocks = (N + 7) / 8;
    if (blocks > 1184) blocks = 1184;
    diag_objective_kernel<<<(unsigned)blocks, 256, 0, s>>>(Y, N, D, C, labels, &diag->objective[slot]);
    diag_near_kernel<<<(unsigned)blocks, 256, 0, s>>>(Y, N, D, K, C, refine_rows, cand_rows, ctl,
                                                      reinterpret_cast<long long *>(&diag->near_tie_rows[slot]));
    count_launch(3);
    return cudaGetLastError();
}

__global__ void reset_control_kernel(Control *ctl)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        ctl->refine_count = 0;
        ctl->cand_count = 0;
        ctl->device_status = CAT_OK;
        ctl->refined_total = 0;
        ctl->refined_last = 0;
        ctl->grid_bar = 0;
    }
}

cudaError_t launch_reset_control(Control *ctl, cudaStream_t s)
{
    reset_control_kernel<<<1, 32, 0, s>>>(ctl);
    count_launch();
    return cudaGetLastError();
}

}  // namespace cat
