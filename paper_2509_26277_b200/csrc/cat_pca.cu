// PCA front-end of CAT (Section 3.1: the LQ outputs are reduced with PCA before clustering, and
// "PCA is only used to obtain clusters"; Algorithm 1 step 1, Algorithm 2 step 1).
//
//   column means            fp64 partial sums per row chunk, added in a fixed order
//   covariance              D x D, fp64 FMA on 64 x 64 register-tiled CTAs over the centred rows
//                           (upper-triangular tiles, mirrored); 1 / (N - 1) normalisation
//   eigen-decomposition     one-sided Jacobi (Hestenes) in fp64 on the device: plane rotations
//                           orthogonalise the columns of G = Sigma V, all D / 2 disjoint column
//                           pairs of a round-robin step in one launch; a sweep that rotates
//                           nothing ends the iteration (later launches return at once)
//   components              the p columns of V with the largest ||g||, sign fixed so that the entry
//                           of largest magnitude is positive, stored as fp32 rows
//   projection              Z = (Y - mean) V_p^T, fp64 accumulation, fp32 result
//   affine with labels      out_i = gamma_l * y_i + beta_l for given cluster ids (Algorithm 2 steps 4-8)
//
// Everything is deterministic: no floating-point atomics, fixed summation orders.
#include "cat_internal.cuh"

#include <cuda_bf16.h>
#include <math_constants.h>

namespace cat {

namespace {

constexpr int PT = 64;          // tile edge of the fp64 contractions
constexpr int PK = 16;          // depth of a shared-memory step
constexpr int P_THREADS = 256;  // 16 x 16 threads, 4 x 4 outputs each
constexpr int MEAN_CHUNKS = 64;
constexpr int JACOBI_MAX_SWEEPS = 30;

struct PcaCtl {
    int done;       // 1 once a whole sweep has rotated nothing
    int rotated;    // rotations of the current sweep
    int sweeps;     // sweeps carried out
    int pad;
};

// ---------------------------------------------------------------- column means
__global__ void __launch_bounds__(128) col_partial_kernel(const float *__restrict__ Y, int64_t N, int D,
                                                          double *__restrict__ part)
{
    const int col = blockIdx.x * 128 + threadIdx.x;
    const int64_t per = (N + gridDim.y - 1) / gridDim.y;
    const int64_t r0 = (int64_t)blockIdx.y * per;
    const int64_t r1 = r0 + per < N ? r0 + per : N;
    if (col >= D) return;
    double s = 0.0;
    for (int64_t r = r0; r < r1; ++r) s += (double)Y[(size_t)r * D + col];
    part[(size_t)blockIdx.y * D + col] = s;
}

__global__ void col_mean_kernel(const double *__restrict__ part, int chunks, int64_t N, int D,
                                double *__restrict__ mean64, float *__restrict__ mean32)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= D) return;
    double s = 0.0;
    for (int c = 0; c < chunks; ++c) s += part[(size_t)c * D + col];
    s /= (double)N;
    mean64[col] = s;
    if (mean32) mean32[col] = (float)s;
}

// ---------------------------------------------------------------- 64 x 64 fp64 tile product
// acc[u][v] += sum_k As[k][ty * 4 + u] * Bs[k][tx * 4 + v] over one shared-memory step
__device__ __forceinline__ void tile_step(const double (*As)[PT], const double (*Bs)[PT], int ty, int tx,
                                          double (&acc)[4][4])
{
#pragma unroll
    for (int k = 0; k < PK; ++k) {
        double a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) a[u] = As[k][ty * 4 + u];
#pragma unroll
        for (int v = 0; v < 4; ++v) b[v] = Bs[k][tx * 4 + v];
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
    }
}

// Covariance tile (bi, bj), bj >= bi, over the rows of split blockIdx.z:
// part[z][a][b] = sum_i (y_ia - mean_a)(y_ib - mean_b)
__global__ void __launch_bounds__(P_THREADS) cov_kernel(const float *__restrict__ Y, int64_t N, int D,
                                                        const double *__restrict__ mean, double *__restrict__ part)
{
    __shared__ double As[PK][PT], Bs[PK][PT];
    const int bi = blockIdx.y, bj = blockIdx.x;
    if (bj < bi) return;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t per = (N + gridDim.z - 1) / gridDim.z;
    const int64_t r0 = (int64_t)blockIdx.z * per;
    const int64_t r1 = r0 + per < N ? r0 + per : N;
    double acc[4][4] = {};
    for (int64_t r = r0; r < r1; r += PK) {
        // 16 rows x 64 columns per operand: 1024 elements, 4 per thread
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int e = tid + q * P_THREADS, k = e >> 6, c = e & 63;
            const int64_t row = r + k;
            const int ca = bi * PT + c, cb = bj * PT + c;
            As[k][c] = (row < r1 && ca < D) ? (double)Y[(size_t)row * D + ca] - mean[ca] : 0.0;
            Bs[k][c] = (row < r1 && cb < D) ? (double)Y[(size_t)row * D + cb] - mean[cb] : 0.0;
        }
        __syncthreads();
        tile_step(As, Bs, ty, tx, acc);
        __syncthreads();
    }
    double *out = part + (size_t)blockIdx.z * D * D;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int a = bi * PT + ty * 4 + u, b = bj * PT + tx * 4 + v;
            if (a < D && b < D) out[(size_t)a * D + b] = acc[u][v];
        }
}

// G = (sum of the splits' upper triangles, mirrored) / (N - 1); V = identity
__global__ void cov_finish_kernel(const double *__restrict__ part, int splits, int D, int64_t N,
                                  double *__restrict__ G, double *__restrict__ V, PcaCtl *ctl)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) {
        ctl->done = 0;
        ctl->rotated = 0;
        ctl->sweeps = 0;
    }
    if (e >= (size_t)D * D) return;
    const int a = (int)(e / D), b = (int)(e % D);
    const int lo = a < b ? a : b, hi = a < b ? b : a;
    double s = 0.0;
    for (int z = 0; z < splits; ++z) s += part[(size_t)z * D * D + (size_t)lo * D + hi];
    G[e] = s / (double)(N > 1 ? N - 1 : 1);
    V[e] = (a == b) ? 1.0 : 0.0;
}

// ---------------------------------------------------------------- one-sided Jacobi
// Column pairs of round-robin step `step` over n = D rounded up to even "players" (index D, if
// present, is a dummy): pair 0 = (n - 1, step), pair k = ((step + k) mod (n - 1), (step - k) mod (n - 1)).
// G and V are column-major (column c at c * D).  One CTA rotates one pair so that the two columns
// of G become orthogonal; the same rotation goes into V.
__global__ void __launch_bounds__(256) jacobi_step_kernel(double *__restrict__ G, double *__restrict__ V, int D, int n,
                                                          int step, PcaCtl *ctl)
{
    if (ctl->done) return;
    __shared__ double red[3][8];
    __shared__ double cs[2];
    const int k = blockIdx.x;
    int i, j;
    if (k == 0) {
        i = n - 1;
        j = step;
    } else {
        i = (step + k) % (n - 1);
        j = (step - k + (n - 1)) % (n - 1);
    }
    if (i >= D || j >= D) return;
    if (i > j) {
        const int t = i;
        i = j;
        j = t;
    }
    double *gi = G + (size_t)i * D, *gj = G + (size_t)j * D;
    double a = 0.0, b = 0.0, c = 0.0;
    for (int r = threadIdx.x; r < D; r += 256) {
        const double x = gi[r], y = gj[r];
        a = fma(x, x, a);
        b = fma(y, y, b);
        c = fma(x, y, c);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
        c += __shfl_xor_sync(0xffffffffu, c, o);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) {
        red[0][w] = a;
        red[1][w] = b;
        red[2][w] = c;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double aa = 0.0, bb = 0.0, cc = 0.0;
        for (int q = 0; q < 8; ++q) {
            aa += red[0][q];
            bb += red[1][q];
            cc += red[2][q];
        }
        double cth = 1.0, sth = 0.0;
        // rotate unless the two columns are orthogonal to working precision already
        if (fabs(cc) > 1e-15 * sqrt(aa * bb) && cc != 0.0) {
            const double zeta = (bb - aa) / (2.0 * cc);
            const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
            cth = 1.0 / sqrt(1.0 + t * t);
            sth = cth * t;
            atomicAdd(&ctl->rotated, 1);
        }
        cs[0] = cth;
        cs[1] = sth;
    }
    __syncthreads();
    const double cth = cs[0], sth = cs[1];
    if (sth == 0.0) return;
    double *vi = V + (size_t)i * D, *vj = V + (size_t)j * D;
    for (int r = threadIdx.x; r < D; r += 256) {
        const double x = gi[r], y = gj[r];
        gi[r] = cth * x - sth * y;
        gj[r] = sth * x + cth * y;
        const double p = vi[r], q = vj[r];
        vi[r] = cth * p - sth * q;
        vj[r] = sth * p + cth * q;
    }
}

__global__ void jacobi_sweep_end_kernel(PcaCtl *ctl)
{
    if (threadIdx.x != 0 || blockIdx.x != 0 || ctl->done) return;
    ctl->sweeps += 1;
    if (ctl->rotated == 0) ctl->done = 1;
    ctl->rotated = 0;
}

// eigenvalue of column c = ||g_c|| (Sigma is positive semi-definite)
__global__ void __launch_bounds__(256) column_norms_kernel(const double *__restrict__ G, int D, double *__restrict__ lam)
{
    __shared__ double red[8];
    const double *g = G + (size_t)blockIdx.x * D;
    double a = 0.0;
    for (int r = threadIdx.x; r < D; r += 256) a = fma(g[r], g[r], a);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int q = 0; q < 8; ++q) t += red[q];
        lam[blockIdx.x] = sqrt(t);
    }
}

// Column c of V becomes component rank(c) if that rank is below p: rank = number of columns with a
// larger eigenvalue (lower index first among equals).  Sign: the entry of largest magnitude (lowest
// index among equals) is made positive.
__global__ void __launch_bounds__(256) select_components_kernel(const double *__restrict__ V, const double *__restrict__ lam,
                                                                int D, int p, float *__restrict__ comps,
                                                                double *__restrict__ eig_out)
{
    __shared__ int s_rank;
    __shared__ double s_best[8];
    __shared__ int s_idx[8];
    const int c = blockIdx.x;
    const double mine = lam[c];
    int cnt = 0;
    for (int j = threadIdx.x; j < D; j += 256) {
        const double o = lam[j];
        cnt += (o > mine || (o == mine && j < c)) ? 1 : 0;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (threadIdx.x == 0) s_rank = 0;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) atomicAdd(&s_rank, cnt);
    __syncthreads();
    const int rank = s_rank;
    if (rank >= p) return;
    const double *v = V + (size_t)c * D;
    double best = -1.0;
    int bi = D;
    for (int r = threadIdx.x; r < D; r += 256) {
        const double m = fabs(v[r]);
        if (m > best) {
            best = m;
            bi = r;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob > best || (ob == best && oi < bi)) {
            best = ob;
            bi = oi;
        }
    }
    if ((threadIdx.x & 31) == 0) {
        s_best[threadIdx.x >> 5] = best;
        s_idx[threadIdx.x >> 5] = bi;
    }
    __syncthreads();
    double b = s_best[0];
    int ix = s_idx[0];
    for (int q = 1; q < 8; ++q)
        if (s_best[q] > b || (s_best[q] == b && s_idx[q] < ix)) {
            b = s_best[q];
            ix = s_idx[q];
        }
    const double sign = (ix < D && v[ix] < 0.0) ? -1.0 : 1.0;
    for (int r = threadIdx.x; r < D; r += 256) comps[(size_t)rank * D + r] = (float)(sign * v[r]);
    if (threadIdx.x == 0 && eig_out) eig_out[rank] = mine;
}

// ---------------------------------------------------------------- projection
// Z[i, r] = sum_j (Y[i, j] - mean[j]) * comps[r, j], fp64 accumulation: one CTA per 64 rows x 64 components.
__global__ void __launch_bounds__(P_THREADS) project_kernel(const float *__restrict__ Y, int64_t N, int D, int p,
                                                            const float *__restrict__ mean, const float *__restrict__ comps,
                                                            float *__restrict__ Z)
{
    __shared__ double As[PK][PT], Bs[PK][PT];
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t row0 = (int64_t)blockIdx.x * PT;
    const int c0 = blockIdx.y * PT;
    double acc[4][4] = {};
    for (int j0 = 0; j0 < D; j0 += PK) {
        // operand element (m, k): 64 x 16 per operand, 4 per thread; k runs fastest so that a row's
        // 16 columns are read together
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int e = tid + q * P_THREADS, m = e >> 4, k = e & 15;
            const int j = j0 + k;
            const int64_t row = row0 + m;
            As[k][m] = (row < N && j < D) ? (double)Y[(size_t)row * D + j] - (double)mean[j] : 0.0;
            const int r = c0 + m;
            Bs[k][m] = (r < p && j < D) ? (double)comps[(size_t)r * D + j] : 0.0;
        }
        __syncthreads();
        tile_step(As, Bs, ty, tx, acc);
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int64_t row = row0 + ty * 4 + u;
            const int r = c0 + tx * 4 + v;
            if (row < N && r < p) Z[(size_t)row * p + r] = (float)acc[u][v];
        }
}

// ---------------------------------------------------------------- affine map for given cluster ids
// one warp per row: out = fma(gamma_l, y, beta_l); a label outside [0, K) leaves the row as it is
__global__ void __launch_bounds__(256) affine_labels_kernel(const float *__restrict__ Y, int64_t N, int D, int K,
                                                            const int32_t *__restrict__ labels,
                                                            const float *__restrict__ gamma, const float *__restrict__ beta,
                                                            float *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const bool vec4 = (D & 3) == 0;
    for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < N; row += (int64_t)gridDim.x * 8) {
        const int l = labels[row];
        const bool ok = l >= 0 && l < K;
        const float *y = Y + (size_t)row * D;
        const float *g = gamma + (size_t)(ok ? l : 0) * D;
        const float *b = beta + (size_t)(ok ? l : 0) * D;
        float *o = out + (size_t)row * D;
        if (vec4) {
            for (int j = lane; j < (D >> 2); j += 32) {
                const float4 yv = __ldcs(reinterpret_cast<const float4 *>(y) + j);
                float4 v = yv;
                if (ok) {
                    const float4 gv = __ldg(reinterpret_cast<const float4 *>(g) + j);
                    const float4 bv = __ldg(reinterpret_cast<const float4 *>(b) + j);
                    v = make_float4(fmaf(gv.x, yv.x, bv.x), fmaf(gv.y, yv.y, bv.y), fmaf(gv.z, yv.z, bv.z),
                                    fmaf(gv.w, yv.w, bv.w));
                }
                __stcs(reinterpret_cast<float4 *>(o) + j, v);
            }
        } else {
            for (int j = lane; j < D; j += 32) o[j] = ok ? fmaf(g[j], y[j], b[j]) : y[j];
        }
    }
}

// The same with a bf16 result (round to nearest even of the fp32 fused multiply-add), for all rows or
// for the rows of the two exact-pass queues (whose lengths are read from ctl).
__global__ void __launch_bounds__(256) affine_bf16_kernel(const float *__restrict__ Y, int64_t N, int D, int K,
                                                          const int32_t *__restrict__ labels,
                                                          const float *__restrict__ gamma, const float *__restrict__ beta,
                                                          __nv_bfloat16 *__restrict__ out,
                                                          const int32_t *__restrict__ refine_rows,
                                                          const int32_t *__restrict__ cand_rows, const Control *ctl)
{
    const int lane = threadIdx.x & 31;
    const bool listed = ctl != nullptr;
    int64_t nref = 0, total = N;
    if (listed) {
        nref = ctl->refine_count < N ? ctl->refine_count : N;
        const int64_t nc = ctl->cand_count < N ? ctl->cand_count : N;
        total = nref + nc;
    }
    const bool vec4 = (D & 3) == 0;
    for (int64_t q = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); q < total; q += (int64_t)gridDim.x * 8) {
        const int64_t row = listed ? (int64_t)(q < nref ? refine_rows[q] : cand_rows[q - nref]) : q;
        if (row < 0 || row >= N) continue;
        const int l = labels[row];
        const bool ok = l >= 0 && l < K;
        const float *y = Y + (size_t)row * D;
        const float *g = gamma + (size_t)(ok ? l : 0) * D;
        const float *b = beta + (size_t)(ok ? l : 0) * D;
        __nv_bfloat16 *o = out + (size_t)row * D;
        if (vec4) {
            for (int j = lane; j < (D >> 2); j += 32) {
                const float4 yv = __ldcs(reinterpret_cast<const float4 *>(y) + j);
                float4 v = yv;
                if (ok) {
                    const float4 gv = __ldg(reinterpret_cast<const float4 *>(g) + j);
                    const float4 bv = __ldg(reinterpret_cast<const float4 *>(b) + j);
                    v = make_float4(fmaf(gv.x, yv.x, bv.x), fmaf(gv.y, yv.y, bv.y), fmaf(gv.z, yv.z, bv.z),
                                    fmaf(gv.w, yv.w, bv.w));
                }
                const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
                uint2 w2;
                w2.x = *reinterpret_cast<const unsigned int *>(&lo);
                w2.y = *reinterpret_cast<const unsigned int *>(&hi);
                reinterpret_cast<uint2 *>(o)[j] = w2;
            }
        } else {
            for (int j = lane; j < D; j += 32) o[j] = __float2bfloat16_rn(ok ? fmaf(g[j], y[j], b[j]) : y[j]);
        }
    }
}

int cov_splits(int D)
{
    const int T = (D + PT - 1) / PT;
    const int tiles = T * (T + 1) / 2;
    if (tiles >= 64) return 1;
    int s = 128 / tiles;
    return s < 1 ? 1 : (s > 32 ? 32 : s);
}

struct PcaWs {
    PcaCtl *ctl;
    double *mean_part;   // [MEAN_CHUNKS][D]
    double *mean64;      // [D]
    double *lam;         // [D]
    double *G;           // [D][D], column-major
    double *V;           // [D][D], column-major
    double *cov_part;    // [splits][D][D]
    size_t bytes;
};

PcaWs carve_pca(void *base, int D)
{
    unsigned char *b = reinterpret_cast<unsigned char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        off = align_up(off, 256);
        void *q = b ? b + off : nullptr;
        off += bytes;
        return q;
    };
    PcaWs w{};
    const size_t DD = (size_t)D * D;
    w.ctl = (PcaCtl *)take(sizeof(PcaCtl));
    w.mean_part = (double *)take((size_t)MEAN_CHUNKS * D * sizeof(double));
    w.mean64 = (double *)take((size_t)D * sizeof(double));
    w.lam = (double *)take((size_t)D * sizeof(double));
    w.G = (double *)take(DD * sizeof(double));
    w.V = (double *)take(DD * sizeof(double));
    w.cov_part = (double *)take((size_t)cov_splits(D) * DD * sizeof(double));
    w.bytes = align_up(off, 256);
    return w;
}

inline bool al16(const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

}  // namespace

cudaError_t launch_affine_bf16(const float *Y, int64_t N, int D, int K, const int32_t *labels, const float *gamma,
                               const float *beta, void *out_bf16, const int32_t *refine_rows, const int32_t *cand_rows,
                               const Control *ctl, cudaStream_t s)
{
    int64_t blocks = (N + 7) / 8;
    if (blocks > 148 * 16) blocks = 148 * 16;
    affine_bf16_kernel<<<(unsigned)blocks, 256, 0, s>>>(Y, N, D, K, labels, gamma, beta,
                                                        reinterpret_cast<__nv_bfloat16 *>(out_bf16), refine_rows, cand_rows, ctl);
    count_launch();
    return cudaGetLastError();
}

}  // namespace cat

using namespace cat;

#define CAT_CUDA(expr)                                  \
    do {                                                \
        if (!cuda_ok((expr))) return CAT_ERR_CUDA;      \
    } while (0)

static cat_status_t pca_shape(int64_t N, int32_t D, int32_t p)
{
    if (N < 2 || D < 1 || p < 1 || p > D) return CAT_ERR_SHAPE;
    if (D > CAT_PCA_MAX_D || p > CAT_PCA_MAX_P || N >= ((int64_t)1 << 31)) return CAT_ERR_UNSUPPORTED;
    return CAT_OK;
}

extern "C" {

size_t cat_pca_workspace_bytes(int64_t N, int32_t D, int32_t p)
{
    if (pca_shape(N, D, p) != CAT_OK) return 0;
    return carve_pca(nullptr, D).bytes;
}

cat_status_t cat_pca_fit(const float *Yq, int64_t N, int32_t D, int32_t p, float *mean_out,
                         float *components_out, double *eigenvalues_out, void *workspace,
                         size_t workspace_bytes, void *stream)
{
    if (!Yq || !mean_out || !components_out) return CAT_ERR_NULL;
    cat_status_t st = pca_shape(N, D, p);
    if (st != CAT_OK) return st;
    if (!al16(Yq) || !al16(mean_out) || !al16(components_out) || (eigenvalues_out && !al16(eigenvalues_out)))
        return CAT_ERR_ALIGN;
    if (!workspace || !al16(workspace) || workspace_bytes < cat_pca_workspace_bytes(N, D, p)) return CAT_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    PcaWs w = carve_pca(workspace, D);

    int chunks = (int)(N < MEAN_CHUNKS ? N : MEAN_CHUNKS);
    col_partial_kernel<<<dim3((D + 127) / 128, chunks), 128, 0, s>>>(Yq, N, D, w.mean_part);
    col_mean_kernel<<<(D + 255) / 256, 256, 0, s>>>(w.mean_part, chunks, N, D, w.mean64, mean_out);
    const int T = (D + PT - 1) / PT;
    int splits = cov_splits(D);
    if ((int64_t)splits > N) splits = (int)N;
    cov_kernel<<<dim3(T, T, splits), P_THREADS, 0, s>>>(Yq, N, D, w.mean64, w.cov_part);
    const size_t DD = (size_t)D * D;
    cov_finish_kernel<<<(unsigned)((DD + 255) / 256), 256, 0, s>>>(w.cov_part, splits, D, N, w.G, w.V, w.ctl);
    count_launch(4);
    CAT_CUDA(cudaGetLastError());
    if (D > 1) {
        const int n = (D + 1) & ~1;
        for (int sweep = 0; sweep < JACOBI_MAX_SWEEPS; ++sweep) {
            for (int step = 0; step < n - 1; ++step)
                jacobi_step_kernel<<<n / 2, 256, 0, s>>>(w.G, w.V, D, n, step, w.ctl);
            jacobi_sweep_end_kernel<<<1, 32, 0, s>>>(w.ctl);
            count_launch(n);
        }
        CAT_CUDA(cudaGetLastError());
    }
    column_norms_kernel<<<D, 256, 0, s>>>(w.G, D, w.lam);
    select_components_kernel<<<D, 256, 0, s>>>(w.V, w.lam, D, p, components_out, eigenvalues_out);
    count_launch(2);
    CAT_CUDA(cudaGetLastError());
    return CAT_OK;
}

cat_status_t cat_pca_project(const float *Y, int64_t N, int32_t D, int32_t p, const float *mean,
                             const float *components, float *Z_out, void *stream)
{
    if (!Y || !mean || !components || !Z_out) return CAT_ERR_NULL;
    if (N < 1 || D < 1 || p < 1 || p > D) return CAT_ERR_SHAPE;
    if (D > CAT_PCA_MAX_D || p > CAT_PCA_MAX_P || N >= ((int64_t)1 << 31)) return CAT_ERR_UNSUPPORTED;
    if (!al16(Y) || !al16(mean) || !al16(components) || !al16(Z_out)) return CAT_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    project_kernel<<<dim3((unsigned)((N + PT - 1) / PT), (p + PT - 1) / PT), P_THREADS, 0, s>>>(Y, N, D, p, mean, components,
                                                                                             Z_out);
    count_launch();
    CAT_CUDA(cudaGetLastError());
    return CAT_OK;
}

cat_status_t cat_affine_with_labels(const float *Yq, int64_t N, int32_t D, int32_t K, const int32_t *labels,
                                    const float *gamma, const float *beta, float *Y_out, void *stream)
{
    if (!Yq || !labels || !gamma || !beta || !Y_out) return CAT_ERR_NULL;
    if (N < 1 || D < 1 || K < 1) return CAT_ERR_SHAPE;
    if (K > CAT_MAX_K || D > CAT_MAX_D || N >= ((int64_t)1 << 31)) return CAT_ERR_UNSUPPORTED;
    if (!al16(Yq) || !al16(labels) || !al16(gamma) || !al16(beta) || !al16(Y_out)) return CAT_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    int64_t blocks = (N + 7) / 8;
    if (blocks > 148 * 16) blocks = 148 * 16;
    affine_labels_kernel<<<(unsigned)blocks, 256, 0, s>>>(Yq, N, D, K, labels, gamma, beta, Y_out);
    count_launch();
    CAT_CUDA(cudaGetLastError());
    return CAT_OK;
}

// ---- Algorithm 1 and Algorithm 2 with the PCA step, composed from the calls above and the
//      clustering / closed-form entry points

namespace {
struct FitPcaWs {
    void *pca;  size_t pca_bytes;
    float *Z;                       // [N, p]
    float *gp, *bp;                 // [K, p] closed form of the reduced rows (not used further)
    int32_t *labels;                // [N]
    double *sumQ, *sumF, *var, *cov, *meanQ, *meanF;   // [K, D]
    int64_t *counts;                // [K]
    void *fit;  size_t fit_bytes;   // cat_fit workspace for (N, p, K), then for (N, D, K)
    size_t bytes;
};
FitPcaWs carve_fit_pca(void *base, int64_t N, int D, int K, int p)
{
    unsigned char *b = reinterpret_cast<unsigned char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        off = align_up(off, 256);
        void *q = b ? b + off : nullptr;
        off += bytes;
        return q;
    };
    FitPcaWs w{};
    const size_t KD = (size_t)K * D;
    w.pca_bytes = cat_pca_workspace_bytes(N, D, p);
    w.pca = take(w.pca_bytes);
    w.Z = (float *)take((size_t)N * p * sizeof(float));
    w.gp = (float *)take((size_t)K * p * sizeof(float));
    w.bp = (float *)take((size_t)K * p * sizeof(float));
    w.labels = (int32_t *)take((size_t)N * sizeof(int32_t));
    w.sumQ = (double *)take(KD * sizeof(double));
    w.sumF = (double *)take(KD * sizeof(double));
    w.var = (double *)take(KD * sizeof(double));
    w.cov = (double *)take(KD * sizeof(double));
    w.meanQ = (double *)take(KD * sizeof(double));
    w.meanF = (double *)take(KD * sizeof(double));
    w.counts = (int64_t *)take((size_t)K * sizeof(int64_t));
    const size_t a = cat_fit_workspace_bytes(N, p, K), c = cat_fit_workspace_bytes(N, D, K);
    w.fit_bytes = a > c ? a : c;
    w.fit = take(w.fit_bytes);
    w.bytes = align_up(off, 256);
    return w;
}
}  // namespace

size_t cat_fit_pca_workspace_bytes(int64_t N, int32_t D, int32_t K, int32_t p)
{
    if (pca_shape(N, D, p) != CAT_OK || cat_fit_workspace_bytes(N, D, K) == 0 || cat_fit_workspace_bytes(N, p, K) == 0)
        return 0;
    return carve_fit_pca(nullptr, N, D, K, p).bytes;
}

cat_status_t cat_fit_pca(const float *Yq, const float *Yfp, int64_t N, int32_t D, int32_t K, int32_t iters,
                         int32_t p, float *mean_out, float *components_out, float *centroids_out,
                         float *gamma_out, float *beta_out, int32_t *labels_out, void *workspace,
                         size_t workspace_bytes, void *stream)
{
    if (!Yq || !Yfp || !mean_out || !components_out || !centroids_out || !gamma_out || !beta_out) return CAT_ERR_NULL;
    cat_status_t st = pca_shape(N, D, p);
    if (st != CAT_OK) return st;
    if (K < 1 || N < K || iters < 0) return CAT_ERR_SHAPE;
    const size_t need = cat_fit_pca_workspace_bytes(N, D, K, p);
    if (need == 0) return CAT_ERR_UNSUPPORTED;
    if (!workspace || !al16(workspace) || workspace_bytes < need) return CAT_ERR_WORKSPACE;
    FitPcaWs w = carve_fit_pca(workspace, N, D, K, p);
    int32_t *labels = labels_out ? labels_out : w.labels;
    // Algorithm 1 step 1: the projection; step 2: K-Means on the reduced rows
    if ((st = cat_pca_fit(Yq, N, D, p, mean_out, components_out, nullptr, w.pca, w.pca_bytes, stream)) != CAT_OK) return st;
    if ((st = cat_pca_project(Yq, N, D, p, mean_out, components_out, w.Z, stream)) != CAT_OK) return st;
    if ((st = cat_fit(w.Z, w.Z, N, p, K, iters, centroids_out, w.gp, w.bp, labels, w.fit, w.fit_bytes, stream)) != CAT_OK)
        return st;
    // the loop over the clusters: moments and the closed form in the original space
    if ((st = cat_cluster_sums(Yq, labels, N, D, K, w.sumQ, w.counts, w.fit, w.fit_bytes, stream)) != CAT_OK) return st;
    if ((st = cat_cluster_sums(Yfp, labels, N, D, K, w.sumF, w.counts, w.fit, w.fit_bytes, stream)) != CAT_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    CAT_CUDA(launch_means_from_sums(w.sumQ, w.counts, D, K, w.meanQ, s));
    CAT_CUDA(launch_means_from_sums(w.sumF, w.counts, D, K, w.meanF, s));
    if ((st = cat_centred_moments(Yq, Yfp, labels, N, D, K, w.meanQ, w.meanF, w.var, w.cov, w.fit, w.fit_bytes, stream)) !=
        CAT_OK)
        return st;
    return cat_solve_gamma_beta(w.sumQ, w.sumF, w.var, w.cov, w.counts, D, K, gamma_out, beta_out, stream);
}

size_t cat_apply_pca_workspace_bytes(int64_t N, int32_t D, int32_t K, int32_t p)
{
    if (N < 1 || D < 1 || p < 1 || p > D || D > CAT_PCA_MAX_D || p > CAT_PCA_MAX_P) return 0;
    const size_t a = cat_apply_workspace_bytes(N, p, K);
    if (a == 0) return 0;
    return align_up((size_t)N * p * sizeof(float), 256) + align_up((size_t)N * sizeof(int32_t), 256) + a;
}

cat_status_t cat_apply_pca(const float *Yq, int64_t N, int32_t D, int32_t K, int32_t p, const float *mean,
                           const float *components, const float *centroids, const float *gamma,
                           const float *beta, float *Y_out, int32_t *labels_out, void *workspace,
                           size_t workspace_bytes, void *stream)
{
    if (!Yq || !mean || !components || !centroids || !gamma || !beta || !Y_out) return CAT_ERR_NULL;
    const size_t need = cat_apply_pca_workspace_bytes(N, D, K, p);
    if (need == 0) return (N < 1 || D < 1 || p < 1 || p > D || K < 1) ? CAT_ERR_SHAPE : CAT_ERR_UNSUPPORTED;
    if (!workspace || !al16(workspace) || workspace_bytes < need) return CAT_ERR_WORKSPACE;
    unsigned char *b = reinterpret_cast<unsigned char *>(workspace);
    float *Z = reinterpret_cast<float *>(b);
    size_t off = align_up((size_t)N * p * sizeof(float), 256);
    int32_t *labels = labels_out ? labels_out : reinterpret_cast<int32_t *>(b + off);
    off += align_up((size_t)N * sizeof(int32_t), 256);
    cat_status_t st;
    // Algorithm 2 step 1: project; step 2: predict the cluster; steps 4-8: correct in the original space
    if ((st = cat_pca_project(Yq, N, D, p, mean, components, Z, stream)) != CAT_OK) return st;
    if ((st = cat_assign(Z, N, p, K, centroids, labels, b + off, workspace_bytes - off, stream)) != CAT_OK) return st;
    return cat_affine_with_labels(Yq, N, D, K, labels, gamma, beta, Y_out, stream);
}

}  // extern "C"
