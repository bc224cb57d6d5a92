// Segmented (per-cluster) sums through a stable sort of the rows by label.
//
//   label_hist_kernel     per-block key histograms (1024 entries per block)
//   label_scan_blocks_kernel  per-block offsets and key totals
//                         (key offsets, segment table and cluster sizes: scan_keys, inside the scatter kernel)
//   label_scatter_kernel  stable scatter of the row indices: order[] lists the rows of
//                         key 0 in ascending row order, then key 1, ...
//
// Two modes.  Full: every row is an entry with key = its label (K keys).  Delta (the Lloyd
// rounds of cat_fit): only rows whose label differs from the previous round's are entries,
// each twice -- under key `new label` (its values enter that cluster's sum) and under key
// K + `old label` (they leave that one) -- so 2K keys over 2N virtual entries, nearly all of
// them empty once the clustering settles.  The running sums S_k += sum(in) - sum(out) are the
// same per-cluster sums up to fp64 rounding, at the cost of the rows that moved.
//   segment_sums_kernel   one CTA per segment (<= seg_rows consecutive entries of order[], all of
//                         one cluster): streams those rows with 128-bit loads and keeps the
//                         column sums in fp64 registers -- no atomics, no shared accumulators,
//                         fixed summation order -- and writes one partial row per segment
//   segment_combine_kernel  adds a cluster's segment partials in order; optionally turns the
//                         sums into centroids
//
// Three reductions use the same machinery: column sums of one matrix (a Lloyd round), of
// two matrices (the final pass: sums of Yq and Yfp), and the centred second moments
// sum (q - muQ)^2, sum (q - muQ)(f - muF) with the cluster means held in registers.
#include "cat_internal.cuh"

#include <cuda_fp16.h>

namespace cat {

namespace {

constexpr int SORT_BLOCK = 1024;     // rows per histogram / scatter block
constexpr int SEG_THREADS = 256;

// Key of virtual entry e: entries [0, N) are the rows under their current label; in delta
// mode (prev != NULL) a row whose label did not change has no entry, and entries [N, 2N)
// are the changed rows under K + previous label.  -1 = no entry.
__device__ __forceinline__ int entry_key(const int32_t *__restrict__ cur, const int32_t *__restrict__ prev,
                                         int64_t N, int K, int64_t e)
{
    if (e < N) {
        const int l = cur[e];
        if (l < 0 || l >= K) return -1;
        if (prev && prev[e] == l) return -1;
        return l;
    }
    if (!prev || e >= 2 * N) return -1;
    const int64_t r = e - N;
    const int o = prev[r];
    if (o < 0 || o >= K || o == cur[r]) return -1;
    return K + o;
}

__global__ void __launch_bounds__(SORT_BLOCK) label_hist_kernel(const int32_t *__restrict__ cur,
                                                                 const int32_t *__restrict__ prev, int64_t N, int K,
                                                                 int KK, uint32_t *__restrict__ blk_hist)
{
    pdl_enter();
    extern __shared__ uint32_t hist[];   // [KK]
    for (int k = threadIdx.x; k < KK; k += SORT_BLOCK) hist[k] = 0;
    __syncthreads();
    const int64_t e = (int64_t)blockIdx.x * SORT_BLOCK + threadIdx.x;
    const int l = entry_key(cur, prev, N, K, e);
    if (l >= 0) atomicAdd(&hist[l], 1u);
    __syncthreads();
    for (int k = threadIdx.x; k < KK; k += SORT_BLOCK) blk_hist[(size_t)k * gridDim.x + blockIdx.x] = hist[k];   // [key][block]
}

// One warp per key: blk_hist[k][b] becomes the number of entries of key k in blocks before
// b, key_total[k] their total.
__global__ void __launch_bounds__(256) label_scan_blocks_kernel(uint32_t *__restrict__ blk_hist, int nblk, int KK,
                                                                 uint32_t *__restrict__ key_total)
{
    pdl_enter();
    const int k = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (k >= KK) return;
    uint32_t carry = 0;
    for (int b0 = 0; b0 < nblk; b0 += 32) {
        const int b = b0 + lane;
        const uint32_t v = (b < nblk) ? blk_hist[(size_t)k * nblk + b] : 0u;
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (b < nblk) blk_hist[(size_t)k * nblk + b] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) key_total[k] = carry;
}

// Exclusive scan over the 1024 threads of the CTA (one value per thread); returns the exclusive
// prefix of the calling thread and, through `total`, the sum of all values.
__device__ __forceinline__ uint32_t cta_exclusive_scan(uint32_t v, uint32_t *wsum /*[33] shared*/, uint32_t &total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();   // wsum may still be read from an earlier scan
    if (lane == 31) wsum[w] = incl;
    __syncthreads();
    if (w == 0) {
        const uint32_t a = wsum[lane];
        uint32_t x = a;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += t;
        }
        wsum[lane] = x - a;   // exclusive
        if (lane == 31) wsum[32] = x;
    }
    __syncthreads();
    total = wsum[32];
    return wsum[w] + incl - v;
}

// One CTA of 1024 threads (KK <= 1024): exclusive scan of the key totals (cluster_start, KK + 1
// entries), the segment length for this sort, the exclusive scan of the segment counts
// ceil(total / length) (seg_start, KK + 1 entries, followed by the length itself), and the cluster
// sizes: full mode counts[k] = total[k]; delta mode counts[k] += total[k] - total[K + k].
// The segment length shrinks with the number of entries M actually present (a delta sort of a
// settled clustering holds a handful): length = seg_rows_max * M / NE rounded up to 16, at least 16,
// so that short lists still spread over many CTAs and the segment count stays within
// NE / seg_rows_max + KK.
// Runs in every CTA of the scatter kernel (each needs the key offsets for its own entries); the CTA
// with `publish` set also writes the tables and updates the cluster sizes.  Returns this thread's
// key offset (thread k < KK).
__device__ __forceinline__ uint32_t scan_keys(const uint32_t *__restrict__ key_total, int K, int KK, int seg_rows_max,
                                              int64_t NE, int delta, bool publish, int64_t *__restrict__ counts,
                                              int32_t *__restrict__ cluster_start, int32_t *__restrict__ seg_start,
                                              uint32_t *wsum /*[33] shared*/)
{
    const int k = threadIdx.x;
    const uint32_t tot = (k < KK) ? key_total[k] : 0u;
    uint32_t M = 0;
    const uint32_t ea = cta_exclusive_scan(tot, wsum, M);
    if (!publish) return ea;
    int64_t sr = ((int64_t)seg_rows_max * (int64_t)M + NE - 1) / NE;
    sr = (sr + 15) / 16 * 16;
    if (sr < 16) sr = 16;
    if (sr > seg_rows_max) sr = seg_rows_max;
    const uint32_t sg = (tot + (uint32_t)sr - 1) / (uint32_t)sr;
    uint32_t nseg = 0;
    const uint32_t es = cta_exclusive_scan(sg, wsum, nseg);
    if (k < KK) {
        cluster_start[k] = (int32_t)ea;
        seg_start[k] = (int32_t)es;
    }
    if (k == 0) {
        cluster_start[KK] = (int32_t)M;
        seg_start[KK] = (int32_t)nseg;
        seg_start[KK + 1] = (int32_t)sr;
    }
    if (k < K) {
        if (delta) counts[k] += (int64_t)tot - (int64_t)key_total[K + k];
        else counts[k] = (int64_t)tot;
    }
    return ea;
}

// Stable scatter.  Within a block, an entry's rank among the entries of its key is
// (entries of that key in earlier warps) + (entries of that key in earlier lanes).
__global__ void __launch_bounds__(SORT_BLOCK) label_scatter_kernel(const int32_t *__restrict__ cur,
                                                                    const int32_t *__restrict__ prev, int64_t N, int K,
                                                                    int KK, const uint32_t *__restrict__ blk_hist,
                                                                    const uint32_t *__restrict__ key_total,
                                                                    int seg_rows_max, int64_t NE, int delta,
                                                                    int64_t *__restrict__ counts,
                                                                    int32_t *__restrict__ cluster_start,
                                                                    int32_t *__restrict__ seg_start,
                                                                    int32_t *__restrict__ order)
{
    pdl_enter();
    extern __shared__ uint32_t scatter_smem[];   // [KK] key offsets, then [32][KK] 16-bit warp histograms
    __shared__ uint32_t wsum[33];
    uint32_t *key_off = scatter_smem;
    uint16_t *warp_hist = reinterpret_cast<uint16_t *>(scatter_smem + KK);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    for (int e = tid; e < 32 * KK; e += SORT_BLOCK) warp_hist[e] = 0;
    {
        const uint32_t ea = scan_keys(key_total, K, KK, seg_rows_max, NE, delta, blockIdx.x == 0, counts, cluster_start,
                                      seg_start, wsum);
        if (tid < KK) key_off[tid] = ea;
    }
    __syncthreads();
    const int64_t e = (int64_t)blockIdx.x * SORT_BLOCK + tid;
    const int l = entry_key(cur, prev, N, K, e);
    const unsigned peers = __match_any_sync(0xffffffffu, l);
    const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
    if (l >= 0 && rank_in_warp == 0) warp_hist[w * KK + l] = (uint16_t)__popc(peers);
    __syncthreads();
    for (int k = tid; k < KK; k += SORT_BLOCK) {
        uint16_t run = 0;
        for (int q = 0; q < 32; ++q) {
            const uint16_t v = warp_hist[q * KK + k];
            warp_hist[q * KK + k] = run;
            run = (uint16_t)(run + v);
        }
    }
    __syncthreads();
    if (l >= 0) {
        const uint32_t pos = key_off[l] + blk_hist[(size_t)l * gridDim.x + blockIdx.x] +
                             warp_hist[w * KK + l] + (uint32_t)rank_in_warp;
        order[pos] = (int32_t)(e < N ? e : e - N);
    }
}

struct SegParams {
    const float *Yq;
    const float *Yf;            // second matrix (modes 1, 2)
    const int32_t *order;
    const int32_t *cluster_start;
    const int32_t *seg_start;
    const double *meanQ;        // mode 2
    const double *meanF;
    double *part;               // [maxsegs][2][D]
    int D;
    int K;
    int seg_rows;
    int tpr;                    // threads per row (power of two <= 256)
};

__device__ __forceinline__ void add4(double (&a)[4], const float4 v)
{
    a[0] += (double)v.x;
    a[1] += (double)v.y;
    a[2] += (double)v.z;
    a[3] += (double)v.w;
}

// One row's contribution (VEC columns) to the accumulators of a segment.
template <int MODE, int VEC>
__device__ __forceinline__ void seg_accumulate(double (&a0)[4], double (&a1)[4], double (&a2)[4], const double (&mq)[4],
                                               const double (&mf)[4], const float4 q4, const float4 f4)
{
    if (MODE == 0) {
        add4(a0, q4);
    } else if (MODE == 1) {
        add4(a0, q4);
        add4(a1, f4);
    } else {
        const float qv[4] = {q4.x, q4.y, q4.z, q4.w};
        const float fv[4] = {f4.x, f4.y, f4.z, f4.w};
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
            const double dq = (double)qv[q] - mq[q];
            const double df = (double)fv[q] - mf[q];
            a0[q] = fma(dq, dq, a0[q]);
            a1[q] = fma(dq, df, a1[q]);
            if (MODE == 3) a2[q] += (double)fv[q];
        }
    }
}

// MODE 0: sums of Yq -> plane 0.  MODE 1: sums of Yq, Yf -> planes 0, 1.
// MODE 2: centred moments -> plane 0 = sum (q-muQ)^2, plane 1 = sum (q-muQ)(f-muF).
// MODE 3: the final pass of cat_fit in one sweep, with the cluster mean muQ known beforehand:
//         plane 0 = sum (q-muQ)^2, plane 1 = sum (q-muQ)(f-muQ), plane 2 = sum f (three planes
//         per segment).  Since sum (q-muQ) = 0, plane 1 is the centred cross moment whatever
//         constant is subtracted from f; muQ keeps the products small.
// VEC: 4 = 128-bit loads (D % 4 == 0), 1 = scalar loads.
template <int MODE, int VEC>
__global__ void __launch_bounds__(SEG_THREADS) segment_sums_kernel(SegParams p)
{
    pdl_enter();
    __shared__ int32_t rows_s[128];
    __shared__ double red_s[SEG_THREADS * VEC];
    const int nseg_total = p.seg_start[p.K];
    for (int seg = blockIdx.x; seg < nseg_total; seg += gridDim.x) {
    // cluster of this segment: last k with seg_start[k] <= seg
    int lo = 0, hi = p.K;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (p.seg_start[mid] <= seg) lo = mid; else hi = mid;
    }
    const int k = lo;
    const int seg_rows = p.seg_start[p.K + 1];   // length chosen by the sort for this list
    const int first = p.cluster_start[k] + (seg - p.seg_start[k]) * seg_rows;
    int nrows = p.cluster_start[k + 1] - first;
    if (nrows > seg_rows) nrows = seg_rows;

    const int tid = threadIdx.x;
    const int tpr = p.tpr;
    const int c = tid & (tpr - 1);      // column unit within the block of columns
    const int g = tid / tpr;            // row group
    const int G = SEG_THREADS / tpr;
    const int units = (p.D + VEC - 1) / VEC;          // column units per row
    const int col0 = blockIdx.y * SEG_THREADS;        // first unit of this column block
    const int unit = col0 + c;
    const bool active = (c < SEG_THREADS) && (unit < units);
    const int col = unit * VEC;

    double a0[4] = {0, 0, 0, 0}, a1[4] = {0, 0, 0, 0}, a2[4] = {0, 0, 0, 0};
    double mq[4] = {0, 0, 0, 0}, mf[4] = {0, 0, 0, 0};
    if (MODE >= 2 && active) {
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
            mq[q] = p.meanQ[(size_t)k * p.D + col + q];
            mf[q] = (MODE == 2) ? p.meanF[(size_t)k * p.D + col + q] : mq[q];
        }
    }

    for (int base = 0; base < nrows; base += 128) {
        const int nb = (nrows - base < 128) ? (nrows - base) : 128;
        __syncthreads();
        if (tid < nb) rows_s[tid] = p.order[first + base + tid];
        __syncthreads();
        if (!active) continue;
        int r = g;
        // four rows in flight per thread
        for (; r + 3 * G < nb; r += 4 * G) {
            float4 q4[4], f4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const size_t o = (size_t)rows_s[r + u * G] * p.D + col;
                if (VEC == 4) {
                    q4[u] = __ldg(reinterpret_cast<const float4 *>(p.Yq + o));
                    if (MODE != 0) f4[u] = __ldg(reinterpret_cast<const float4 *>(p.Yf + o));
                } else {
                    q4[u] = make_float4(__ldg(p.Yq + o), 0.f, 0.f, 0.f);
                    if (MODE != 0) f4[u] = make_float4(__ldg(p.Yf + o), 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) seg_accumulate<MODE, VEC>(a0, a1, a2, mq, mf, q4[u], f4[u]);
        }
        for (; r < nb; r += G) {
            const size_t o = (size_t)rows_s[r] * p.D + col;
            float4 q4, f4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (VEC == 4) {
                q4 = __ldg(reinterpret_cast<const float4 *>(p.Yq + o));
                if (MODE != 0) f4 = __ldg(reinterpret_cast<const float4 *>(p.Yf + o));
            } else {
                q4 = make_float4(__ldg(p.Yq + o), 0.f, 0.f, 0.f);
                if (MODE != 0) f4 = make_float4(__ldg(p.Yf + o), 0.f, 0.f, 0.f);
            }
            seg_accumulate<MODE, VEC>(a0, a1, a2, mq, mf, q4, f4);
        }
    }

    // add the row groups in a fixed order and publish the segment's partial row
    constexpr int NPLANES = (MODE == 0) ? 1 : (MODE == 3 ? 3 : 2);
    constexpr int PSTRIDE = (MODE == 3) ? 3 : 2;   // planes per segment in `part`
#pragma unroll
    for (int pl = 0; pl < NPLANES; ++pl) {
        __syncthreads();
#pragma unroll
        for (int q = 0; q < VEC; ++q) red_s[tid * VEC + q] = (pl == 0) ? a0[q] : (pl == 1 ? a1[q] : a2[q]);
        __syncthreads();
        if (g == 0 && active) {
            double *dst = p.part + ((size_t)seg * PSTRIDE + pl) * p.D + col;
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
                double s = 0.0;
                for (int gg = 0; gg < G; ++gg) s += red_s[(gg * tpr + c) * VEC + q];
                dst[q] = s;
            }
        }
    }
    __syncthreads();   // red_s and rows_s are reused by the next segment
    }
}

// out0/out1[k*D+j] = sum over the segments of key k of plane 0/1 (out1 may be NULL); in
// delta mode out0[k*D+j] += (segments of key k) - (segments of key K + k).  With C != NULL
// also C[k*D+j] = float(out0 / n_k) where n_k > 0.
__global__ void segment_combine_kernel(const double *__restrict__ part, const int32_t *__restrict__ seg_start,
                                       const int64_t *__restrict__ counts, int D, int K, size_t KD, int delta,
                                       double *__restrict__ out0, double *__restrict__ out1,
                                       float *__restrict__ C)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    const int k = (int)(e / D);
    const int j = (int)(e - (size_t)k * D);
    const int s0 = seg_start[k], s1 = seg_start[k + 1];
    double a = 0.0, b = 0.0;
    for (int sgm = s0; sgm < s1; ++sgm) {
        a += part[((size_t)sgm * 2) * D + j];
        if (out1) b += part[((size_t)sgm * 2 + 1) * D + j];
    }
    if (delta) {
        double m = 0.0;
        for (int sgm = seg_start[K + k]; sgm < seg_start[K + k + 1]; ++sgm) m += part[((size_t)sgm * 2) * D + j];
        a = out0[e] + (a - m);
    }
    out0[e] = a;
    if (out1) out1[e] = b;
    if (C) {
        const int64_t n = counts[k];
        if (n > 0) C[e] = (float)(a / (double)n);
    }
}

// Three-plane partials (MODE 3) added up per cluster.
__global__ void segment_combine3_kernel(const double *__restrict__ part, const int32_t *__restrict__ seg_start, int D,
                                        size_t KD, double *__restrict__ out0, double *__restrict__ out1,
                                        double *__restrict__ out2)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= KD) return;
    const int k = (int)(e / D);
    const int j = (int)(e - (size_t)k * D);
    double a = 0.0, b = 0.0, c = 0.0;
    for (int sgm = seg_start[k]; sgm < seg_start[k + 1]; ++sgm) {
        a += part[((size_t)sgm * 3) * D + j];
        b += part[((size_t)sgm * 3 + 1) * D + j];
        c += part[((size_t)sgm * 3 + 2) * D + j];
    }
    out0[e] = a;
    out1[e] = b;
    out2[e] = c;
}

// Delta-mode centroid update, one CTA per cluster: S_k += (partials of key k) - (partials of key
// K + k); c_k = float(S_k / n_k) where n_k > 0; and for the next assignment the squared norm
// of c_k (fp64, rounded up), optionally the fp16 copy fp16(c_k * scale[0]), and the reset of the
// exact-pass queues.
__global__ void __launch_bounds__(1024) centroid_update_kernel(const double *__restrict__ part,
                                                              const int32_t *__restrict__ seg_start,
                                                              const int64_t *__restrict__ counts, int D, int K,
                                                              double *__restrict__ sums, float *__restrict__ C,
                                                              float *__restrict__ cnorm, const float *__restrict__ scale,
                                                              __half *__restrict__ Ch, Control *ctl)
{
    pdl_enter();
    __shared__ double red[32];
    const int k = blockIdx.x;
    if (k == 0 && threadIdx.x == 0) {
        ctl->refine_count = 0;
        ctl->cand_count = 0;
    }
    const int a0 = seg_start[k], a1 = seg_start[k + 1], m0 = seg_start[K + k], m1 = seg_start[K + k + 1];
    const int64_t n = counts[k];
    const float sc = Ch ? scale[0] : 1.f;
    double nrm = 0.0;
    for (int j = threadIdx.x; j < D; j += blockDim.x) {
        const size_t e = (size_t)k * D + j;
        double a = 0.0, m = 0.0;
        for (int sgm = a0; sgm < a1; ++sgm) a += part[((size_t)sgm * 2) * D + j];
        for (int sgm = m0; sgm < m1; ++sgm) m += part[((size_t)sgm * 2) * D + j];
        const double sum = sums[e] + (a - m);
        sums[e] = sum;
        float c = C[e];
        if (n > 0) {
            c = (float)(sum / (double)n);
            C[e] = c;
        }
        nrm += (double)c * (double)c;
        if (Ch) Ch[e] = __float2half_rn(c * sc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = nrm;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
        cnorm[k] = __double2float_ru(t);
    }
}

int tpr_for(int units)
{
    int t = 1;
    while (t < units && t < SEG_THREADS) t <<= 1;
    return t;
}

}  // namespace

// Geometry for NE virtual entries over KK keys.
SegGeom seg_geometry(int64_t NE, int D, int KK)
{
    SegGeom g{};
    g.nblk = (int)((NE + SORT_BLOCK - 1) / SORT_BLOCK);
    int64_t sr = (NE + 2047) / 2048;
    if (sr < 128) sr = 128;
    sr = (sr + 127) / 128 * 128;
    g.seg_rows = (int)sr;
    g.max_segs = (int)((NE + sr - 1) / sr) + KK;
    (void)D;
    return g;
}

cudaError_t launch_label_sort(const int32_t *labels, const int32_t *prev, int64_t N, int K, const SegGeom &g,
                              uint32_t *blk_hist, uint32_t *key_total, int64_t *counts, int32_t *cluster_start,
                              int32_t *seg_start, int32_t *order, cudaStream_t s)
{
    const int KK = prev ? 2 * K : K;
    launch_pdl(label_hist_kernel, dim3(g.nblk), dim3(SORT_BLOCK), (size_t)KK * sizeof(uint32_t), s, labels, prev, N, K, KK, blk_hist);
    launch_pdl(label_scan_blocks_kernel, dim3((KK * 32 + 255) / 256), dim3(256), 0, s, blk_hist, g.nblk, KK, key_total);
    // (the scan over the keys -- key offsets, segment table, cluster sizes -- runs inside the scatter
    // kernel: every CTA needs the offsets, CTA 0 publishes the tables)
    const size_t sc_smem = (size_t)KK * sizeof(uint32_t) + (size_t)32 * KK * sizeof(uint16_t);
    if (sc_smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(label_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)sc_smem);
        if (e != cudaSuccess) return e;
    }
    launch_pdl(label_scatter_kernel, dim3(g.nblk), dim3(SORT_BLOCK), sc_smem, s, labels, prev, N, K, KK, blk_hist, key_total,
               g.seg_rows, prev ? 2 * N : N, prev ? 1 : 0, counts, cluster_start, seg_start, order);
    count_launch(3);
    return cudaGetLastError();
}

template <int MODE>
static cudaError_t launch_segment_sums_mode(const SegParams &p, const SegGeom &g, cudaStream_t s)
{
    const bool vec = (p.D % 4 == 0);
    const int units = vec ? p.D / 4 : p.D;
    // a CTA walks segments blockIdx.x, blockIdx.x + gridDim.x, ...: in delta mode most of the
    // max_segs slots are empty, so the grid stays at a few CTAs per SM
    const unsigned gx = (unsigned)(g.max_segs < 1184 ? g.max_segs : 1184);
    dim3 grid(gx, (unsigned)((units + SEG_THREADS - 1) / SEG_THREADS));
    if (vec)
        launch_pdl(segment_sums_kernel<MODE, 4>, grid, dim3(SEG_THREADS), 0, s, p);
    else
        launch_pdl(segment_sums_kernel<MODE, 1>, grid, dim3(SEG_THREADS), 0, s, p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_segment_sums(int mode, const float *Yq, const float *Yf, const int32_t *order,
                                const int32_t *cluster_start, const int32_t *seg_start, const double *meanQ,
                                const double *meanF, int D, int K, const SegGeom &g, double *part,
                                cudaStream_t s)
{
    SegParams p{};
    p.Yq = Yq;
    p.Yf = Yf;
    p.order = order;
    p.cluster_start = cluster_start;
    p.seg_start = seg_start;
    p.meanQ = meanQ;
    p.meanF = meanF;
    p.part = part;
    p.D = D;
    p.K = K;
    p.seg_rows = g.seg_rows;
    const int units = (D % 4 == 0) ? D / 4 : D;
    p.tpr = tpr_for(units);
    switch (mode) {
    case 0: return launch_segment_sums_mode<0>(p, g, s);
    case 1: return launch_segment_sums_mode<1>(p, g, s);
    case 2: return launch_segment_sums_mode<2>(p, g, s);
    default: return launch_segment_sums_mode<3>(p, g, s);
    }
}

cudaError_t launch_segment_combine(const double *part, const int32_t *seg_start, const int64_t *counts, int D,
                                   int K, bool delta, double *out0, double *out1, float *C, cudaStream_t s)
{
    const size_t KD = (size_t)K * D;
    const int threads = 256;
    const unsigned blocks = (unsigned)((KD + threads - 1) / threads);
    segment_combine_kernel<<<blocks, threads, 0, s>>>(part, seg_start, counts, D, K, KD, delta ? 1 : 0, out0, out1, C);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_segment_combine3(const double *part, const int32_t *seg_start, int D, int K, double *out0,
                                    double *out1, double *out2, cudaStream_t s)
{
    const size_t KD = (size_t)K * D;
    const int threads = 256;
    const unsigned blocks = (unsigned)((KD + threads - 1) / threads);
    segment_combine3_kernel<<<blocks, threads, 0, s>>>(part, seg_start, D, KD, out0, out1, out2);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_centroid_update(const double *part, const int32_t *seg_start, const int64_t *counts, int D,
                                   int K, double *sums, float *C, float *cnorm, const float *scale, void *Ch,
                                   Control *ctl, cudaStream_t s)
{
    // one thread per column where the row is short enough: the loads of a column depend on each other
    const int threads = D >= 1024 ? 1024 : (D >= 512 ? 512 : 256);
    launch_pdl(centroid_update_kernel, dim3(K), dim3(threads), 0, s, part, seg_start, counts, D, K, sums, C, cnorm, scale,
               reinterpret_cast<__half *>(Ch), ctl);
    count_launch();
    return cudaGetLastError();
}

}  // namespace cat
