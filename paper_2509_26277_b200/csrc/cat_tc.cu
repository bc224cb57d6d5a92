// Tensor-core path of the nearest-centroid assignment (sm_100a: tcgen05 + TMEM + TMA).
//
// The N x K x D distance contraction y_i . c_k runs as a TF32 UMMA: a persistent CTA
// walks 128-row tiles; TMA streams 128 x 32 fp32 slabs of the rows and K x 32 slabs of
// the centroids into 128-byte-swizzled shared memory, one thread issues
// tcgen05.mma.kind::tf32 into a TMEM accumulator (128 lanes x K columns, two buffers),
// and the epilogue warps read the scores back with tcgen05.ld, take best / second /
// argmin per row and run the same certainty test as the fp32 path, with the TF32 error
// bound
//     e <= (2^-8 + (2D+2) 2^-22) ||y|| cmax + 4 u cmax^2
// (operands cut to 11 significant bits: <= 2^-10 each; fp32 accumulation inside the
// tensor core taken as <= 2^-22 per term).  Rows it cannot decide go to the same exact
// fp64 pass, so labels stay exact.  For inference the epilogue then streams each decided
// row once more (it is still in L2) and writes gamma_l * y + beta_l.
//
// Every wait on an mbarrier is bounded (about 2 s): on a timeout the CTA records
// CAT_ERR_DEVICE_TIMEOUT in the control block, all roles leave their loops, outstanding
// copies and MMAs are drained with bounded waits, TMEM is freed and the kernel returns.
#include "cat_internal.cuh"

#include <cuda.h>
#include <math_constants.h>

namespace cat {

namespace {

constexpr int TC_BM = 128;                   // rows per tile (UMMA M)
constexpr int TC_BK = 32;                    // fp32 per slab = 128 B = one swizzle row
constexpr int TC_A_BYTES = TC_BM * TC_BK * 4;  // 16 KB
constexpr int TC_STAGES = 4;
constexpr int TC_SCORE_WARPS = 4;
constexpr int TC_STREAM_WARPS = 12;          // AFFINE only; includes the 4 score warps
constexpr uint64_t TC_TIMEOUT_NS = 2000000000ull;

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false after a timeout or once another role has given up.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((it & 63u) == 63u) {
            uint64_t now = global_timer();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > TC_TIMEOUT_NS) {
                *abort_flag = 1;
                atomicExch(&ctl->device_status, (int)CAT_ERR_DEVICE_TIMEOUT);
                return false;
            }
        }
    }
}

// Warp-uniform form: every lane waits; the warp proceeds only if all lanes succeeded.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl)
{
    bool ok = mbar_wait(bar, parity, abort_flag, ctl);
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// K-major, 128-byte-swizzled operand tile whose rows are 128 B apart: 8-row groups every
// 1024 B (stride byte offset), leading byte offset unused (1), descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// D = F32, A = B = TF32, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t make_idesc_tf32(int n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

struct TcParams {
    const float *Y;
    const float *cnorm;
    const float *ynorm2;   // [N] squared row norms (labels-only mode)
    int32_t *labels;
    int32_t *refine_rows;
    int32_t *cand_rows;    // rows whose exact decision only needs the listed candidates
    uint64_t *cand_list;   // four 16-bit centroid indices per entry (0xFFFF = unused)
    Control *ctl;
    const float *gamma;
    const float *beta;
    float *out;
    int64_t N;
    int D;
    int K;
    int npad;       // K rounded up to 16
    int tmem_cols;  // power of two >= 2 * npad, >= 32
};

struct TcShared {
    uint64_t full[TC_STAGES];
    uint64_t empty[TC_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t lab_full[2];
    uint64_t lab_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    float red[16];
    float cn[256];
    float4 top_score[2][TC_BM];   // four smallest scores of each row, ascending
    int4 top_idx[2][TC_BM];       // their centroid indices
};

__device__ __forceinline__ float tc_error_bound(int D, float ysq, float cmax2)
{
    const float u = 5.9604645e-8f;   // 2^-24
    const float a = 3.90625e-3f + (2.f * (float)D + 2.f) * 2.3841858e-7f;  // 2^-8 + (2D+2) 2^-22
    return 1.0625f * (a * sqrtf(ysq) * sqrtf(cmax2) + 4.f * u * cmax2);
}

// Decision for one row from its four smallest scores.  Returns true when the fast argmin is
// certainly exact.  Otherwise the row is queued: with the centroids whose score lies within
// 2e of the best when those are known to be among the four, else for a scan of all K.
__device__ __forceinline__ bool tc_decide(const TcParams &p, int64_t row, float4 sc, int4 id, float e)
{
    const float lim = 2.f * e;
    if (p.K == 1 || (sc.y - sc.x) > lim) return true;
    const bool more = !((sc.w - sc.x) > lim);   // the 4th is a candidate too (or NaN): others may be
    if (more && p.K > 4) {
        int slot = atomicAdd(&p.ctl->refine_count, 1);
        p.refine_rows[slot] = (int32_t)row;
    } else {
        uint64_t c = (uint64_t)(uint16_t)id.x | ((uint64_t)(uint16_t)id.y << 16);
        c |= (uint64_t)(((sc.z - sc.x) > lim || p.K < 3) ? 0xFFFFu : (uint16_t)id.z) << 32;
        c |= (uint64_t)(((sc.w - sc.x) > lim || p.K < 4) ? 0xFFFFu : (uint16_t)id.w) << 48;
        int slot = atomicAdd(&p.ctl->cand_count, 1);
        p.cand_rows[slot] = (int32_t)row;
        p.cand_list[slot] = c;
    }
    return false;
}

template <bool AFFINE>
__global__ void __launch_bounds__(AFFINE ? 32 * (2 + TC_STREAM_WARPS) : 32 * (2 + TC_SCORE_WARPS), 1)
assign_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcParams p)
{
    constexpr int NEPI = AFFINE ? TC_STREAM_WARPS : TC_SCORE_WARPS;
    extern __shared__ unsigned char smem_raw[];
    // operand tiles need 1024-byte alignment for the 128-byte swizzle
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char *tiles = smem_raw + (tiles_base - raw);
    const int b_bytes = p.npad * 128;
    const int stage_bytes = TC_A_BYTES + b_bytes;
    TcShared &sh = *reinterpret_cast<TcShared *>(tiles + (size_t)TC_STAGES * stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *abort_flag = &sh.abort_flag;
    const int64_t num_tiles = (p.N + TC_BM - 1) / TC_BM;
    const int nslabs = (p.D + TC_BK - 1) / TC_BK;

    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh.tmem_full[b]), 1);
            mbar_init(smem_u32(&sh.tmem_empty[b]), TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.lab_full[b]), TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.lab_empty[b]), NEPI);
        }
        mbar_init(smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // centroid norms (+inf beyond K) and their maximum
    {
        float m = 0.f;
        for (int k = tid; k < 256; k += blockDim.x) {
            float v = (k < p.K) ? p.cnorm[k] : CUDART_INF_F;
            sh.cn[k] = v;
            if (k < p.K) m = fmaxf(m, v);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) sh.red[warp] = m;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    float cmax2 = 0.f;
    for (int w2 = 0; w2 < (int)(blockDim.x >> 5); ++w2) cmax2 = fmaxf(cmax2, sh.red[w2]);
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                for (int sl = 0; sl < nslabs; ++sl, ++it) {
                    const int s = it % TC_STAGES;
                    const uint32_t ph = (it / TC_STAGES) & 1u;
                    if (!mbar_wait(smem_u32(&sh.empty[s]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                    const uint32_t full = smem_u32(&sh.full[s]);
                    mbar_arrive_expect_tx(full, (uint32_t)stage_bytes);
                    const uint32_t a_dst = tiles_base + (uint32_t)(s * stage_bytes);
                    tma_load_2d(a_dst, &mapA, full, sl * TC_BK, (int)(tile * TC_BM));
                    tma_load_2d(a_dst + TC_A_BYTES, &mapB, full, sl * TC_BK, 0);
                }
            }
            if (!ok) {
                // give copies that are still in flight a bounded time to land
                for (int s = 0; s < TC_STAGES; ++s)
                    for (int tries = 0; tries < 100000; ++tries)
                        if (mbar_try_wait(smem_u32(&sh.full[s]), 0) || mbar_try_wait(smem_u32(&sh.full[s]), 1)) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_tf32(p.npad);
            uint32_t it = 0, ti = 0;
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++ti) {
                const int b = ti & 1;
                if (!mbar_wait(smem_u32(&sh.tmem_empty[b]), ((ti >> 1) & 1u) ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(b * p.npad);
                for (int sl = 0; sl < nslabs; ++sl, ++it) {
                    const int s = it % TC_STAGES;
                    if (!mbar_wait(smem_u32(&sh.full[s]), (it / TC_STAGES) & 1u, abort_flag, p.ctl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tiles_base + (uint32_t)(s * stage_bytes);
                    const uint64_t adesc = make_smem_desc(a_addr);
                    const uint64_t bdesc = make_smem_desc(a_addr + TC_A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < TC_BK / 8; ++kk)   // 8 tf32 = 32 B per MMA: +2 in 16-byte units
                        mma_tf32(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, (sl > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&sh.empty[s]));
                }
                if (ok) tc_commit(smem_u32(&sh.tmem_full[b]));
            }
            // all MMAs issued by this thread have completed once this commit arrives
            tc_commit(smem_u32(&sh.drain));
            for (int tries = 0; tries < 4000000; ++tries)
                if (mbar_try_wait(smem_u32(&sh.drain), 0)) break;
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int ew = warp - 2;                  // 0 .. NEPI-1
        const bool scorer = ew < TC_SCORE_WARPS;
        const int quarter = warp & 3;             // TMEM lanes this warp may read
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            const int64_t row0 = tile * TC_BM;
            if (scorer) {
                if (!mbar_wait_warp(smem_u32(&sh.tmem_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
                tc_fence_after();
                float b1 = CUDART_INF_F, b2 = CUDART_INF_F, b3 = CUDART_INF_F, b4 = CUDART_INF_F;
                int i1 = 0, i2 = 0, i3 = 0, i4 = 0;
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * p.npad);
                for (int c = 0; c < p.npad; c += 16) {
                    float v[16];
                    tmem_ld16(taddr + (uint32_t)c, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float sc = fmaf(-2.f, v[j], sh.cn[c + j]);
                        if (sc < b4) {
                            const int n = c + j;
                            if (sc < b3) {
                                b4 = b3; i4 = i3;
                                if (sc < b2) {
                                    b3 = b2; i3 = i2;
                                    if (sc < b1) { b2 = b1; i2 = i1; b1 = sc; i1 = n; }
                                    else { b2 = sc; i2 = n; }
                                } else { b3 = sc; i3 = n; }
                            } else { b4 = sc; i4 = n; }
                        }
                    }
                }
                // accumulator buffer b may be overwritten from here on
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.tmem_empty[b]));
                const int r = quarter * 32 + lane;
                if (AFFINE) {
                    if (!mbar_wait_warp(smem_u32(&sh.lab_empty[b]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                    sh.top_score[b][r] = make_float4(b1, b2, b3, b4);
                    sh.top_idx[b][r] = make_int4(i1, i2, i3, i4);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh.lab_full[b]));
                } else {
                    const int64_t row = row0 + r;
                    if (row < p.N) {
                        const float e = tc_error_bound(p.D, p.ynorm2[row], cmax2);
                        p.labels[row] = i1;
                        tc_decide(p, row, make_float4(b1, b2, b3, b4), make_int4(i1, i2, i3, i4), e);
                    }
                }
            }
            if (AFFINE) {
                if (!mbar_wait_warp(smem_u32(&sh.lab_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
                const int D4 = p.D >> 2;
                const float4 *Y4 = reinterpret_cast<const float4 *>(p.Y);
                const float4 *G4 = reinterpret_cast<const float4 *>(p.gamma);
                const float4 *B4 = reinterpret_cast<const float4 *>(p.beta);
                float4 *O4 = reinterpret_cast<float4 *>(p.out);
                for (int r = ew; r < TC_BM; r += NEPI) {
                    const int64_t row = row0 + r;
                    if (row >= p.N) break;
                    const float4 tsc = sh.top_score[b][r];
                    const int4 tid4 = sh.top_idx[b][r];
                    const int l = tid4.x;
                    const float4 *y4 = Y4 + (size_t)row * D4;
                    const float4 *g4 = G4 + (size_t)l * D4;
                    const float4 *b4 = B4 + (size_t)l * D4;
                    float4 *o4 = O4 + (size_t)row * D4;
                    if (D4 <= 256) {
                        float4 res[8];
                        float ysq = 0.f;
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const int c = lane + 32 * q;
                            if (c < D4) {
                                float4 y = __ldcs(y4 + c);
                                float4 g = __ldg(g4 + c);
                                float4 bb = __ldg(b4 + c);
                                ysq = fmaf(y.x, y.x, ysq);
                                ysq = fmaf(y.y, y.y, ysq);
                                ysq = fmaf(y.z, y.z, ysq);
                                ysq = fmaf(y.w, y.w, ysq);
                                res[q].x = fmaf(g.x, y.x, bb.x);
                                res[q].y = fmaf(g.y, y.y, bb.y);
                                res[q].z = fmaf(g.z, y.z, bb.z);
                                res[q].w = fmaf(g.w, y.w, bb.w);
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) ysq += __shfl_xor_sync(0xffffffffu, ysq, o);
                        const float e = tc_error_bound(p.D, ysq, cmax2);
                        const bool certain = (p.K == 1) || ((tsc.y - tsc.x) > 2.f * e);
                        if (certain) {
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const int c = lane + 32 * q;
                                if (c < D4) __stcs(o4 + c, res[q]);
                            }
                        }
                        if (lane == 0) {
                            p.labels[row] = l;
                            if (!certain) tc_decide(p, row, tsc, tid4, e);
                        }
                    } else {
                        float ysq = 0.f;
                        for (int c = lane; c < D4; c += 32) {
                            float4 y = __ldg(y4 + c);
                            ysq = fmaf(y.x, y.x, ysq);
                            ysq = fmaf(y.y, y.y, ysq);
                            ysq = fmaf(y.z, y.z, ysq);
                            ysq = fmaf(y.w, y.w, ysq);
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) ysq += __shfl_xor_sync(0xffffffffu, ysq, o);
                        const float e = tc_error_bound(p.D, ysq, cmax2);
                        const bool certain = (p.K == 1) || ((tsc.y - tsc.x) > 2.f * e);
                        if (certain) {
                            for (int c = lane; c < D4; c += 32) {
                                float4 y = __ldcs(y4 + c);
                                float4 g = __ldg(g4 + c);
                                float4 bb = __ldg(b4 + c);
                                float4 v;
                                v.x = fmaf(g.x, y.x, bb.x);
                                v.y = fmaf(g.y, y.y, bb.y);
                                v.z = fmaf(g.z, y.z, bb.z);
                                v.w = fmaf(g.w, y.w, bb.w);
                                __stcs(o4 + c, v);
                            }
                        }
                        if (lane == 0) {
                            p.labels[row] = l;
                            if (!certain) tc_decide(p, row, tsc, tid4, e);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.lab_empty[b]));
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// squared row norms (labels-only mode): one warp per row
__global__ void row_norms_kernel(const float *__restrict__ Y, int64_t N, int D, float *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= N) return;
    const float4 *y4 = reinterpret_cast<const float4 *>(Y + (size_t)row * D);
    float s = 0.f;
    for (int c = lane; c < (D >> 2); c += 32) {
        float4 v = __ldg(y4 + c);
        s = fmaf(v.x, v.x, s);
        s = fmaf(v.y, v.y, s);
        s = fmaf(v.z, v.z, s);
        s = fmaf(v.w, v.w, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    // a slight over-estimate keeps the error bound on the safe side
    if (lane == 0) out[row] = s * 1.0001f;
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 2-D fp32 row-major [rows, D] viewed in boxes of box_rows x 32 columns, 128-byte swizzle,
// zero fill outside the matrix.
bool make_map(CUtensorMap *map, const float *base, int64_t rows, int D, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * sizeof(float)};
    cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace

bool tc_supported(int64_t N, int D, int K)
{
    return (D % 4 == 0) && D >= 4 && K <= 256 && N >= 1 && encode_fn() != nullptr;
}

cudaError_t launch_row_norms(const float *Y, int64_t N, int D, float *out, cudaStream_t s)
{
    const int threads = 256;
    const int64_t blocks = (N * 32 + threads - 1) / threads;
    row_norms_kernel<<<(unsigned)blocks, threads, 0, s>>>(Y, N, D, out);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_assign_tc(const float *Y, int64_t N, int D, int K, const float *C, const float *cnorm,
                             const float *ynorm2, int32_t *labels, int32_t *refine_rows,
                             int32_t *cand_rows, uint64_t *cand_list, Control *ctl,
                             const float *gamma, const float *beta, float *out, cudaStream_t s)
{
    TcParams p{};
    p.Y = Y;
    p.cnorm = cnorm;
    p.ynorm2 = ynorm2;
    p.labels = labels;
    p.refine_rows = refine_rows;
    p.cand_rows = cand_rows;
    p.cand_list = cand_list;
    p.ctl = ctl;
    p.gamma = gamma;
    p.beta = beta;
    p.out = out;
    p.N = N;
    p.D = D;
    p.K = K;
    p.npad = (K + 15) / 16 * 16;
    int cols = 32;
    while (cols < 2 * p.npad) cols <<= 1;
    p.tmem_cols = cols;

    CUtensorMap mapA, mapB;
    if (!make_map(&mapA, Y, N, D, TC_BM) || !make_map(&mapB, C, K, D, p.npad)) return cudaErrorInvalidValue;

    const size_t smem = 1024 + (size_t)TC_STAGES * (TC_A_BYTES + (size_t)p.npad * 128) + sizeof(TcShared);
    const int64_t tiles = (N + TC_BM - 1) / TC_BM;
    const int sms = sm_count();
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    const bool affine = out != nullptr;
    cudaError_t e;
    if (affine) {
        auto kern = assign_tc_kernel<true>;
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        kern<<<grid, 32 * (2 + TC_STREAM_WARPS), smem, s>>>(mapA, mapB, p);
    } else {
        auto kern = assign_tc_kernel<false>;
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        kern<<<grid, 32 * (2 + TC_SCORE_WARPS), smem, s>>>(mapA, mapB, p);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace cat
