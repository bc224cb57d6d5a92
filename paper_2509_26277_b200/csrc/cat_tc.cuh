// Device-side building blocks of the tensor-core kernels (sm_100a): PTX wrappers for mbarriers,
// TMA, tcgen05 and TMEM, bounded waits, the packed score keys, the error bounds of the fast
// scores and the certainty test, and the row-streaming loop of the fused inference kernels.
#pragma once

#include "cat_internal.cuh"

#include <atomic>

#include <cuda.h>
#include <cuda_fp16.h>
#include <math_constants.h>

namespace cat {

// Host helpers shared by the tensor-core translation units (defined in cat_tc.cu).
// A 2-D row-major [rows, D] matrix of fp32 (or fp16) viewed in boxes of box_rows x 128 bytes with
// the 128-byte swizzle and zero fill outside the matrix; false if the encoder is unavailable.
bool tc_make_map(CUtensorMap *map, const void *base, bool half, int64_t rows, int D, int box_rows);
int tc_sm_count();

namespace {

constexpr int TC_BM = 128;                   // rows per CTA tile (UMMA M per CTA)
constexpr int TC_SLAB_BYTES = 128;           // bytes of a row per slab = one swizzle row (32 fp32 or 64 fp16)
constexpr int TC_A_BYTES = TC_BM * TC_SLAB_BYTES;  // 16 KB
constexpr int TC_MAX_A_STAGES = 8;           // ring of row slabs (filled from HBM: deep)
constexpr int TC_MAX_B_STAGES = 4;           // ring of centroid slabs (filled from L2: shallow)
constexpr uint64_t TC_TIMEOUT_NS = 2000000000ull;

// Warp roles.  Warp 0: TMA producer of the row slabs, warp 1: MMA issuer, warp 2: TMA producer
// of the centroid slabs (warp 3 idle), warps 4-7: score warps
// (TMEM lane quarter = warp & 3); with the affine epilogue also warps 8-19: streaming warps.
constexpr int TC_FIRST_SCORE_WARP = 4;
constexpr int TC_SCORE_WARPS = 4;
constexpr int TC_FIRST_STREAM_WARP = 8;
constexpr int TC_STREAM_WARPS = 12;
constexpr int TC_THREADS_LABELS = 32 * TC_FIRST_STREAM_WARP;                       // 256
constexpr int TC_THREADS_AFFINE = 32 * (TC_FIRST_STREAM_WARP + TC_STREAM_WARPS);   // 640
// Register split of the affine kernel (per thread, by warpgroup of 128 threads): the kernel
// is launched with TC_REGS_LAUNCH registers per thread; the producer/MMA warpgroup and the
// score warpgroup give registers back, the three streaming warpgroups take them.  The shares
// add up to no more than the launch total (checked again on the host before every launch).
constexpr int TC_REGS_LAUNCH = 96;
constexpr int TC_REGS_CONTROL = 24;
constexpr int TC_REGS_SCORE = 72;
constexpr int TC_REGS_STREAM = 128;
static_assert(128 * (TC_REGS_CONTROL + TC_REGS_SCORE + 3 * TC_REGS_STREAM) <= TC_REGS_LAUNCH * TC_THREADS_AFFINE,
              "register split exceeds what the block is launched with");
// The streaming warps read through L1, and the number of loads an SM keeps in flight shrinks
// with L1: a shared-memory carve-out of 200 KB and more costs a third of the streaming rate
// (measured), about 100 KB costs nothing.  The tile period of the affine kernel is long
// enough for shallow TMA rings, so that kernel takes the smaller carve-out.
constexpr int TC_AFFINE_A_STAGES = 4;
constexpr int TC_AFFINE_B_STAGES = 2;

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
// (Inlined on purpose: a called function inside the re-divided register budgets of the
// affine kernel sends ptxas into a very long compile.)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl,
                                          uint64_t limit_ns = TC_TIMEOUT_NS)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((it & 63u) == 63u) {
            uint64_t now = global_timer();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
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

// Bounded wait until *counter >= need.  Returns false after a timeout or an abort.
__device__ __forceinline__ bool wait_progress(volatile int *counter, int need, volatile int *abort_flag, Control *ctl)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (*counter >= need) return true;
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
__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// ---- cluster / cta_group::2 forms (every tcgen05 instruction of a kernel uses one cta_group)
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in the CTA of the given rank
__device__ __forceinline__ uint32_t mapa_cluster(uint32_t cta_addr, uint32_t rank)
{
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(cta_addr), "r"(rank));
    return a;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load whose completion is reported to a barrier that may live in the peer CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t cluster_bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
        ::"r"(bar)
        : "memory");
}
// arrives on this CTA's barrier only
__device__ __forceinline__ void tc_commit_pair_local(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mma_tf32_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_f16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <int R>
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(R)); }
template <int R>
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(R)); }

// 16 consecutive fp32 columns of this thread's TMEM lane.  The load is asynchronous: the
// registers hold the data only after tmem_ld_wait16 on the same array, which also keeps
// the compiler from reading them any earlier.
#define CAT_OUT(x) "=r"(x)
#define CAT_INOUT(x) "+r"(x)
#define CAT_R16(r, o) o(r[0]), o(r[1]), o(r[2]), o(r[3]), o(r[4]), o(r[5]), o(r[6]), o(r[7]), o(r[8]), o(r[9]), \
    o(r[10]), o(r[11]), o(r[12]), o(r[13]), o(r[14]), o(r[15])
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : CAT_R16(r, CAT_OUT)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait16(uint32_t (&r)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : CAT_R16(r, CAT_INOUT)::"memory");
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

// D = F32, A and B of one type (fmt 2 = TF32, 0 = F16), both K-major, M = m (128, or 256 over a
// CTA pair), N = n.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, uint32_t fmt)
{
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct TcParams {
    const float *Y;
    const float *cnorm;
    const float *ynorm2;   // [N] squared row norms (labels-only mode)
    const float *scale;    // fp16 operands: {centroid scale s_c, -2 / s_c, 2^-25 / s_c, -} followed by
                           // [N] 1 / (row scale), in device memory
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
    int npad;       // K rounded up to 32 (the score warps read TMEM 32 columns per step)
    int tmem_cols;  // power of two >= 2 * npad
    int a_stages;   // ring depths (<= TC_MAX_A_STAGES, TC_MAX_B_STAGES)
    int b_stages;
    FastOut fast;   // optional record of the fast pass (labels-only kernels)
};

struct TcShared {
    uint64_t a_full[TC_MAX_A_STAGES];
    uint64_t a_empty[TC_MAX_A_STAGES];
    uint64_t b_full[TC_MAX_B_STAGES];
    uint64_t b_empty[TC_MAX_B_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t lab_full[2];
    uint64_t lab_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    int rows_streamed;            // row slots the streaming warps have finished, all tiles
    float red[32];
    float cn[256];
    float4 top_key[2][TC_BM];     // four smallest keys of each row, ascending
};

constexpr float TC_KEY_INIT = 3.0e38f;   // larger than any finite score's key

// key = score with the centroid index in the low 8 mantissa bits
__device__ __forceinline__ float make_key(float sc, int n)
{
    return __uint_as_float((__float_as_uint(sc) & 0xFFFFFF00u) | (uint32_t)n);
}
__device__ __forceinline__ int key_index(float key) { return (int)(__float_as_uint(key) & 0xFFu); }

// fast label of a row: index of its smallest key (0 if no centroid ever won, e.g. all NaN)
__device__ __forceinline__ int key_label(float key, int K)
{
    const int l = key_index(key);
    return l < K ? l : 0;
}

// keeps (b1 <= b2 <= b3 <= b4) the four smallest keys seen
__device__ __forceinline__ void key_insert(float key, float &b1, float &b2, float &b3, float &b4)
{
    float t;
    t = fminf(b1, key); key = fmaxf(b1, key); b1 = t;
    t = fminf(b2, key); key = fmaxf(b2, key); b2 = t;
    t = fminf(b3, key); key = fmaxf(b3, key); b3 = t;
    b4 = fminf(b4, key);
}

__device__ __forceinline__ float tc_error_bound(int D, float ysq, float cmax2)
{
    const float u = 5.9604645e-8f;   // 2^-24
    const float a = 3.90625e-3f + (2.f * (float)D + 2.f) * 2.3841858e-7f;  // 2^-8 + (2D+2) 2^-22
    const float pk = 3.0517578e-5f;                                         // 2^-15: index packed into the key
    const float yc = sqrtf(ysq) * sqrtf(cmax2);
    return 1.0625f * ((a + 2.f * pk) * yc + (4.f * u + pk) * cmax2);
}

// Same for fp16 operands (round to nearest, scaled by powers of two; ay, ac = absolute rounding
// error of a row / centroid element that falls into fp16's subnormal range).
__device__ __forceinline__ float tc_error_bound_half(int D, float ysq, float cmax2, float ay, float ac)
{
    const float u = 5.9604645e-8f;   // 2^-24
    const float r = 1.953125e-3f * 1.001f + (2.f * (float)D + 2.f) * 2.3841858e-7f;  // 2^-9 (1 + 2^-12) + (2D+2) 2^-22
    const float pk = 3.0517578e-5f;
    const float yn = sqrtf(ysq), cn = sqrtf(cmax2);
    return 1.0625f * ((r + 2.f * pk) * yn * cn + 2.f * sqrtf((float)D) * (ac * yn + ay * cn) +
                      2.f * (float)D * ay * ac + (4.f * u + pk) * cmax2);
}

// Decision for one row from its four smallest keys.  Returns true when the fast argmin is
// certainly exact.  Otherwise the row is queued: with the centroids whose key lies within
// 2e of the best when those are known to be among the four, else for a scan of all K.
__device__ __forceinline__ bool tc_decide(const TcParams &p, int64_t row, float4 sc, float e)
{
    const float lim = 2.f * e;
    if (p.K == 1 || (sc.y - sc.x) > lim) return true;
    const bool more = !((sc.w - sc.x) > lim);   // the 4th is a candidate too (or NaN): others may be
    if (more && p.K > 4) {
        int slot = atomicAdd(&p.ctl->refine_count, 1);
        p.refine_rows[slot] = (int32_t)row;
    } else {
        uint64_t c = (uint64_t)(uint16_t)key_index(sc.x) | ((uint64_t)(uint16_t)key_index(sc.y) << 16);
        c |= (uint64_t)(((sc.z - sc.x) > lim || p.K < 3) ? 0xFFFFu : (uint16_t)key_index(sc.z)) << 32;
        c |= (uint64_t)(((sc.w - sc.x) > lim || p.K < 4) ? 0xFFFFu : (uint16_t)key_index(sc.w)) << 48;
        int slot = atomicAdd(&p.ctl->cand_count, 1);
        p.cand_rows[slot] = (int32_t)row;
        p.cand_list[slot] = c;
    }
    return false;
}

// One warp streams one row (1024 columns per step, all loads of a step in flight together):
// out = gamma_l * y + beta_l for the fast label l, written whether or not the label is
// certain (an undecided row is queued and the exact pass rewrites it).  Returns ||y||^2,
// accumulated on the way and complete in every lane.
__device__ __forceinline__ float stream_row_affine(const TcParams &p, int64_t row, int l, int lane)
{
    const int D4 = p.D >> 2;
    const float4 *y4 = reinterpret_cast<const float4 *>(p.Y) + (size_t)row * D4 + lane;
    const float4 *g4 = reinterpret_cast<const float4 *>(p.gamma) + (size_t)l * D4 + lane;
    const float4 *b4 = reinterpret_cast<const float4 *>(p.beta) + (size_t)l * D4 + lane;
    float4 *o4 = reinterpret_cast<float4 *>(p.out) + (size_t)row * D4 + lane;
    float ysq = 0.f;
#pragma unroll 1
    for (int h = 0; h < D4; h += 256) {
        float4 y[8], g[8], bb[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int c = h + 32 * q;
            if (c + lane < D4) {
                y[q] = __ldcs(y4 + c);
                g[q] = __ldg(g4 + c);
                bb[q] = __ldg(b4 + c);
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int c = h + 32 * q;
            if (c + lane < D4) {
                float4 v;
                v.x = fmaf(g[q].x, y[q].x, bb[q].x);
                v.y = fmaf(g[q].y, y[q].y, bb[q].y);
                v.z = fmaf(g[q].z, y[q].z, bb[q].z);
                v.w = fmaf(g[q].w, y[q].w, bb[q].w);
                __stcs(o4 + c, v);
                ysq = fmaf(y[q].x, y[q].x, ysq);
                ysq = fmaf(y[q].y, y[q].y, ysq);
                ysq = fmaf(y[q].z, y[q].z, ysq);
                ysq = fmaf(y[q].w, y[q].w, ysq);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ysq += __shfl_xor_sync(0xffffffffu, ysq, o);
    return ysq;
}

// The row-tile kernel decides certainty right after streaming the row, in the streaming warp.
// (The column-split kernel decides in its score warps instead: its streaming loop has no
// register to spare.)
__device__ __forceinline__ void stream_row(const TcParams &p, int64_t row, float4 keys, float cmax2, int lane)
{
    const int l = key_label(keys.x, p.K);
    const float ysq = stream_row_affine(p, row, l, lane);
    if (lane == 0) {
        // the row norm enters the bound slightly over-estimated
        const float e = tc_error_bound(p.D, ysq * 1.0001f, cmax2);
        p.labels[row] = l;
        tc_decide(p, row, keys, e);
    }
}

}  // namespace
}  // namespace cat
