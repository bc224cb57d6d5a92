// Fused inference kernel on 64-row tiles with fp16 operands made on the fly (sm_100a).
//
// Algorithm 2 without PCA: label_i = argmin_k ||y_i - c_k||^2, out_i = gamma_l * y_i + beta_l.
//
// The fused kernel has to read a row twice: once for the distance contraction and once, when
// its label is known, for the affine step.  Whether the second read still finds the row in L2
// depends on how many bytes every SM pulls in between, i.e. on the rows a CTA has in flight.
// The TF32 row-tile kernel needs 128 rows per CTA to keep the tensor pipe fed (its MMA takes
// 128 rows per SM at full rate only); this kernel halves that.  Its CTA pairs run
// cta_group::2 MMAs with M = 128 (64 rows per CTA, N = K split over the pair), which use the
// tensor pipe at half efficiency -- affordable because the operands are fp16 (twice the TF32
// rate): converter warps turn every fp32 row slab that TMA delivers into an fp16 operand slab
// in shared memory, scaled by a per-row power of two, and take the row norm on the way.
//
//   warp 0      TMA producer: pairs of fp32 row slabs (64 rows x 32 columns each) into a staging
//               ring, and fp16 centroid slabs (K / 2 centroids x 64 columns per CTA) into their ring
//   warp 1      MMA issuer (CTA of rank 0): tcgen05.mma.cta_group::2.kind::f16, M = 128, N = K
//   warps 4-7   score warps: TMEM -> four smallest keys per row.  With M = 128 over two CTAs a
//               CTA's accumulator holds its 64 rows twice: lanes 0-63 with the first half of
//               the centroids, lanes 64-127 with the second half; the halves are merged through
//               shared memory, then certainty test, label, queue entry for undecided rows
//   warps 8-11  converters: two threads per row; a pair of staging slabs -> registers -> one fp16
//               operand slab (128-byte swizzle written by hand), row scale, ||y||^2, overflow check
//   warps 12-19 streaming warps: second read of the row, out = gamma_l * y + beta_l
//
// Row scale.  fp16 needs the row's magnitudes inside its range, and the converter sees a row
// slab by slab, so it fixes the scale from the first step: the power of two that puts the
// largest magnitude of the first 64 columns into [2^10, 2^11).  Later elements up to 32 times
// larger still fit; if one does not (it would become inf), the row is marked and goes to the
// exact pass like any undecided row.  Elements that fall into fp16's subnormal range enter the
// error bound with their absolute rounding error, as in the fp16 path of the fit.
//
// Every wait is bounded; a wait that runs out records CAT_ERR_DEVICE_TIMEOUT and all roles
// leave.  No TMA multicast; all tensor maps cover this GPU's memory.
#include "cat_tc.cuh"

#include <cuda_bf16.h>

namespace cat {

namespace {

constexpr int H_ROWS = 64;                    // rows per CTA tile
constexpr int H_SLAB_BYTES = H_ROWS * 128;    // staging slab (64 x 32 fp32) and operand slab (64 x 64 fp16): 8 KB
constexpr int H_NS = 4;                       // staging ring, in pairs of slabs (filled from HBM)
constexpr int H_NA = 3;                       // operand ring (filled by the converters)
constexpr int H_NB = 3;                       // centroid ring (filled from L2)
constexpr int H_GATE_SLACK = 32;                // rows of tile t - 2 that may still be unstreamed when the loads of tile t start
constexpr int H_FIRST_CONV_WARP = 8;
constexpr int H_CONV_WARPS = 4;
constexpr int H_FIRST_STREAM_WARP = 12;
constexpr int H_STREAM_WARPS = 8;
constexpr int H_THREADS = 32 * (H_FIRST_STREAM_WARP + H_STREAM_WARPS);   // 640
// Register split by warpgroup; the shares add up to no more than the launch total (checked again
// on the host before every launch).
constexpr int H_REGS_LAUNCH = 96;
constexpr int H_REGS_CONTROL = 40;            // producer, MMA issuer
constexpr int H_REGS_SCORE = 72;
constexpr int H_REGS_CONV = 56;
constexpr int H_REGS_STREAM = 152;
constexpr int H_REGS_SUM = H_REGS_CONTROL + H_REGS_SCORE + H_REGS_CONV + (H_STREAM_WARPS / 4) * H_REGS_STREAM;
static_assert(128 * H_REGS_SUM <= H_REGS_LAUNCH * H_THREADS, "register split exceeds what the block is launched with");

struct H64Shared {
    uint64_t s_full[H_NS];
    uint64_t s_empty[H_NS];
    uint64_t a_full[H_NA];
    uint64_t a_empty[H_NA];
    uint64_t b_full[H_NB];
    uint64_t b_empty[H_NB];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t norm_full[2];
    uint64_t norm_empty[2];
    uint64_t half_full[2];
    uint64_t lab_full[2];
    uint64_t lab_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    int rows_streamed;
    float red[32];
    float cn[256];
    float rinv[2][H_ROWS];        // 1 / (row scale)
    float ysq[2][H_ROWS];         // ||y||^2, slightly over-estimated; +inf for a row that left the fp16 range
    float4 half_key[2][H_ROWS];   // four smallest keys over the second half of the centroids
    int lab[2][H_ROWS];           // fast labels for the streaming warps
};

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// makes this thread's earlier shared-memory writes visible to the async proxy (the MMA's operand reads)
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_half2(float a, float b)
{
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t *>(&h);
}

// Bounded wait on a barrier that CTAs of the cluster arrive on (acquire at cluster scope).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
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
// One warp streams one row: out = gamma_l * y + beta_l, all loads of a 1024-column step in flight together.
// OUT_BF16: the corrected row is stored as bf16 (round to nearest even of the fp32 result), 8 bytes per lane and step.
template <bool OUT_BF16>
__device__ __forceinline__ void stream_row_plain(const TcParams &p, int64_t row, int l, int lane)
{
    const int D4 = p.D >> 2;
    const float4 *y4 = reinterpret_cast<const float4 *>(p.Y) + (size_t)row * D4 + lane;
    const float4 *g4 = reinterpret_cast<const float4 *>(p.gamma) + (size_t)l * D4 + lane;
    const float4 *b4 = reinterpret_cast<const float4 *>(p.beta) + (size_t)l * D4 + lane;
    float4 *o4 = reinterpret_cast<float4 *>(p.out) + (size_t)row * D4 + lane;
    uint2 *o2 = reinterpret_cast<uint2 *>(p.out) + (size_t)row * D4 + lane;   // bf16 output: four values in 8 bytes
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
                if (OUT_BF16) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
                    uint2 w;
                    w.x = *reinterpret_cast<const unsigned int *>(&lo);
                    w.y = *reinterpret_cast<const unsigned int *>(&hi);
                    __stcs(o2 + c, w);
                } else {
                    __stcs(o4 + c, v);
                }
            }
        }
    }
}

// Asks L2 for the lines of a row ahead of its second read (one 128-byte line per lane and step).
__device__ __forceinline__ void prefetch_row_l2(const TcParams &p, int64_t row, int lane)
{
    const char *base = reinterpret_cast<const char *>(p.Y) + (size_t)row * p.D * 4;
    for (int off = lane * 128; off < p.D * 4; off += 32 * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
}

struct H64Params {
    TcParams t;       // Y, cnorm, scale (= {s_c, -2 / s_c, 2^-25 / s_c, -}), labels, queues, ctl, gamma, beta, out, N, D, K, npad, tmem_cols
    int nh;           // fp16 slabs (64 columns) per row
};

template <bool OUT_BF16>
__global__ void __launch_bounds__(H_THREADS, 1)
apply_h64_kernel(const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapC, H64Params hp)
{
    pdl_enter();
    const TcParams &p = hp.t;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;      // operand tiles need 1024-byte alignment for the swizzle
    unsigned char *tiles = smem_raw + (tiles_base - raw);
    const int nb_rows = p.npad >> 1;                         // centroid rows this CTA stages per slab
    const int b_bytes = nb_rows * 128;
    const uint32_t stg_base = tiles_base;
    const uint32_t a_base = stg_base + (uint32_t)(2 * H_NS * H_SLAB_BYTES);
    const uint32_t b_base = a_base + (uint32_t)(H_NA * H_SLAB_BYTES);
    H64Shared &sh = *reinterpret_cast<H64Shared *>(tiles + (size_t)(2 * H_NS + H_NA) * H_SLAB_BYTES + (size_t)H_NB * b_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                 // 0 = the CTA that issues the MMAs
    volatile int *abort_flag = &sh.abort_flag;
    const int64_t num_units = (p.N + 2 * H_ROWS - 1) / (2 * H_ROWS);     // 128-row pair tiles
    const int64_t unit_first = (int64_t)(blockIdx.x >> 1);
    const int64_t unit_step = (int64_t)(gridDim.x >> 1);
    const int nh = hp.nh;
    const int nhalf = p.npad >> 1;                           // accumulator columns per buffer

    if (tid == 0) {
        for (int s = 0; s < H_NS; ++s) {
            mbar_init(smem_u32(&sh.s_full[s]), 1);
            mbar_init(smem_u32(&sh.s_empty[s]), H_CONV_WARPS);
        }
        for (int s = 0; s < H_NA; ++s) {
            mbar_init(smem_u32(&sh.a_full[s]), 2 * H_CONV_WARPS);    // both CTAs' converter warps report to rank 0
            mbar_init(smem_u32(&sh.a_empty[s]), 1);
        }
        for (int s = 0; s < H_NB; ++s) {
            mbar_init(smem_u32(&sh.b_full[s]), 2);                   // one expect_tx arrival per CTA
            mbar_init(smem_u32(&sh.b_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh.tmem_full[b]), 1);
            mbar_init(smem_u32(&sh.tmem_empty[b]), 2 * TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.norm_full[b]), H_CONV_WARPS);
            mbar_init(smem_u32(&sh.norm_empty[b]), TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.half_full[b]), TC_SCORE_WARPS / 2);
            mbar_init(smem_u32(&sh.lab_full[b]), TC_SCORE_WARPS / 2);
            mbar_init(smem_u32(&sh.lab_empty[b]), H_STREAM_WARPS);
        }
        mbar_init(smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        sh.rows_streamed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // centroid norms (a huge finite value beyond K) and their maximum
    {
        float m = 0.f;
        for (int k = tid; k < 256; k += blockDim.x) {
            float v = (k < p.K) ? p.cnorm[k] : TC_KEY_INIT;
            sh.cn[k] = v;
            if (k < p.K) m = fmaxf(m, v);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) sh.red[warp] = m;
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&sh.tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();   // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    float cmax2 = 0.f;
    for (int w2 = 0; w2 < (int)(blockDim.x >> 5); ++w2) cmax2 = fmaxf(cmax2, sh.red[w2]);
    const uint32_t tmem_base = sh.tmem_base;
    const float s_c = p.scale[0];          // centroid scale
    const float coef_c = p.scale[1];       // -2 / s_c
    const float abs_err_c = p.scale[2];    // 2^-25 / s_c

    if (warp < TC_FIRST_SCORE_WARP) {
        setmaxnreg_dec<H_REGS_CONTROL>();   // (warps 2 and 3 have no role)
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer (rows and centroids)
            if (lane == 0) {
                uint32_t ti = 0, phs = 0, phb = 0;
                int is = 0, ib = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
                    const int64_t row0 = (unit * 2 + rank) * H_ROWS;
                    if (ti > 1) {
                        // at most one tile ahead of the streaming warps: tile ti - 2 is streamed out
                        if (!wait_progress(&sh.rows_streamed, (int)(ti - 1) * H_ROWS - H_GATE_SLACK, abort_flag, p.ctl)) { ok = false; break; }
                    }
                    for (int h = 0; h < nh && ok; ++h) {
                        if (!mbar_wait(smem_u32(&sh.b_empty[ib]), phb ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                        {
                            const uint32_t full = mapa_cluster(smem_u32(&sh.b_full[ib]), 0);
                            mbar_arrive_expect_tx_cluster(full, (uint32_t)b_bytes);
                            tma_load_2d_pair(b_base + (uint32_t)(ib * b_bytes), &mapC, full, h * 64, (int)rank * nb_rows);
                        }
                        if (++ib == H_NB) { ib = 0; phb ^= 1u; }
                        if (!mbar_wait(smem_u32(&sh.s_empty[is]), phs ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                        {
                            const uint32_t full = smem_u32(&sh.s_full[is]);
                            const uint32_t dst = stg_base + (uint32_t)(is * 2 * H_SLAB_BYTES);
                            mbar_arrive_expect_tx(full, (uint32_t)(2 * H_SLAB_BYTES));
                            // (columns beyond D read as zero)
                            tma_load_2d(dst, &mapY, full, (2 * h) * 32, (int)row0);
                            tma_load_2d(dst + (uint32_t)H_SLAB_BYTES, &mapY, full, (2 * h + 1) * 32, (int)row0);
                        }
                        if (++is == H_NS) { is = 0; phs ^= 1u; }
                    }
                }
                if (!ok) {
                    // give copies that are still in flight a bounded time to land
                    for (int s = 0; s < H_NS; ++s)
                        for (int tries = 0; tries < 100000; ++tries)
                            if (mbar_try_wait(smem_u32(&sh.s_full[s]), 0) || mbar_try_wait(smem_u32(&sh.s_full[s]), 1)) break;
                    if (rank == 0)
                        for (int s = 0; s < H_NB; ++s)
                            for (int tries = 0; tries < 100000; ++tries)
                                if (mbar_try_wait(smem_u32(&sh.b_full[s]), 0) || mbar_try_wait(smem_u32(&sh.b_full[s]), 1)) break;
                }
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------ MMA issuer
            if (lane == 0 && rank == 0) {
                const uint32_t idesc = make_idesc(2 * H_ROWS, p.npad, 0u);
                const uint64_t adesc0 = make_smem_desc(a_base), bdesc0 = make_smem_desc(b_base);
                int sa = 0, sb = 0;
                uint32_t pha = 0, phb = 0, ti = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
                    const int b = ti & 1;
                    if (!mbar_wait_cluster(smem_u32(&sh.tmem_empty[b]), ((ti >> 1) & 1u) ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + (uint32_t)(b * nhalf);
                    for (int h = 0; h < nh; ++h) {
                        if (!mbar_wait_cluster(smem_u32(&sh.b_full[sb]), phb, abort_flag, p.ctl)) { ok = false; break; }
                        if (!mbar_wait_cluster(smem_u32(&sh.a_full[sa]), pha, abort_flag, p.ctl)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t adesc = adesc0 + (uint64_t)(uint32_t)(sa * (H_SLAB_BYTES >> 4));
                        const uint64_t bdesc = bdesc0 + (uint64_t)(uint32_t)(sb * (b_bytes >> 4));
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)   // 16 fp16 = 32 B per MMA: +2 in 16-byte units
                            mma_f16_pair(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, (h > 0 || kk > 0) ? 1u : 0u);
                        // both slabs are free (in both CTAs) once these MMAs have read them
                        tc_commit_pair(smem_u32(&sh.a_empty[sa]));
                        tc_commit_pair(smem_u32(&sh.b_empty[sb]));
                        if (++sa == H_NA) { sa = 0; pha ^= 1u; }
                        if (++sb == H_NB) { sb = 0; phb ^= 1u; }
                    }
                    if (ok) tc_commit_pair(smem_u32(&sh.tmem_full[b]));
                }
                // all MMAs issued by this thread have completed once this commit arrives
                tc_commit_pair_local(smem_u32(&sh.drain));
                for (int tries = 0; tries < 4000000; ++tries)
                    if (mbar_try_wait(smem_u32(&sh.drain), 0)) break;
            }
        }
    } else if (warp < TC_FIRST_STREAM_WARP) {
        // ------------------------------------------------------------ score warps
        setmaxnreg_dec<H_REGS_SCORE>();
        const int quarter = warp & 3;             // TMEM lanes this warp may read
        const int r = (quarter & 1) * 32 + lane;  // row of the tile in this thread's lane
        const int chalf = quarter >> 1;           // which half of the centroids
        const int cbase = chalf * nhalf;
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            if (!mbar_wait_warp(smem_u32(&sh.norm_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            const float rinv = sh.rinv[b][r];
            if (!mbar_wait_warp(smem_u32(&sh.tmem_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            tc_fence_after();
            const float coef = coef_c * rinv;
            float b1 = TC_KEY_INIT, b2 = TC_KEY_INIT, b3 = TC_KEY_INIT, b4 = TC_KEY_INIT;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * nhalf);
            uint32_t ra[16], rb[16];
            tmem_ld16_issue(taddr, ra);
            for (int c = 0; c < nhalf; c += 32) {
                tmem_ld_wait16(ra);
                tmem_ld16_issue(taddr + (uint32_t)(c + 16), rb);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    key_insert(make_key(fmaf(coef, __uint_as_float(ra[j]), sh.cn[cbase + c + j]), cbase + c + j), b1, b2, b3, b4);
                tmem_ld_wait16(rb);
                if (c + 32 < nhalf) tmem_ld16_issue(taddr + (uint32_t)(c + 32), ra);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    key_insert(make_key(fmaf(coef, __uint_as_float(rb[j]), sh.cn[cbase + c + 16 + j]), cbase + c + 16 + j), b1, b2, b3, b4);
            }
            tc_fence_before();
            if (chalf == 1) {
                // hand this half's keys to the thread that holds the same row with the first half
                sh.half_key[b][r] = make_float4(b1, b2, b3, b4);
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&sh.norm_empty[b]));
                    mbar_arrive(smem_u32(&sh.half_full[b]));
                    mbar_arrive_cluster(mapa_cluster(smem_u32(&sh.tmem_empty[b]), 0));
                }
            } else {
                if (!mbar_wait_warp(smem_u32(&sh.half_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
                const float4 o = sh.half_key[b][r];
                key_insert(o.x, b1, b2, b3, b4);
                key_insert(o.y, b1, b2, b3, b4);
                key_insert(o.z, b1, b2, b3, b4);
                key_insert(o.w, b1, b2, b3, b4);
                const float yn2 = sh.ysq[b][r];
                __syncwarp();
                // accumulator buffer b, half_key[b] and the norms of buffer b may be overwritten from here on
                if (lane == 0) {
                    mbar_arrive(smem_u32(&sh.norm_empty[b]));
                    mbar_arrive_cluster(mapa_cluster(smem_u32(&sh.tmem_empty[b]), 0));
                }
                // fast label to the streaming warps (buffer b is free once tile ti - 2 is streamed)
                if (!mbar_wait_warp(smem_u32(&sh.lab_empty[b]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                const int l = key_label(b1, p.K);
                sh.lab[b][r] = l;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.lab_full[b]));
                const int64_t row = (unit * 2 + rank) * H_ROWS + r;
                if (row < p.N) {
                    const float e = tc_error_bound_half(p.D, yn2, cmax2, 2.9802322e-8f * rinv, abs_err_c);
                    p.labels[row] = l;
                    tc_decide(p, row, make_float4(b1, b2, b3, b4), e);
                }
            }
        }
    } else if (warp < H_FIRST_STREAM_WARP) {
        // ------------------------------------------------------------ converters (two threads per row of the tile)
        setmaxnreg_dec<H_REGS_CONV>();
        const int r = (warp - H_FIRST_CONV_WARP) * 16 + (lane >> 1);   // row of the tile
        const int half = lane & 1;                                     // which slab of each pair
        const uint32_t swz = (uint32_t)(r & 7);
        const float norm_slack = 1.0001f + (float)p.D * 6.0e-8f;       // covers the rounding of the running sum
        uint32_t ti = 0, phs = 0, pha = 0;
        int is = 0, ja = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            float ysq = 0.f, amax = 0.f, sc = 1.f;
            int shv = 0;
            for (int h = 0; h < nh; ++h) {
                if (!mbar_wait_warp(smem_u32(&sh.s_full[is]), phs, abort_flag, p.ctl)) { ok = false; break; }
                const uint32_t src = stg_base + (uint32_t)(is * 2 * H_SLAB_BYTES + r * 128);
                // This thread takes the 32 columns of its row in slab `half` of the pair, as eight 16-byte
                // chunks; the two threads of a row start at opposite ends (chunk j ^ 4 half at step j) so that
                // eight neighbouring lanes always touch eight different bank groups.
                float4 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    v[j] = lds128(src + (uint32_t)(half * H_SLAB_BYTES) + ((((uint32_t)(j ^ (4 * half))) ^ swz) << 4));
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.s_empty[is]));   // the slabs are in registers
                if (++is == H_NS) { is = 0; phs ^= 1u; }
                if (h == 0) {
                    // the row's scale comes from its first 64 columns
                    float m = 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        m = fmaxf(fmaxf(m, fmaxf(fabsf(v[j].x), fabsf(v[j].y))), fmaxf(fabsf(v[j].z), fabsf(v[j].w)));
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
                    int e = 0;
                    if (m > 0.f && m < CUDART_INF_F) {
                        frexpf(m, &e);          // m = f * 2^e, f in [0.5, 1)
                        shv = 11 - e;           // largest magnitude of these columns to [2^10, 2^11)
                        if (shv > 100) shv = 100;
                        if (shv < -100) shv = -100;
                    } else {
                        // all zero (or not finite): fall back to the centroids' scale
                        frexpf(s_c, &e);
                        shv = e - 1;
                    }
                    sc = ldexpf(1.f, shv);
                }
                if (!mbar_wait_warp(smem_u32(&sh.a_empty[ja]), pha ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                const uint32_t dst = a_base + (uint32_t)(ja * H_SLAB_BYTES + r * 128);
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    uint32_t hw[4];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const float4 t = v[2 * jj + u];
                        const float x0 = t.x * sc, x1 = t.y * sc, x2 = t.z * sc, x3 = t.w * sc;
                        amax = fmaxf(fmaxf(amax, fmaxf(fabsf(x0), fabsf(x1))), fmaxf(fabsf(x2), fabsf(x3)));
                        ysq = fmaf(t.x, t.x, ysq);
                        ysq = fmaf(t.y, t.y, ysq);
                        ysq = fmaf(t.z, t.z, ysq);
                        ysq = fmaf(t.w, t.w, ysq);
                        hw[2 * u] = pack_half2(x0, x1);
                        hw[2 * u + 1] = pack_half2(x2, x3);
                    }
                    // fp32 chunks (2 jj, 2 jj + 1) ^ 4 half of slab `half` make fp16 chunk 4 half + (jj ^ 2 half) of the operand row
                    const uint32_t c16 = (uint32_t)(4 * half + (jj ^ (2 * half)));
                    sts128(dst + ((c16 ^ swz) << 4), hw[0], hw[1], hw[2], hw[3]);
                }
                // The proxy fence makes this thread's operand writes visible to the tensor core of its
                // own SM; the arrival on the barrier of the issuing CTA then needs no wider release
                // (a release at cluster scope here stalls the warp for 0.5 - 1 us per slab).
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(mapa_cluster(smem_u32(&sh.a_full[ja]), 0));
                if (++ja == H_NA) { ja = 0; pha ^= 1u; }
            }
            if (!ok) break;
            ysq += __shfl_xor_sync(0xffffffffu, ysq, 1);
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            // row scale and norm for the score warps (buffer b is free once tile ti - 2 has been scored)
            if (!mbar_wait_warp(smem_u32(&sh.norm_empty[b]), ((ti >> 1) & 1u) ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
            if (half == 0) {
                sh.rinv[b][r] = ldexpf(1.f, -shv);
                // a value beyond the fp16 range (or NaN) makes the row undecidable for the fast scores
                sh.ysq[b][r] = (amax < 65000.f) ? ysq * norm_slack : CUDART_INF_F;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.norm_full[b]));
        }
    } else {
        // ------------------------------------------------------------ streaming warps
        setmaxnreg_inc<H_REGS_STREAM>();
        const int ew = warp - H_FIRST_STREAM_WARP;
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            const int64_t row0 = (unit * 2 + rank) * H_ROWS;
            if (!mbar_wait_warp(smem_u32(&sh.lab_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            for (int r = ew; r < H_ROWS; r += H_STREAM_WARPS) {
                const int64_t row = row0 + r;
                // the warp's next row (of this tile, or the first one of its next tile) on its way into L2
                const int64_t nrow = (r + H_STREAM_WARPS < H_ROWS) ? row + H_STREAM_WARPS
                                     : ((unit + unit_step < num_units) ? ((unit + unit_step) * 2 + rank) * H_ROWS + ew : p.N);
                if (nrow < p.N) prefetch_row_l2(p, nrow, lane);
                if (row < p.N) stream_row_plain<OUT_BF16>(p, row, sh.lab[b][r], lane);
                __syncwarp();
                if (lane == 0) atomicAdd(&sh.rows_streamed, 1);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.lab_empty[b]));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync();   // neither CTA's shared memory or TMEM goes away under the other
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// largest magnitude of a matrix (float bits, atomicMax into *amax_bits, which starts at 0)
__global__ void __launch_bounds__(256) absmax_kernel(const float4 *__restrict__ src, size_t n4, unsigned int *amax_bits)
{
    pdl_enter();
    float m = 0.f;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const float4 v = __ldg(src + i);
        m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m == m && m < CUDART_INF_F) atomicMax(amax_bits, __float_as_uint(m));
}

}  // namespace

bool apply_h64_supported(int64_t N, int D, int K)
{
    return tc_supported(N, D, K) && D >= 128 && (D % 8 == 0) && N > H_ROWS;
}

cudaError_t launch_absmax(const float *src, size_t n, float *scale, cudaStream_t s)
{
    cudaError_t e = cudaMemsetAsync(scale, 0, 4 * sizeof(float), s);
    if (e != cudaSuccess) return e;
    const size_t n4 = n / 4;
    size_t cb = (n4 + 255) / 256;
    if (cb > (size_t)tc_sm_count()) cb = (size_t)tc_sm_count();
    if (cb < 1) cb = 1;
    absmax_kernel<<<(unsigned)cb, 256, 0, s>>>(reinterpret_cast<const float4 *>(src), n4, reinterpret_cast<unsigned int *>(scale));
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_apply_h64(const float *Y, int64_t N, int D, int K, const void *Ch, const float *scale,
                             const float *cnorm, int32_t *labels, int32_t *refine_rows, int32_t *cand_rows,
                             uint64_t *cand_list, Control *ctl, const float *gamma, const float *beta, float *out,
                             cudaStream_t s, bool out_bf16)
{
    H64Params hp{};
    TcParams &p = hp.t;
    p.Y = Y;
    p.cnorm = cnorm;
    p.scale = scale;
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
    p.npad = (K + 63) / 64 * 64;     // each half of the centroids is read from TMEM 32 columns per step
    int cols = 32;
    while (cols < p.npad) cols <<= 1;   // two accumulator buffers of npad / 2 columns
    p.tmem_cols = cols;
    hp.nh = (D + 63) / 64;
    const int nb_rows = p.npad / 2;

    CUtensorMap mapY, mapC;
    if (!tc_make_map(&mapY, Y, false, N, D, H_ROWS) || !tc_make_map(&mapC, Ch, true, K, D, nb_rows))
        return cudaErrorInvalidValue;
    const size_t b_bytes = (size_t)nb_rows * 128;
    const size_t smem = 1024 + (size_t)(2 * H_NS + H_NA) * H_SLAB_BYTES + (size_t)H_NB * b_bytes + sizeof(H64Shared);
    const size_t smem_budget = 227 * 1024;
    const int carveout = (int)((smem * 100 + smem_budget - 1) / smem_budget);
    const int sms = tc_sm_count();
    const int64_t units = (N + 2 * H_ROWS - 1) / (2 * H_ROWS);
    const int64_t clusters = units < sms / 2 ? units : sms / 2;

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(2 * clusters), 1, 1);
    cfg.blockDim = dim3(H_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // (the kernel starts with pdl_enter)
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;

    auto kern = out_bf16 ? apply_h64_kernel<true> : apply_h64_kernel<false>;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, carveout)) != cudaSuccess) return e;
    {
        // a register split larger than what the block is launched with would wait forever
        cudaFuncAttributes fa{};
        if (cudaFuncGetAttributes(&fa, reinterpret_cast<const void *>(kern)) != cudaSuccess) return cudaErrorInvalidValue;
        if ((long)fa.numRegs * H_THREADS < 128L * H_REGS_SUM)
            return cudaErrorLaunchOutOfResources;
    }
    e = cudaLaunchKernelEx(&cfg, kern, mapY, mapC, hp);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

}  // namespace cat
