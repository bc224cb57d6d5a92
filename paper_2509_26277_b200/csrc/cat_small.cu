// Small problems (rows of at most 128 columns, at most 128 centroids): a whole Lloyd round -- and
// a whole run of rounds -- of the K-Means step of the fitting algorithm (Algorithm 1, step 2), or
// the whole of inference (Algorithm 2: nearest centroid, then gamma_l * y + beta_l), in ONE
// persistent launch of one CTA per SM.
//
// At these shapes the bytes are few (a round reads the rows once: tens of MB) and a chain of
// short kernels spends its time between launches.  Here a CTA walks its own 128-row tiles:
//
//   warp 0      TMA producer: a row tile (128 x D fp32, 128-byte swizzle) per ring stage
//   warp 1      issues the TF32 tcgen05.mma of the tile against all centroids (accumulator in
//               TMEM, one buffer per ring stage)
//   warps 4-11  score warps, two sets of four that take alternate tiles: a thread owns a row, reads
//               its scores from TMEM, keeps the four smallest keys and takes the certainty test; a
//               row that fails it is settled at once by its own thread (fp64 direct form over the
//               centroids whose key lies within the error bound of the best -- found by a second
//               read of the scores when there may be more than four), so the labels that leave
//               these warps are final
//   warps 12-27 worker warps: either add the tile's rows to per-cluster fp64 sums in shared memory
//               (warp w owns the clusters k = w mod 16, a lane owns D / 32 columns), or write
//               gamma_l * y + beta_l.
//
// After its last tile a CTA stores its partial sums; a bounded grid-wide barrier later every warp
// of the grid adds up, in a fixed order, the partials of a few (cluster, column) pairs and writes
// the new centroid entry.  A second barrier publishes the centroids for the next round.  Every
// order of summation is fixed by the launch geometry, so results repeat bit for bit.
//
// The launch is cooperative (all CTAs resident), and every wait -- on an mbarrier or on the grid
// barrier -- gives up after a time limit, raises the device status and lets the kernel return.
//
// Measured on 200 704 x 64 rows, K = 64: inference 44 us against 86 us for the general path; a
// Lloyd round 50 us against 57 us, a fit of 25 rounds 1.42 ms against 1.73 ms.
#include "cat_tc.cuh"

namespace cat {
namespace {

constexpr int SM_ROWS = 128;                 // rows per tile
constexpr int SM_MAX_STAGES = 4;
constexpr unsigned SM_POLL_SLEEP_NS = 100;
constexpr int SM_PART_PAD = 48;              // doubles between the CTAs' planes of partial sums (no power-of-two stride)
constexpr int SM_FIRST_SCORE_WARP = 4;
constexpr int SM_FIRST_WORKER_WARP = 12;     // warps 4-11: two sets of four score warps
constexpr int SM_WORKERS = 16;
constexpr int SM_WARPS = SM_FIRST_WORKER_WARP + SM_WORKERS;   // 28
constexpr int SM_THREADS = 32 * SM_WARPS;                     // 896

struct SmallParams {
    const float *Y;          // [N, D]
    float *C;                // [K, D] centroids, updated in place by a round
    int32_t *labels;         // [N] labels of the last pass (written in that pass only; may be null)
    double *part;            // [grid, K * D] partial sums of a CTA
    int32_t *part_counts;    // [2, K + 1] cluster sizes, then the count of queued rows, of the even and odd passes
                             // (both planes zero at launch)
    double *sums;            // [K * D] per-cluster sums of the last pass
    int64_t *counts;         // [K]
    const float *gamma;      // inference only
    const float *beta;
    float *out;
    Control *ctl;
    unsigned int bar_base;   // value of the counter when this launch starts
    int64_t N;
    int D;
    int K;
    int npad;                // K rounded up to 32
    int stages;              // ring depth, a power of two
    int stage_shift;         // its logarithm
    int tmem_cols;
    int passes;              // assignments to run
    int update_last;         // does the last pass move the centroids too?
};

struct SmallShared {
    uint64_t a_full[SM_MAX_STAGES];
    uint64_t a_empty[SM_MAX_STAGES];
    uint64_t tmem_full[SM_MAX_STAGES];
    uint64_t lab_full[SM_MAX_STAGES];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    int queued_pass;                        // rows this CTA queued in the current pass
    float cmax2;
    float cn[128];
    int32_t label[SM_MAX_STAGES][SM_ROWS];
};

// byte offset of element (row, col) in a 128-byte-swizzled operand tile of `rows` rows: 32-column
// slabs one after another, rows 128 B apart inside a slab, 16-byte chunks XORed with the row
__device__ __forceinline__ uint32_t swz(int rows, int row, int col)
{
    return (uint32_t)((col >> 5) * rows * 128 + row * 128 + ((((col & 31) >> 2) ^ (row & 7)) << 4) + ((col & 3) << 2));
}

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier for a cooperative launch: the whole CTA calls it.  `target` is the counter
// value once every CTA has arrived.  False after a timeout or when any CTA has given up (the
// device status is raised then, and every CTA sees it here at the latest).
__device__ __forceinline__ bool grid_barrier(const SmallParams &p, unsigned int target, volatile int *abort_flag)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&p.ctl->grid_bar, 1u);
        uint64_t t0 = 0;
        for (uint32_t it = 0;; ++it) {
            // (wrap-safe comparison: the counter only grows)
            if ((int)(ld_acquire_gpu(&p.ctl->grid_bar) - target) >= 0) break;
            if ((it & 15u) == 15u) {
                if (*abort_flag || *(volatile int *)&p.ctl->device_status != (int)CAT_OK) { *abort_flag = 1; break; }
                uint64_t now = global_timer();
                if (t0 == 0) t0 = now;
                else if (now - t0 > TC_TIMEOUT_NS) {
                    *abort_flag = 1;
                    atomicExch(&p.ctl->device_status, (int)CAT_ERR_DEVICE_TIMEOUT);
                    break;
                }
            }
        }
        __threadfence();
    }
    __syncthreads();
    return *abort_flag == 0;
}

// Bounded waits of this kernel.  Some twenty warps of a CTA are waiting at any time; a failed
// poll is followed by a short pause, which leaves the issue slots to the warps that have work
// (it costs nothing measurable).  Every lane of a waiting warp polls: a variant in which lane 0
// polled alone and told the others by a shuffle ran the kernel at half the speed.
__device__ __forceinline__ bool wait_one(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        __nanosleep(SM_POLL_SLEEP_NS);
        if ((it & 63u) == 63u) {
            const uint64_t now = global_timer();
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
// every lane polls; the warp goes on only if all lanes succeeded
__device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl, int lane)
{
    (void)lane;
    return __all_sync(0xffffffffu, wait_one(bar, parity, abort_flag, ctl));
}

// CPL consecutive columns of one row of a swizzled tile (CPL = 1, 2 or 4: inside one 16-byte chunk)
template <int CPL>
__device__ __forceinline__ void load_cols(const unsigned char *tile, int rows, int row, int col0, float (&v)[CPL])
{
    const unsigned char *src = tile + swz(rows, row, col0);
    if (CPL == 4) {
        const float4 t = *reinterpret_cast<const float4 *>(src);
        v[0] = t.x; v[1] = t.y; v[2 % CPL] = t.z; v[3 % CPL] = t.w;
    } else if (CPL == 2) {
        const float2 t = *reinterpret_cast<const float2 *>(src);
        v[0] = t.x; v[1 % CPL] = t.y;
    } else {
        v[0] = *reinterpret_cast<const float *>(src);
    }
}

__device__ __forceinline__ double warp_sum_f64(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// index of the lowest set bit of a 128-bit mask held in four words, which it clears; -1 if none
__device__ __forceinline__ int pop_lowest(uint32_t &m0, uint32_t &m1, uint32_t &m2, uint32_t &m3)
{
    int k = -1;
    if (m0) { k = __ffs(m0) - 1; m0 &= m0 - 1; }
    else if (m1) { k = 31 + __ffs(m1); m1 &= m1 - 1; }
    else if (m2) { k = 63 + __ffs(m2); m2 &= m2 - 1; }
    else if (m3) { k = 95 + __ffs(m3); m3 &= m3 - 1; }
    return k;
}

// ||y - c_a||^2 and ||y - c_b||^2 in fp32 (direct form) for row r of the staged tile, by one thread
template <int CPL>
__device__ __forceinline__ void fast_pair(const unsigned char *atile, const unsigned char *btile, int npad, int r,
                                          int ka, int kb, float &sa, float &sb)
{
    float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
#pragma unroll 4
    for (int c4 = 0; c4 < 8 * CPL; ++c4) {
        const float4 y = *reinterpret_cast<const float4 *>(atile + swz(SM_ROWS, r, c4 * 4));
        const float4 ca = *reinterpret_cast<const float4 *>(btile + swz(npad, ka, c4 * 4));
        const float4 cb = *reinterpret_cast<const float4 *>(btile + swz(npad, kb, c4 * 4));
        float d;
        d = y.x - ca.x; a0 = fmaf(d, d, a0);
        d = y.y - ca.y; a1 = fmaf(d, d, a1);
        d = y.z - ca.z; a0 = fmaf(d, d, a0);
        d = y.w - ca.w; a1 = fmaf(d, d, a1);
        d = y.x - cb.x; b0 = fmaf(d, d, b0);
        d = y.y - cb.y; b1 = fmaf(d, d, b1);
        d = y.z - cb.z; b0 = fmaf(d, d, b0);
        d = y.w - cb.w; b1 = fmaf(d, d, b1);
    }
    sa = a0 + a1;
    sb = b0 + b1;
}

// ||y - c_a||^2 and ||y - c_b||^2 in fp64 (direct form) for row r of the staged tile, by one thread:
// columns in order, even and odd columns in two partial sums each.
template <int CPL>
__device__ __forceinline__ void exact_pair(const unsigned char *atile, const unsigned char *btile, int npad, int r,
                                           int ka, int kb, double &da, double &db)
{
    double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;
#pragma unroll 4
    for (int c4 = 0; c4 < 8 * CPL; ++c4) {
        const float4 y = *reinterpret_cast<const float4 *>(atile + swz(SM_ROWS, r, c4 * 4));
        const float4 ca = *reinterpret_cast<const float4 *>(btile + swz(npad, ka, c4 * 4));
        const float4 cb = *reinterpret_cast<const float4 *>(btile + swz(npad, kb, c4 * 4));
        const double y0 = (double)y.x, y1 = (double)y.y, y2 = (double)y.z, y3 = (double)y.w;
        double d;
        d = y0 - (double)ca.x; a0 = fma(d, d, a0);
        d = y1 - (double)ca.y; a1 = fma(d, d, a1);
        d = y2 - (double)ca.z; a0 = fma(d, d, a0);
        d = y3 - (double)ca.w; a1 = fma(d, d, a1);
        d = y0 - (double)cb.x; b0 = fma(d, d, b0);
        d = y1 - (double)cb.y; b1 = fma(d, d, b1);
        d = y2 - (double)cb.z; b0 = fma(d, d, b0);
        d = y3 - (double)cb.w; b1 = fma(d, d, b1);
    }
    da = a0 + a1;
    db = b0 + b1;
}

// APPLY: inference (one pass, no sums, no grid barrier).  CPL = D / 32 columns per lane,

template <bool APPLY, int CPL>
__global__ void __launch_bounds__(SM_THREADS, 1)
small_kernel(const __grid_constant__ CUtensorMap mapA, SmallParams p)
{
    pdl_enter();
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;   // the 128-byte swizzle wants 1024-byte alignment
    unsigned char *tiles = smem_raw + (tiles_base - raw);
    const int a_bytes = SM_ROWS * p.D * 4;                // one row tile: D / 32 slabs of 16 KB
    const int b_bytes = p.npad * p.D * 4;
    const int na = p.stages;
    unsigned char *btile = tiles + (size_t)na * a_bytes;
    const uint32_t b_base = tiles_base + (uint32_t)(na * a_bytes);
    // per-cluster sums (fp64) and sizes of this CTA's rows in the current pass (fitting only)
    double *sacc = reinterpret_cast<double *>(btile + b_bytes);
    int *scnt = reinterpret_cast<int *>(sacc + (APPLY ? 0 : p.K * p.D));
    SmallShared &sh = *reinterpret_cast<SmallShared *>(scnt + (APPLY ? 0 : 128));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *abort_flag = &sh.abort_flag;
    const int num_tiles = (int)((p.N + SM_ROWS - 1) / SM_ROWS);
    const int nslabs = p.D >> 5;
    const int G = (int)gridDim.x;

    if (tid == 0) {
        for (int s = 0; s < na; ++s) {
            mbar_init(smem_u32(&sh.a_full[s]), 1);
            mbar_init(smem_u32(&sh.a_empty[s]), SM_WORKERS);
            mbar_init(smem_u32(&sh.tmem_full[s]), 1);
            mbar_init(smem_u32(&sh.lab_full[s]), 4);
        }
        mbar_init(smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        sh.queued_pass = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!APPLY) {
        for (int i = tid; i < p.K * p.D; i += SM_THREADS) sacc[i] = 0.0;
        if (tid < 128) scnt[tid] = 0;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    // tiles this CTA has been through, all passes: ring stage = count mod depth, phase = next bit
    uint32_t tcount = 0;
    unsigned int bar_next = p.bar_base;
    bool alive = true;

    for (int pass = 0; pass < p.passes && alive; ++pass) {
        // ---------------------------------------------------------------- centroids of this pass
        // into the swizzled operand tile (rows beyond K are zero), read past L1: other CTAs wrote them
        for (int i = tid; i < p.npad * (p.D >> 2); i += SM_THREADS) {
            const int k = i / (p.D >> 2), c4 = i - k * (p.D >> 2);
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k < p.K) v = __ldcg(reinterpret_cast<const float4 *>(p.C) + (size_t)k * (p.D >> 2) + c4);
            *reinterpret_cast<float4 *>(btile + swz(p.npad, k, c4 * 4)) = v;
        }
        __syncthreads();
        // squared norms in fp64, rounded up; beyond K a huge finite value
        for (int k = warp; k < 128; k += SM_WARPS) {
            float cn = TC_KEY_INIT;
            if (k < p.K) {
                float c[CPL];
                load_cols<CPL>(btile, p.npad, k, lane * CPL, c);
                double s = 0.0;
#pragma unroll
                for (int j = 0; j < CPL; ++j) s = fma((double)c[j], (double)c[j], s);
                cn = __double2float_ru(warp_sum_f64(s));
            }
            if (lane == 0) sh.cn[k] = cn;
        }
        // the MMA reads the tile through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            float m = 0.f;
            for (int k = 0; k < p.K; ++k) m = fmaxf(m, sh.cn[k]);
            sh.cmax2 = m;
        }
        __syncthreads();
        const float cmax2 = sh.cmax2;

        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            if (lane == 0) {
                for (int tile = (int)blockIdx.x; tile < num_tiles; tile += G, ++tcount) {
                    const int rs = (int)(tcount & (uint32_t)(na - 1));
                    const uint32_t rph = (tcount >> p.stage_shift) & 1u;
                    if (!wait_one(smem_u32(&sh.a_empty[rs]), rph ^ 1u, abort_flag, p.ctl)) break;
                    const uint32_t full = smem_u32(&sh.a_full[rs]);
                    mbar_arrive_expect_tx(full, (uint32_t)a_bytes);
                    for (int sl = 0; sl < nslabs; ++sl)
                        tma_load_2d(tiles_base + (uint32_t)(rs * a_bytes + sl * TC_A_BYTES), &mapA, full, sl * 32,
                                    (int)(tile * SM_ROWS));
                }
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------ MMA issuer
            if (lane == 0) {
                const uint32_t idesc = make_idesc(SM_ROWS, p.npad, 2u);
                for (int tile = (int)blockIdx.x; tile < num_tiles; tile += G, ++tcount) {
                    const int rs = (int)(tcount & (uint32_t)(na - 1));
                    const uint32_t rph = (tcount >> p.stage_shift) & 1u;
                    // (the accumulator of this stage is free: the stage itself was released by the
                    // workers, who run after the score warps, before the producer refilled it)
                    if (!wait_one(smem_u32(&sh.a_full[rs]), rph, abort_flag, p.ctl)) break;
                    tc_fence_after();
                    const uint32_t accum_at = tmem_base + (uint32_t)(rs * p.npad);
                    for (int sl = 0; sl < nslabs; ++sl) {
                        const uint64_t adesc = make_smem_desc(tiles_base + (uint32_t)(rs * a_bytes + sl * TC_A_BYTES));
                        const uint64_t bdesc = make_smem_desc(b_base + (uint32_t)(sl * p.npad * 128));
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)   // 8 tf32 = 32 B per MMA: +2 in 16-byte units
                            mma_tf32(accum_at, adesc + 2 * kk, bdesc + 2 * kk, idesc, (sl > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&sh.tmem_full[rs]));
                }
            }
        } else if (warp >= SM_FIRST_SCORE_WARP && warp < SM_FIRST_WORKER_WARP) {
            // ------------------------------------------------------------ score warps
            // Two sets of four warps take alternate tiles.  A thread owns one row: its norm, its four
            // smallest keys, the certainty test.  Rows that fail the test are then settled exactly by
            // the warp together, one row at a time, so the labels that leave here are final.
            const int set = (warp - SM_FIRST_SCORE_WARP) >> 2;
            const int quarter = warp & 3;   // the TMEM lanes this warp may read
            const int r = quarter * 32 + lane;
            int settled = 0;
            for (int tile = (int)blockIdx.x; tile < num_tiles; tile += G, ++tcount) {
                if ((int)(tcount & 1u) != set) continue;
                const int rs = (int)(tcount & (uint32_t)(na - 1));
                const uint32_t rph = (tcount >> p.stage_shift) & 1u;
                const int64_t row = (int64_t)tile * SM_ROWS + r;
                const unsigned char *atile = tiles + (size_t)rs * a_bytes;
                // (the tile itself was written through the async proxy: its own barrier makes it visible)
                if (!wait_warp(smem_u32(&sh.a_full[rs]), rph, abort_flag, p.ctl, lane)) break;
                // squared norm of this thread's row, for the error bound (fp32; over-estimated below)
                float yn2;
                {
                    // (four partial sums: one chain of D dependent FMAs would cost more than the key scan)
                    float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
#pragma unroll
                    for (int c4 = 0; c4 < 8 * CPL; ++c4) {
                        const float4 v = *reinterpret_cast<const float4 *>(atile + swz(SM_ROWS, r, c4 * 4));
                        q0 = fmaf(v.x, v.x, q0);
                        q1 = fmaf(v.y, v.y, q1);
                        q2 = fmaf(v.z, v.z, q2);
                        q3 = fmaf(v.w, v.w, q3);
                    }
                    yn2 = (q0 + q1) + (q2 + q3);
                }
                if (!wait_warp(smem_u32(&sh.tmem_full[rs]), rph, abort_flag, p.ctl, lane)) break;
                tc_fence_after();
                float b1 = TC_KEY_INIT, b2 = TC_KEY_INIT, b3 = TC_KEY_INIT, b4 = TC_KEY_INIT;
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(rs * p.npad);
                uint32_t ra[16], rb[16];
                tmem_ld16_issue(taddr, ra);
                for (int c = 0; c < p.npad; c += 32) {
                    tmem_ld_wait16(ra);
                    tmem_ld16_issue(taddr + (uint32_t)(c + 16), rb);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        key_insert(make_key(fmaf(-2.f, __uint_as_float(ra[j]), sh.cn[c + j]), c + j), b1, b2, b3, b4);
                    tmem_ld_wait16(rb);
                    if (c + 32 < p.npad) tmem_ld16_issue(taddr + (uint32_t)(c + 32), ra);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        key_insert(make_key(fmaf(-2.f, __uint_as_float(rb[j]), sh.cn[c + 16 + j]), c + 16 + j), b1, b2, b3, b4);
                }
                int lab = -1;
                // Candidates of an undecided row, one bit per centroid: those whose key lies within the
                // limit of the best.  When the fourth smallest key is still inside the limit the row's
                // scores are read once more from TMEM to find them all.
                uint32_t m0 = 0u, m1 = 0u, m2 = 0u, m3 = 0u;
                bool undecided = false, wide = false;
                float lim = 0.f;
                if (row < p.N) {
                    lab = key_label(b1, p.K);
                    lim = 2.f * tc_error_bound(p.D, yn2 * 1.0001f, cmax2);
                    if (p.K > 1 && !((b2 - b1) > lim)) {
                        undecided = true;
                        wide = !((b4 - b1) > lim) && p.K > 4;
                        if (!wide) {
                            const float bk[4] = {b1, b2, b3, b4};
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                const int k = key_index(bk[t]);
                                if (t < p.K && !((bk[t] - b1) > lim)) {
                                    const uint32_t bit = 1u << (k & 31);
                                    if (k < 32) m0 |= bit;
                                    else if (k < 64) m1 |= bit;
                                    else if (k < 96) m2 |= bit;
                                    else if (k < 128) m3 |= bit;
                                }
                            }
                        }
                    }
                }
                if (__any_sync(0xffffffffu, wide)) {
                    // (the TMEM loads are warp-wide; only the rows that asked use what they return)
#pragma unroll
                    for (int c = 0; c < 128; c += 16) {
                        if (c < p.npad) {
                            tmem_ld16_issue(taddr + (uint32_t)c, ra);
                            tmem_ld_wait16(ra);
                            uint32_t bits = 0;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float key = make_key(fmaf(-2.f, __uint_as_float(ra[j]), sh.cn[c + j]), c + j);
                                if (c + j < p.K && !((key - b1) > lim)) bits |= 1u << j;
                            }
                            if (wide) {   // (c is a constant here: one of these lines remains)
                                if (c < 32) m0 |= bits << (c & 16);
                                else if (c < 64) m1 |= bits << (c & 16);
                                else if (c < 96) m2 |= bits << (c & 16);
                                else m3 |= bits << (c & 16);
                            }
                        }
                    }
                }
                tc_fence_before();
                // Undecided rows are settled inside the thread that owns the row (all such rows of the warp
                // at once), the candidates in ascending index order, two at a time.
                settled += __popc(__ballot_sync(0xffffffffu, undecided));
                {
                    // First ||y - c||^2 in fp32, direct form.  Every term is a square, so the computed sum
                    // is within (D + 8) 2^-24, relative, of the true one: the smallest is the winner for
                    // certain when it stays the smallest with both sums moved by that much.  (Sums so small
                    // that squares may have underflowed are left to fp64.)
                    uint32_t f0 = m0, f1 = m1, f2 = m2, f3 = m3;
                    float fbest = CUDART_INF_F, fsecond = CUDART_INF_F;
                    int fk = -1;
                    while (__any_sync(0xffffffffu, (f0 | f1 | f2 | f3) != 0u)) {
                        const int ka = pop_lowest(f0, f1, f2, f3), kb = pop_lowest(f0, f1, f2, f3);
                        if (ka >= 0) {
                            float sa, sb;
                            const int kaa = ka < p.K ? ka : 0, kbb = (kb >= 0 && kb < p.K) ? kb : 0;
                            fast_pair<CPL>(atile, btile, p.npad, r, kaa, kbb, sa, sb);
                            if (ka < p.K) {
                                if (sa < fbest) { fsecond = fbest; fbest = sa; fk = ka; }
                                else fsecond = fminf(fsecond, sa);
                            }
                            if (kb >= 0 && kb < p.K) {
                                if (sb < fbest) { fsecond = fbest; fbest = sb; fk = kb; }
                                else fsecond = fminf(fsecond, sb);
                            }
                        }
                    }
                    const float eps = (float)(p.D + 8) * 5.9604645e-8f;
                    if (undecided && fk >= 0 && fbest > 1e-30f && (fsecond - fbest) > eps * (fsecond + fbest)) {
                        lab = fk;
                        m0 = m1 = m2 = m3 = 0u;
                    }
                }
                {
                    // What is left: fp64, direct form; the smallest wins, the lowest index among equals.
                    double best = CUDART_INF;
                    int bk = -1;
                    while (__any_sync(0xffffffffu, (m0 | m1 | m2 | m3) != 0u)) {
                        const int ka = pop_lowest(m0, m1, m2, m3), kb = pop_lowest(m0, m1, m2, m3);
                        if (ka >= 0) {
                            double da, db;
                            const int kaa = ka < p.K ? ka : 0, kbb = (kb >= 0 && kb < p.K) ? kb : 0;
                            exact_pair<CPL>(atile, btile, p.npad, r, kaa, kbb, da, db);
                            if (ka < p.K && da < best) { best = da; bk = ka; }
                            if (kb >= 0 && kb < p.K && db < best) { best = db; bk = kb; }
                        }
                    }
                    if (bk >= 0) lab = bk;   // (else every distance is NaN: the fast label stands)
                }
                sh.label[rs][r] = lab;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.lab_full[rs]));
            }
            if (lane == 0 && settled) atomicAdd(&sh.queued_pass, settled);
        } else if (warp >= SM_FIRST_WORKER_WARP) {
            // ------------------------------------------------------------ worker warps
            const int w = warp - SM_FIRST_WORKER_WARP;
            const int col0 = lane * CPL;
            for (int tile = (int)blockIdx.x; tile < num_tiles; tile += G, ++tcount) {
                const int rs = (int)(tcount & (uint32_t)(na - 1));
                const uint32_t rph = (tcount >> p.stage_shift) & 1u;
                if (!wait_warp(smem_u32(&sh.lab_full[rs]), rph, abort_flag, p.ctl, lane)) break;
                if (!wait_warp(smem_u32(&sh.a_full[rs]), rph, abort_flag, p.ctl, lane)) break;   // (visibility of the tile)
                const unsigned char *atile = tiles + (size_t)rs * a_bytes;
                const int64_t row0 = (int64_t)tile * SM_ROWS;
                if (w < 4 && p.labels && pass + 1 == p.passes) {
                    const int64_t row = row0 + w * 32 + lane;
                    if (row < p.N) p.labels[row] = sh.label[rs][w * 32 + lane];
                }
                if (APPLY) {
                    // rows w, w + 16, ...: four in flight
#pragma unroll 1
                    for (int r0 = w; r0 < SM_ROWS; r0 += 4 * SM_WORKERS) {
                        int l[4];
                        float y[4][CPL], g[4][CPL], b[4][CPL];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const int r = r0 + t * SM_WORKERS;
                            l[t] = sh.label[rs][r];
                            load_cols<CPL>(atile, SM_ROWS, r, col0, y[t]);
                        }
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const size_t at = (size_t)(l[t] < 0 ? 0 : l[t]) * p.D + col0;
#pragma unroll
                            for (int j = 0; j < CPL; ++j) {
                                g[t][j] = __ldg(p.gamma + at + j);
                                b[t][j] = __ldg(p.beta + at + j);
                            }
                        }
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            if (l[t] < 0) continue;   // beyond the last row (warp-uniform)
                            float o[CPL];
#pragma unroll
                            for (int j = 0; j < CPL; ++j) o[j] = fmaf(g[t][j], y[t][j], b[t][j]);
                            float *dst = p.out + (size_t)(row0 + r0 + t * SM_WORKERS) * p.D + col0;
                            if (CPL == 4) __stcs(reinterpret_cast<float4 *>(dst), make_float4(o[0], o[1 % CPL], o[2 % CPL], o[3 % CPL]));
                            else if (CPL == 2) __stcs(reinterpret_cast<float2 *>(dst), make_float2(o[0], o[1 % CPL]));
                            else __stcs(dst, o[0]);
                        }
                    }
                } else {
                    // The rows of this warp's clusters in tile order, so every sum has one fixed order.
                    // The sums live in shared memory (fp64), each cluster touched by its own warp only.
                    // A few rows are loaded before they are added.
#pragma unroll 1
                    for (int ch = 0; ch < SM_ROWS / 32; ++ch) {
                        const int lab = sh.label[rs][ch * 32 + lane];
                        unsigned m = __ballot_sync(0xffffffffu, lab >= 0 && (lab & (SM_WORKERS - 1)) == w);
                        while (m) {
                            constexpr int NB = 4;
                            int k[NB];
                            float y[NB][CPL];
#pragma unroll
                            for (int t = 0; t < NB; ++t) {
                                k[t] = -1;
                                if (m) {   // (warp-uniform)
                                    const int i = __ffs(m) - 1;
                                    m &= m - 1;
                                    k[t] = __shfl_sync(0xffffffffu, lab, i);
                                    load_cols<CPL>(atile, SM_ROWS, ch * 32 + i, col0, y[t]);
                                }
                            }
#pragma unroll
                            for (int t = 0; t < NB; ++t) {
                                if (k[t] >= 0) {   // (warp-uniform)
                                    double *a = sacc + (size_t)k[t] * p.D + col0;
#pragma unroll
                                    for (int j = 0; j < CPL; ++j) a[j] += (double)y[t][j];
                                    if (lane == 0) ++scnt[k[t]];
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.a_empty[rs]));
            }
            if (!APPLY) {
                // this CTA's partial sums, and zeros for the next pass (a pass that was cut short leaves
                // garbage: the status says so)
                __syncwarp();
                for (int k = w; k < p.K; k += SM_WORKERS) {
                    double *a = sacc + (size_t)k * p.D + col0;
#pragma unroll
                    for (int j = 0; j < CPL; ++j) {
                        __stcg(p.part + (size_t)blockIdx.x * (p.K * p.D + SM_PART_PAD) + (size_t)k * p.D + col0 + j, a[j]);
                        a[j] = 0.0;
                    }
                    if (lane == 0) {
                        // (integer sums do not depend on the order: one atomic a cluster and CTA)
                        if (scnt[k]) atomicAdd(p.part_counts + (size_t)(pass & 1) * (p.K + 1) + k, scnt[k]);
                        scnt[k] = 0;
                    }
                }
            }
        }

        __syncthreads();
        if (APPLY) {
            // rows that took the exact pass, for the caller's counters (zeroed before the launch)
            if (tid == 0 && sh.queued_pass) {
                atomicAdd(reinterpret_cast<unsigned long long *>(&p.ctl->refined_total), (unsigned long long)sh.queued_pass);
                atomicAdd(reinterpret_cast<unsigned long long *>(&p.ctl->refined_last), (unsigned long long)sh.queued_pass);
            }
            break;
        }
        const int KD = p.K * p.D;
        if (tid == 0) {
            if (sh.queued_pass) atomicAdd(p.part_counts + (size_t)(pass & 1) * (p.K + 1) + p.K, sh.queued_pass);
            sh.queued_pass = 0;
        }
        bar_next += (unsigned int)G;
        if (!grid_barrier(p, bar_next, abort_flag)) { alive = false; break; }

        // ---------------------------------------------------------------- grid-wide combine
        // One warp per four neighbouring columns of a cluster: lane (g8, c) takes column c of the CTAs
        // g8, g8 + 8, ... in that order, so that the four lanes of a CTA read one 32-byte sector
        // together, and a fixed three-step tree adds the eight partial sums.  The last pass of a fit
        // leaves the centroids alone (its sums and sizes feed the closed form).
        const bool update = pass + 1 < p.passes || p.update_last != 0;
        const int32_t *kcount = p.part_counts + (size_t)(pass & 1) * (p.K + 1);
        static_assert(SMALL_MAX_GRID <= 8 * 20, "a lane holds at most twenty CTAs' partials");
        for (int e4 = (int)blockIdx.x * SM_WARPS + warp; e4 < (KD >> 2); e4 += G * SM_WARPS) {
            const int e = 4 * e4 + (lane & 3);
            const int k = e / p.D;
            // (a lane's loads are all issued before the first is used: they are L2 round trips)
            double v[20];
#pragma unroll
            for (int t = 0; t < 20; ++t) {
                const int g = (lane >> 2) + 8 * t;
                v[t] = g < G ? __ldcg(p.part + (size_t)g * (KD + SM_PART_PAD) + e) : 0.0;
            }
            const long long n = __ldcg(kcount + k);
            double s = v[0];
#pragma unroll
            for (int t = 1; t < 20; ++t)
                if ((lane >> 2) + 8 * t < G) s += v[t];   // (never adds a +0.0 that could turn -0.0 around)
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane < 4) {
                p.sums[e] = s;
                if (e == k * p.D) p.counts[k] = n;
                if (update && n > 0) __stcg(p.C + e, (float)(s / (double)n));
            }
        }
        if (blockIdx.x == 0 && warp == 0 && lane == 0) {
            const long long q = __ldcg(kcount + p.K);
            p.ctl->refined_last = q;
            p.ctl->refined_total += q;
        }
        // the other plane of counts is the next pass's: nobody reads or adds to it before the barrier below
        if (blockIdx.x == 0)
            for (int i = tid; i <= p.K; i += SM_THREADS) p.part_counts[(size_t)((pass + 1) & 1) * (p.K + 1) + i] = 0;
        if (pass + 1 < p.passes) {
            bar_next += (unsigned int)G;
            if (!grid_barrier(p, bar_next, abort_flag)) { alive = false; break; }
        }
    }

    // ---------------------------------------------------------------- teardown
    if (warp == 1 && lane == 0) {
        // every MMA this thread issued has completed once this commit arrives
        tc_commit(smem_u32(&sh.drain));
        for (int tries = 0; tries < 4000000; ++tries)
            if (mbar_try_wait(smem_u32(&sh.drain), 0)) break;
    }
    if (warp == 0 && lane == 0 && *abort_flag) {
        // give copies that are still in flight a bounded time to land
        for (int s = 0; s < na; ++s)
            for (int tries = 0; tries < 100000; ++tries)
                if (mbar_try_wait(smem_u32(&sh.a_full[s]), 0) || mbar_try_wait(smem_u32(&sh.a_full[s]), 1)) break;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

}  // namespace

namespace {

struct SmallGeom {
    int cpl, npad, stages, stage_shift, tmem_cols;
    size_t smem;
};

bool small_geometry(int D, int K, bool apply, SmallGeom *g)
{
    if (!(D == 32 || D == 64 || D == 128) || K < 1 || K > 128) return false;
    g->cpl = D / 32;
    if (!apply && K * D > 4096) return false;   // the fp64 sums take K * D * 8 bytes of shared memory
    g->npad = (K + 31) / 32 * 32;
    const int a_bytes = SM_ROWS * D * 4;
    g->stages = 131072 / a_bytes < SM_MAX_STAGES ? 131072 / a_bytes : SM_MAX_STAGES;   // 4, or 2 at D = 128
    g->stage_shift = g->stages == 4 ? 2 : 1;
    int cols = 32;
    while (cols < g->stages * g->npad) cols <<= 1;
    g->tmem_cols = cols;
    g->smem = 1024 + (size_t)g->stages * a_bytes + (size_t)g->npad * D * 4 + (apply ? 0 : (size_t)K * D * 8 + 512) +
              sizeof(SmallShared);
    return cols <= 512 && g->smem <= 227 * 1024;
}

template <bool APPLY, int CPL>
cudaError_t launch_one(const CUtensorMap &map, const SmallParams &p, int grid, size_t smem, cudaStream_t s)
{
    auto kern = small_kernel<APPLY, CPL>;
    static std::atomic<bool> prepared{false};
    if (!prepared.load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        prepared.store(true, std::memory_order_release);
    }
    if constexpr (APPLY) {
        // no CTA waits for another: an ordinary launch, allowed to start early
        launch_pdl(kern, dim3(grid), dim3(SM_THREADS), smem, s, map, p);
    } else {
        // the grid barrier needs every CTA resident
        int per_sm = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, SM_THREADS, smem);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
        void *args[] = {(void *)&map, (void *)&p};
        e = cudaLaunchCooperativeKernel((const void *)kern, dim3(grid), dim3(SM_THREADS), args, smem, s);
        if (e != cudaSuccess) return e;
    }
    count_launch();
    return cudaGetLastError();
}

template <bool APPLY>
cudaError_t dispatch(const SmallGeom &g, const CUtensorMap &map, const SmallParams &p, int grid, cudaStream_t s)
{
    if (g.cpl == 1) return launch_one<APPLY, 1>(map, p, grid, g.smem, s);
    if (g.cpl == 2) return launch_one<APPLY, 2>(map, p, grid, g.smem, s);
    if (g.cpl == 4) return launch_one<APPLY, 4>(map, p, grid, g.smem, s);
    return cudaErrorInvalidValue;
}

}  // namespace

bool small_fit_supported(int64_t N, int D, int K)
{
    SmallGeom g;
    return N >= SM_ROWS && N < ((int64_t)1 << 31) - SM_ROWS && small_geometry(D, K, false, &g);
}

bool small_apply_supported(int64_t N, int D, int K)
{
    SmallGeom g;
    return N >= SM_ROWS && N < ((int64_t)1 << 31) - SM_ROWS && small_geometry(D, K, true, &g);
}

size_t small_part_doubles(int D, int K) { return (size_t)SMALL_MAX_GRID * ((size_t)K * D + SM_PART_PAD); }
size_t small_part_counts(int K) { return 2 * ((size_t)K + 1); }

static int small_grid(int64_t N)
{
    int grid = tc_sm_count();
    if (grid > SMALL_MAX_GRID) grid = SMALL_MAX_GRID;
    const int64_t tiles = (N + SM_ROWS - 1) / SM_ROWS;
    if (tiles < grid) grid = (int)tiles;
    return grid < 1 ? 1 : grid;
}

// `passes` assignments from the centroids in C; all but the last (and the last too with
// update_last) replace C by the cluster means.  labels, sums and counts describe the last pass.
// *bar_count follows the grid barrier's counter (zero after launch_reset_control).
cudaError_t launch_small_fit(const float *Y, int64_t N, int D, int K, float *C, int passes, bool update_last,
                             int32_t *labels, double *part, int32_t *part_counts, double *sums, int64_t *counts,
                             Control *ctl, unsigned int *bar_count, cudaStream_t s)
{
    SmallGeom g;
    if (!small_geometry(D, K, false, &g) || passes < 1) return cudaErrorInvalidValue;
    CUtensorMap map;
    if (!tc_make_map(&map, Y, false, N, D, SM_ROWS)) return cudaErrorNotSupported;
    SmallParams p{};
    p.Y = Y; p.C = C; p.labels = labels; p.part = part; p.part_counts = part_counts; p.sums = sums; p.counts = counts;
    p.ctl = ctl; p.bar_base = *bar_count; p.N = N; p.D = D; p.K = K; p.npad = g.npad; p.stages = g.stages; p.stage_shift = g.stage_shift;
    p.tmem_cols = g.tmem_cols; p.passes = passes; p.update_last = update_last ? 1 : 0;
    cudaError_t e0 = cudaMemsetAsync(part_counts, 0, small_part_counts(K) * sizeof(int32_t), s);
    if (e0 != cudaSuccess) return e0;
    const int grid = small_grid(N);
    *bar_count += (unsigned int)grid * (unsigned int)(2 * passes - 1);
    return dispatch<false>(g, map, p, grid, s);
}

cudaError_t launch_small_apply(const float *Y, int64_t N, int D, int K, const float *C, const float *gamma,
                               const float *beta, float *out, int32_t *labels, Control *ctl, cudaStream_t s)
{
    SmallGeom g;
    if (!small_geometry(D, K, true, &g)) return cudaErrorInvalidValue;
    CUtensorMap map;
    if (!tc_make_map(&map, Y, false, N, D, SM_ROWS)) return cudaErrorNotSupported;
    SmallParams p{};
    p.Y = Y; p.C = const_cast<float *>(C); p.labels = labels; p.gamma = gamma; p.beta = beta; p.out = out; p.ctl = ctl;
    p.N = N; p.D = D; p.K = K; p.npad = g.npad; p.stages = g.stages; p.stage_shift = g.stage_shift; p.tmem_cols = g.tmem_cols; p.passes = 1;
    return dispatch<true>(g, map, p, small_grid(N), s);
}

}  // namespace cat
