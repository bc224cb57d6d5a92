// Tensor-core path of the nearest-centroid assignment (sm_100a: tcgen05 + TMEM + TMA).
//
// The N x K x D distance contraction y_i . c_k runs as a TF32 UMMA.  A persistent CTA
// walks 128-row tiles; TMA streams 128 x 32 fp32 slabs of the rows and slabs of the
// centroids into 128-byte-swizzled shared memory, one thread issues
// tcgen05.mma.kind::tf32 into a TMEM accumulator (128 lanes x K columns, two buffers),
// and the score warps read the scores back with tcgen05.ld and keep the four smallest per
// row.  With more than one tile of rows the CTAs work in pairs (cta_group::2, M = 256):
// each CTA of a pair stages its own 128 rows and HALF the centroids, which halves the
// centroid bytes that leave L2 per row.
//
// A score travels as a "key": its fp32 bits with the low 8 bits replaced by the centroid
// index, so that the four smallest come out of a branch-free min/max insertion network.
// The certainty test is the one of the fp32 path with the error bound
//     e <= (2^-8 + (2D+2) 2^-22) ||y|| cmax + 4 u cmax^2 + 2^-15 (cmax^2 + 2 ||y|| cmax)
// (operands cut to 11 significant bits: <= 2^-10 each; fp32 accumulation inside the
// tensor core taken as <= 2^-22 per term; the last term is the index packed into the
// key).  Rows it cannot decide go to the same exact fp64 pass, so labels stay exact.
//
// cat_fit assigns the same rows many times, so it keeps an fp16 copy of them (each row scaled
// by its own power of two so that its largest magnitude sits near 2^14, rounded to nearest;
// the centroids by one power of two taken from the largest magnitude of the whole matrix) and
// runs the labels kernel on that copy with kind::f16: twice the MMA rate of TF32, half the row
// bytes, and a tighter operand bound (2^-11 per operand instead of 2^-10):
//     e <= (2^-9 + (2D+2) 2^-22) ||y|| cmax + 2 sqrt(D) (a_c ||y|| + a_y cmax) + 2 D a_y a_c + 4 u cmax^2 + (packing term)
// where a_y = 2^-25 / (row scale), a_c = 2^-25 / (centroid scale) are the absolute rounding
// errors of an element that falls into fp16's subnormal range.
//
// For inference, streaming warps then read every row of the tile once more and write
// gamma_l * y + beta_l for the fast label l; an undecided row is queued and the exact pass
// rewrites its output.  The TMA producer may run at most one tile ahead of the streaming
// warps, which bounds the bytes between a row's first read and its second.  A second form of the
// same step (apply_split_kernel, selectable, off by default) shares one 128-row tile among the CTAs
// of a cluster by columns and sums the partial scores through distributed shared memory.
//
// Every wait on an mbarrier or a progress counter is bounded (about 2 s): on a timeout the
// CTA records CAT_ERR_DEVICE_TIMEOUT in the control block, all roles leave their loops,
// outstanding copies and MMAs are drained with bounded waits, TMEM is freed and the kernel
// returns.
#include "cat_tc.cuh"

#include <mutex>

namespace cat {

namespace {

// The same for short rows (D < 128): a row takes only G = 1 .. 32 lanes, so a warp streams all
// of its rows of the tile (ew, ew + TC_STREAM_WARPS, ...) in one step, 32 / G rows per load slot.
__device__ __forceinline__ void stream_rows_short(const TcParams &p, int64_t row0, const float4 *tile_keys, int ew,
                                                  float cmax2, int lane)
{
    const int D4 = p.D >> 2;
    int G = 1;
    while (G < D4) G <<= 1;
    const int rps = 32 / G;            // rows per slot
    const int c = lane & (G - 1);      // float4 column of this lane
    const int sub = lane / G;          // which of the slot's rows
    // batches of four load slots (4 * rps rows) until the warp's rows of the tile are done
#pragma unroll 1
    for (int i0 = 0; ew + TC_STREAM_WARPS * i0 < TC_BM; i0 += 4 * rps) {
        float4 y[4], g[4], bb[4];
        unsigned act = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int r = ew + TC_STREAM_WARPS * (i0 + q * rps + sub);
            const int64_t row = row0 + r;
            if ((r < TC_BM) && (row < p.N) && (c < D4)) {
                act |= 1u << q;
                const int l = key_label(tile_keys[r].x, p.K);
                y[q] = __ldcs(reinterpret_cast<const float4 *>(p.Y) + (size_t)row * D4 + c);
                g[q] = __ldg(reinterpret_cast<const float4 *>(p.gamma) + (size_t)l * D4 + c);
                bb[q] = __ldg(reinterpret_cast<const float4 *>(p.beta) + (size_t)l * D4 + c);
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float ysq = 0.f;
            const int r = ew + TC_STREAM_WARPS * (i0 + q * rps + sub);
            const int64_t row = row0 + r;
            if (act & (1u << q)) {
                float4 v;
                v.x = fmaf(g[q].x, y[q].x, bb[q].x);
                v.y = fmaf(g[q].y, y[q].y, bb[q].y);
                v.z = fmaf(g[q].z, y[q].z, bb[q].z);
                v.w = fmaf(g[q].w, y[q].w, bb[q].w);
                __stcs(reinterpret_cast<float4 *>(p.out) + (size_t)row * D4 + c, v);
                ysq = fmaf(y[q].x, y[q].x, fmaf(y[q].y, y[q].y, fmaf(y[q].z, y[q].z, y[q].w * y[q].w)));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
                if (o < G) ysq += __shfl_xor_sync(0xffffffffu, ysq, o);
            if ((act & (1u << q)) && c == 0) {
                const float4 keys = tile_keys[r];
                const float e = tc_error_bound(p.D, ysq * 1.0001f, cmax2);
                p.labels[row] = key_label(keys.x, p.K);
                tc_decide(p, row, keys, e);
            }
        }
    }
}

// PAIR: the two CTAs of a cluster work as one cta_group::2 unit on 256 rows.  Each CTA
// loads the slabs of its own 128 rows and of HALF the centroids; the MMA (M = 256, issued
// by the CTA of rank 0) reads both halves, and each CTA finds the scores of its own rows in
// its own TMEM.
// HALF: operands are the fp16 copies of the rows and centroids (64 columns per slab, kind::f16).
// SHORT (affine epilogue only): rows of fewer than 128 columns, streamed several per warp step.
template <bool AFFINE, bool PAIR, bool HALF, bool SHORT>
__global__ void __launch_bounds__(AFFINE ? TC_THREADS_AFFINE : TC_THREADS_LABELS, 1)
assign_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcParams p)
{
    pdl_enter();
    extern __shared__ unsigned char smem_raw[];
    // operand tiles need 1024-byte alignment for the 128-byte swizzle
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char *tiles = smem_raw + (tiles_base - raw);
    const int nb_rows = PAIR ? (p.npad >> 1) : p.npad;   // centroid rows this CTA stages per slab
    const int b_bytes = nb_rows * 128;
    const int na = p.a_stages, nb = p.b_stages;
    const uint32_t b_base = tiles_base + (uint32_t)(na * TC_A_BYTES);   // the centroid ring follows the row ring
    TcShared &sh = *reinterpret_cast<TcShared *>(tiles + (size_t)na * TC_A_BYTES + (size_t)nb * b_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // 0 = the CTA that issues the MMAs
    volatile int *abort_flag = &sh.abort_flag;
    // work units: 128-row tiles, or 256-row pair tiles shared by the two CTAs of a cluster
    const int64_t num_units = PAIR ? (p.N + 2 * TC_BM - 1) / (2 * TC_BM) : (p.N + TC_BM - 1) / TC_BM;
    const int64_t unit_first = PAIR ? (int64_t)(blockIdx.x >> 1) : (int64_t)blockIdx.x;
    const int64_t unit_step = PAIR ? (int64_t)(gridDim.x >> 1) : (int64_t)gridDim.x;
    constexpr int BK = HALF ? 64 : 32;   // columns per slab
    const int nslabs = (p.D + BK - 1) / BK;
    const float coef_c = HALF ? p.scale[1] : -2.f;             // score = cn + coef * accumulator
    const float abs_err_c = HALF ? p.scale[2] : 0.f;

    if (tid == 0) {
        for (int s = 0; s < na; ++s) {
            mbar_init(smem_u32(&sh.a_full[s]), PAIR ? 2 : 1);    // one expect_tx arrival per CTA
            mbar_init(smem_u32(&sh.a_empty[s]), 1);
        }
        for (int s = 0; s < nb; ++s) {
            mbar_init(smem_u32(&sh.b_full[s]), PAIR ? 2 : 1);
            mbar_init(smem_u32(&sh.b_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh.tmem_full[b]), 1);
            mbar_init(smem_u32(&sh.tmem_empty[b]), (PAIR ? 2 : 1) * TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.lab_full[b]), TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.lab_empty[b]), TC_STREAM_WARPS);
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
        if (PAIR) {
            tmem_alloc_pair(smem_u32(&sh.tmem_base), (uint32_t)p.tmem_cols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(&sh.tmem_base), (uint32_t)p.tmem_cols);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync();   // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    float cmax2 = 0.f;
    for (int w2 = 0; w2 < (int)(blockDim.x >> 5); ++w2) cmax2 = fmaxf(cmax2, sh.red[w2]);
    const uint32_t tmem_base = sh.tmem_base;

    // With the affine epilogue each warpgroup first trades registers: the control and score
    // warpgroups give some back, the streaming warpgroups take them.
    if (warp < TC_FIRST_SCORE_WARP) {
        if (AFFINE) setmaxnreg_dec<TC_REGS_CONTROL>();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            if (lane == 0) {
                uint32_t ti = 0, ph = 0;
                int s = 0;   // ring position and phase, carried along
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
                    const int64_t row0 = PAIR ? (unit * 2 + rank) * TC_BM : unit * TC_BM;
                    if (AFFINE && !SHORT && ti > 1) {
                        // at most one tile ahead of the streaming warps: tile ti - 2 is streamed out
                        // (short rows: a tile is a few KB, the ring depths alone bound the lead)
                        if (!wait_progress(&sh.rows_streamed, (int)(ti - 1) * TC_BM, abort_flag, p.ctl)) { ok = false; break; }
                    }
                    for (int sl = 0; sl < nslabs; ++sl) {
                        if (!mbar_wait(smem_u32(&sh.a_empty[s]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                        const uint32_t a_dst = tiles_base + (uint32_t)(s * TC_A_BYTES);
                        if (PAIR) {
                            // both CTAs report to the barrier of the MMA-issuing CTA
                            const uint32_t full = mapa_cluster(smem_u32(&sh.a_full[s]), 0);
                            mbar_arrive_expect_tx_cluster(full, (uint32_t)TC_A_BYTES);
                            tma_load_2d_pair(a_dst, &mapA, full, sl * BK, (int)row0);
                        } else {
                            const uint32_t full = smem_u32(&sh.a_full[s]);
                            mbar_arrive_expect_tx(full, (uint32_t)TC_A_BYTES);
                            tma_load_2d(a_dst, &mapA, full, sl * BK, (int)row0);
                        }
                        if (++s == na) { s = 0; ph ^= 1u; }
                    }
                }
                if (!ok && rank == 0) {
                    // give copies that are still in flight a bounded time to land
                    for (int s = 0; s < na; ++s)
                        for (int tries = 0; tries < 100000; ++tries)
                            if (mbar_try_wait(smem_u32(&sh.a_full[s]), 0) || mbar_try_wait(smem_u32(&sh.a_full[s]), 1)) break;
                }
            }
        } else if (warp == 2) {
            // ------------------------------------------------------------ TMA producer, centroid slabs
            if (lane == 0) {
                uint32_t ph = 0;
                int s = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step) {
                    for (int sl = 0; sl < nslabs; ++sl) {
                        if (!mbar_wait(smem_u32(&sh.b_empty[s]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                        const uint32_t b_dst = b_base + (uint32_t)(s * b_bytes);
                        if (PAIR) {
                            const uint32_t full = mapa_cluster(smem_u32(&sh.b_full[s]), 0);
                            mbar_arrive_expect_tx_cluster(full, (uint32_t)b_bytes);
                            tma_load_2d_pair(b_dst, &mapB, full, sl * BK, (int)rank * nb_rows);
                        } else {
                            const uint32_t full = smem_u32(&sh.b_full[s]);
                            mbar_arrive_expect_tx(full, (uint32_t)b_bytes);
                            tma_load_2d(b_dst, &mapB, full, sl * BK, 0);
                        }
                        if (++s == nb) { s = 0; ph ^= 1u; }
                    }
                }
                if (!ok && rank == 0) {
                    for (int s = 0; s < nb; ++s)
                        for (int tries = 0; tries < 100000; ++tries)
                            if (mbar_try_wait(smem_u32(&sh.b_full[s]), 0) || mbar_try_wait(smem_u32(&sh.b_full[s]), 1)) break;
                }
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------ MMA issuer
            if (lane == 0 && rank == 0) {
                const uint32_t idesc = make_idesc(PAIR ? 2 * TC_BM : TC_BM, p.npad, HALF ? 0u : 2u);
                const uint64_t adesc0 = AFFINE ? 0 : make_smem_desc(tiles_base), bdesc0 = AFFINE ? 0 : make_smem_desc(b_base);
                int sa = 0, sb = 0;
                uint32_t pha = 0, phb = 0, ti = 0, it = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
                    const int b = ti & 1;
                    if (!mbar_wait(smem_u32(&sh.tmem_empty[b]), ((ti >> 1) & 1u) ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + (uint32_t)(b * p.npad);
                    for (int sl = 0; sl < nslabs; ++sl) {
                        // ring positions and phases are carried along (no division in this loop: the
                        // issuing thread's own instruction count is what paces the MMAs)
                        if (!mbar_wait(smem_u32(&sh.b_full[sb]), phb, abort_flag, p.ctl)) { ok = false; break; }
                        if (!mbar_wait(smem_u32(&sh.a_full[sa]), pha, abort_flag, p.ctl)) { ok = false; break; }
                        tc_fence_after();
                        // (the start address sits in the low bits of the descriptor, in 16-byte units)
                        const uint64_t adesc = AFFINE ? make_smem_desc(tiles_base + (uint32_t)(sa * TC_A_BYTES))
                                                      : adesc0 + (uint64_t)(uint32_t)(sa * (TC_A_BYTES >> 4));
                        const uint64_t bdesc = AFFINE ? make_smem_desc(b_base + (uint32_t)(sb * b_bytes))
                                                      : bdesc0 + (uint64_t)(uint32_t)(sb * (b_bytes >> 4));
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {   // 8 tf32 or 16 f16 = 32 B per MMA: +2 in 16-byte units
                            const uint32_t accum = (sl > 0 || kk > 0) ? 1u : 0u;
                            if (HALF) {
                                if (PAIR) mma_f16_pair(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, accum);
                                else mma_f16(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, accum);
                            } else {
                                if (PAIR) mma_tf32_pair(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, accum);
                                else mma_tf32(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, accum);
                            }
                        }
                        // both slabs are free (in both CTAs) once these MMAs have read them
                        if (PAIR) {
                            tc_commit_pair(smem_u32(&sh.a_empty[sa]));
                            tc_commit_pair(smem_u32(&sh.b_empty[sb]));
                        } else {
                            tc_commit(smem_u32(&sh.a_empty[sa]));
                            tc_commit(smem_u32(&sh.b_empty[sb]));
                        }
                        if (AFFINE) {
                            // (the 24-register budget of this warp in the affine kernel has no room for
                            // the carried positions; the MMAs are not what bounds that kernel)
                            ++it;
                            sa = (int)(it % (uint32_t)na);
                            pha = (it / (uint32_t)na) & 1u;
                            sb = (int)(it % (uint32_t)nb);
                            phb = (it / (uint32_t)nb) & 1u;
                        } else {
                            if (++sa == na) { sa = 0; pha ^= 1u; }
                            if (++sb == nb) { sb = 0; phb ^= 1u; }
                        }
                    }
                    if (ok) {
                        if (PAIR) tc_commit_pair(smem_u32(&sh.tmem_full[b])); else tc_commit(smem_u32(&sh.tmem_full[b]));
                    }
                }
                // all MMAs issued by this thread have completed once this commit arrives
                if (PAIR) tc_commit_pair_local(smem_u32(&sh.drain)); else tc_commit(smem_u32(&sh.drain));
                for (int tries = 0; tries < 4000000; ++tries)
                    if (mbar_try_wait(smem_u32(&sh.drain), 0)) break;
            }
        }
    } else if (warp < TC_FIRST_STREAM_WARP) {
        // ------------------------------------------------------------ score warps
        if (AFFINE) setmaxnreg_dec<TC_REGS_SCORE>();
        const int quarter = warp & 3;             // TMEM lanes this warp may read
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            const int64_t row0 = PAIR ? (unit * 2 + rank) * TC_BM : unit * TC_BM;
            // what the certainty test needs from global memory is requested before the wait for the
            // scores, so that its latency passes during the MMAs (fp16 operands: this thread's row has
            // its own scale)
            float rinv = 1.f, yn2 = 0.f;
            if (HALF && row0 + quarter * 32 + lane < p.N) rinv = p.scale[4 + row0 + quarter * 32 + lane];
            if (!AFFINE && row0 + quarter * 32 + lane < p.N) yn2 = p.ynorm2[row0 + quarter * 32 + lane];
            if (!mbar_wait_warp(smem_u32(&sh.tmem_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            tc_fence_after();
            const float coef = coef_c * rinv;
            float b1 = TC_KEY_INIT, b2 = TC_KEY_INIT, b3 = TC_KEY_INIT, b4 = TC_KEY_INIT;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * p.npad);
            // two register buffers: the next 16 columns are in flight while these are scanned
            uint32_t ra[16], rb[16];
            tmem_ld16_issue(taddr, ra);
            for (int c = 0; c < p.npad; c += 32) {
                tmem_ld_wait16(ra);
                tmem_ld16_issue(taddr + (uint32_t)(c + 16), rb);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    key_insert(make_key(fmaf(coef, __uint_as_float(ra[j]), sh.cn[c + j]), c + j), b1, b2, b3, b4);
                tmem_ld_wait16(rb);
                if (c + 32 < p.npad) tmem_ld16_issue(taddr + (uint32_t)(c + 32), ra);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    key_insert(make_key(fmaf(coef, __uint_as_float(rb[j]), sh.cn[c + 16 + j]), c + 16 + j), b1, b2, b3, b4);
            }
            // accumulator buffer b may be overwritten from here on
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(mapa_cluster(smem_u32(&sh.tmem_empty[b]), 0));
                else mbar_arrive(smem_u32(&sh.tmem_empty[b]));
            }
            const int r = quarter * 32 + lane;
            if (AFFINE) {
                // hand the keys to the streaming warps (buffer b is free once tile ti - 2 is streamed)
                if (!mbar_wait_warp(smem_u32(&sh.lab_empty[b]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                sh.top_key[b][r] = make_float4(b1, b2, b3, b4);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.lab_full[b]));
            } else {
                const int64_t row = row0 + r;
                if (row < p.N) {
                    const float e = HALF ? tc_error_bound_half(p.D, yn2, cmax2, 2.9802322e-8f * rinv, abs_err_c)
                                         : tc_error_bound(p.D, yn2, cmax2);
                    p.labels[row] = key_label(b1, p.K);
                    if (p.fast.best) p.fast.best[row] = b1;
                    if (p.fast.second) p.fast.second[row] = b2;
                    if (p.fast.bound) p.fast.bound[row] = e;
                    if (p.fast.label) p.fast.label[row] = key_label(b1, p.K);
                    tc_decide(p, row, make_float4(b1, b2, b3, b4), e);
                }
            }
        }
    } else if (AFFINE) {
        // ------------------------------------------------------------ streaming warps
        setmaxnreg_inc<TC_REGS_STREAM>();
        const int ew = warp - TC_FIRST_STREAM_WARP;
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            const int64_t row0 = PAIR ? (unit * 2 + rank) * TC_BM : unit * TC_BM;
            if (!mbar_wait_warp(smem_u32(&sh.lab_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            if (SHORT) {
                stream_rows_short(p, row0, sh.top_key[b], ew, cmax2, lane);
                __syncwarp();
                if (lane == 0) atomicAdd(&sh.rows_streamed, (TC_BM - ew + TC_STREAM_WARPS - 1) / TC_STREAM_WARPS);
            } else {
                for (int r = ew; r < TC_BM; r += TC_STREAM_WARPS) {
                    const int64_t row = row0 + r;
                    if (row < p.N) stream_row(p, row, sh.top_key[b][r], cmax2, lane);
                    __syncwarp();
                    if (lane == 0) atomicAdd(&sh.rows_streamed, 1);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.lab_empty[b]));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync();   // neither CTA's shared memory or TMEM goes away under the other
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
        else tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ------------------------------------------------------------------ column-split inference kernel
//
// The bytes between a row's first read (TMA, for the MMA) and its second (the streaming warps)
// decide whether the second read still finds the row in L2, and they grow with the rows a CTA
// has in flight.  Here the CS CTAs of a cluster share ONE 128-row tile: CTA c stages columns
// [c D / CS, (c + 1) D / CS) of the rows and of ALL centroids and accumulates partial dot
// products (cta_group::1, M = 128, N = K) in its own TMEM.  The partial scores are then summed
// across the cluster through distributed shared memory: CTA c collects, for all 128 rows, the
// partials of centroids [c W, (c + 1) W), W = npad / CS, finds the four smallest keys among
// those, and sends them to the CTA that owns the row (rows [q 128 / CS, (q + 1) 128 / CS) belong
// to CTA q), which merges the CS lists and streams the row out.  Per CTA only 128 / CS rows'
// worth of bytes is in flight; the price is CS times the centroid bytes out of L2 per row.
// Its warp roles and register split are those of the row-tile kernel (three streaming warpgroups of
// 128 registers).  The streaming loop holds 24 float4 per lane in flight, which leaves 32 registers
// for everything else: the certainty test therefore runs in the score warps (one thread per row,
// from the row norms the streaming warps leave in shared memory), not in the streaming loop.  With
// the test inside the loop the compiler spilled there, and a spill in that loop doubles the
// kernel's run time.
constexpr int TCS_STREAM_WARPS = 12;
constexpr int TCS_THREADS = 32 * (TC_FIRST_STREAM_WARP + TCS_STREAM_WARPS);   // 640
constexpr int TCS_REGS_LAUNCH = 96;
constexpr int TCS_REGS_STREAM = 128;
static_assert(128 * (TC_REGS_CONTROL + TC_REGS_SCORE + (TCS_STREAM_WARPS / 4) * TCS_REGS_STREAM) <= TCS_REGS_LAUNCH * TCS_THREADS,
              "register split exceeds what the block is launched with");

struct TcSplitShared {
    uint64_t a_full[TC_MAX_A_STAGES];
    uint64_t a_empty[TC_MAX_A_STAGES];
    uint64_t b_full[TC_MAX_B_STAGES];
    uint64_t b_empty[TC_MAX_B_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t lab_full[2];
    uint64_t lab_empty[2];
    uint64_t x_full;              // the peers' partial scores of a tile have landed here
    uint64_t x_empty;             // the peers have read what this CTA sent them
    uint64_t k_full[2];           // the peers' keys of the rows this CTA owns have landed
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    int rows_streamed;
    float red[32];
    float cn[256];
    float4 top_key[2][TC_BM];     // merged keys of the rows this CTA owns (the first 128 / CS entries)
    float4 peer_key[2][TC_BM];    // [buffer][source CTA * (128 / CS) + row]
    float row_norm[2][TC_BM];     // ||y||^2 of the rows this CTA streamed, by the streaming warps
};

__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// arrival on a barrier of another CTA that publishes this thread's earlier (fenced) writes to it
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_acq_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded, warp-uniform wait on a barrier that CTAs of the cluster arrive on.
__device__ __forceinline__ bool mbar_wait_cluster_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, Control *ctl)
{
    bool ok = true;
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait_acq_cluster(bar, parity)) break;
        if (*abort_flag) { ok = false; break; }
        if ((it & 63u) == 63u) {
            uint64_t now = global_timer();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > TC_TIMEOUT_NS) {
                *abort_flag = 1;
                atomicExch(&ctl->device_status, (int)CAT_ERR_DEVICE_TIMEOUT);
                ok = false;
                break;
            }
        }
    }
    return __all_sync(0xffffffffu, ok);
}

template <int CS>
__global__ void __launch_bounds__(TCS_THREADS, 1)
apply_split_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcParams p)
{
    constexpr int RP = TC_BM / CS;                 // rows of a tile this CTA owns
    constexpr int OWNER_WARPS = TC_SCORE_WARPS / CS;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char *tiles = smem_raw + (tiles_base - raw);
    const int b_bytes = p.npad * 128;
    const int na = p.a_stages, nb = p.b_stages;
    const int W = p.npad / CS;                     // centroids this CTA reduces
    const uint32_t b_base = tiles_base + (uint32_t)(na * TC_A_BYTES);
    const uint32_t x_base = b_base + (uint32_t)(nb * b_bytes);          // [CS - 1][128][W] fp32, 16-byte chunks swizzled
    const int x_bytes = (CS - 1) * TC_BM * W * 4;
    unsigned char *x_ptr = tiles + (size_t)na * TC_A_BYTES + (size_t)nb * b_bytes;
    TcSplitShared &sh = *reinterpret_cast<TcSplitShared *>(x_ptr + x_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t crank = cluster_ctarank();
    volatile int *abort_flag = &sh.abort_flag;
    const int64_t num_units = (p.N + TC_BM - 1) / TC_BM;
    const int64_t unit_first = (int64_t)(blockIdx.x / CS);
    const int64_t unit_step = (int64_t)(gridDim.x / CS);
    const int nslabs = p.D / (32 * CS);            // slabs of this CTA's columns
    const int slab0 = (int)crank * nslabs;

    if (tid == 0) {
        for (int s = 0; s < na; ++s) {
            mbar_init(smem_u32(&sh.a_full[s]), 1);
            mbar_init(smem_u32(&sh.a_empty[s]), 1);
        }
        for (int s = 0; s < nb; ++s) {
            mbar_init(smem_u32(&sh.b_full[s]), 1);
            mbar_init(smem_u32(&sh.b_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh.tmem_full[b]), 1);
            mbar_init(smem_u32(&sh.tmem_empty[b]), TC_SCORE_WARPS);
            mbar_init(smem_u32(&sh.lab_full[b]), OWNER_WARPS);
            mbar_init(smem_u32(&sh.lab_empty[b]), TCS_STREAM_WARPS);
            mbar_init(smem_u32(&sh.k_full[b]), (CS - 1) * OWNER_WARPS);
        }
        mbar_init(smem_u32(&sh.x_full), (CS - 1) * TC_SCORE_WARPS);
        mbar_init(smem_u32(&sh.x_empty), (CS - 1) * TC_SCORE_WARPS);
        mbar_init(smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        sh.rows_streamed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
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
        tmem_alloc(smem_u32(&sh.tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();   // the peers' barriers exist before anything arrives on them
    tc_fence_after();
    float cmax2 = 0.f;
    for (int w2 = 0; w2 < (int)(blockDim.x >> 5); ++w2) cmax2 = fmaxf(cmax2, sh.red[w2]);
    const uint32_t tmem_base = sh.tmem_base;

    if (warp < TC_FIRST_SCORE_WARP) {
        setmaxnreg_dec<TC_REGS_CONTROL>();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer, row slabs
            if (lane == 0) {
                uint32_t ti = 0, ph = 0;
                int s = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
                    const int row0 = (int)(unit * TC_BM);
                    if (ti > 1) {
                        // at most one tile ahead of the streaming warps
                        if (!wait_progress(&sh.rows_streamed, (int)(ti - 1) * RP - RP / 2, abort_flag, p.ctl)) { ok = false; break; }
                    }
                    for (int sl = 0; sl < nslabs; ++sl) {
                        if (!mbar_wait(smem_u32(&sh.a_empty[s]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                        const uint32_t full = smem_u32(&sh.a_full[s]);
                        mbar_arrive_expect_tx(full, (uint32_t)TC_A_BYTES);
                        tma_load_2d(tiles_base + (uint32_t)(s * TC_A_BYTES), &mapA, full, (slab0 + sl) * 32, row0);
                        if (++s == na) { s = 0; ph ^= 1u; }
                    }
                }
                if (!ok) {
                    for (int s2 = 0; s2 < na; ++s2)
                        for (int tries = 0; tries < 100000; ++tries)
                            if (mbar_try_wait(smem_u32(&sh.a_full[s2]), 0) || mbar_try_wait(smem_u32(&sh.a_full[s2]), 1)) break;
                }
            }
        } else if (warp == 2) {
            // ------------------------------------------------------------ TMA producer, centroid slabs
            if (lane == 0) {
                uint32_t ph = 0;
                int s = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step) {
                    for (int sl = 0; sl < nslabs; ++sl) {
                        if (!mbar_wait(smem_u32(&sh.b_empty[s]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                        const uint32_t full = smem_u32(&sh.b_full[s]);
                        mbar_arrive_expect_tx(full, (uint32_t)b_bytes);
                        tma_load_2d(b_base + (uint32_t)(s * b_bytes), &mapB, full, (slab0 + sl) * 32, 0);
                        if (++s == nb) { s = 0; ph ^= 1u; }
                    }
                }
                if (!ok) {
                    for (int s2 = 0; s2 < nb; ++s2)
                        for (int tries = 0; tries < 100000; ++tries)
                            if (mbar_try_wait(smem_u32(&sh.b_full[s2]), 0) || mbar_try_wait(smem_u32(&sh.b_full[s2]), 1)) break;
                }
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------ MMA issuer
            if (lane == 0) {
                const uint32_t idesc = make_idesc(TC_BM, p.npad, 2u);
                int sa = 0, sb = 0;
                uint32_t pha = 0, phb = 0, ti = 0;
                bool ok = true;
                for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
                    const int b = ti & 1;
                    if (!mbar_wait(smem_u32(&sh.tmem_empty[b]), ((ti >> 1) & 1u) ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + (uint32_t)(b * p.npad);
                    for (int sl = 0; sl < nslabs; ++sl) {
                        if (!mbar_wait(smem_u32(&sh.b_full[sb]), phb, abort_flag, p.ctl)) { ok = false; break; }
                        if (!mbar_wait(smem_u32(&sh.a_full[sa]), pha, abort_flag, p.ctl)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t adesc = make_smem_desc(tiles_base + (uint32_t)(sa * TC_A_BYTES));
                        const uint64_t bdesc = make_smem_desc(b_base + (uint32_t)(sb * b_bytes));
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_tf32(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, (sl > 0 || kk > 0) ? 1u : 0u);
                        tc_commit(smem_u32(&sh.a_empty[sa]));
                        tc_commit(smem_u32(&sh.b_empty[sb]));
                        if (++sa == na) { sa = 0; pha ^= 1u; }
                        if (++sb == nb) { sb = 0; phb ^= 1u; }
                    }
                    if (ok) tc_commit(smem_u32(&sh.tmem_full[b]));
                }
                tc_commit(smem_u32(&sh.drain));
                for (int tries = 0; tries < 4000000; ++tries)
                    if (mbar_try_wait(smem_u32(&sh.drain), 0)) break;
            }
        }
    } else if (warp < TC_FIRST_STREAM_WARP) {
        // ------------------------------------------------------------ score warps
        setmaxnreg_dec<TC_REGS_SCORE>();
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;            // row of the tile = TMEM lane
        const uint32_t owner = (uint32_t)(r / RP);    // CTA that owns this row
        const uint32_t swz = (uint32_t)(r & 7);
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            if (!mbar_wait_warp(smem_u32(&sh.tmem_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * p.npad);
            uint32_t ra[16], rb[16];
            // ---- send: the peers' centroid ranges of this CTA's partial scores
            if (!mbar_wait_cluster_warp(smem_u32(&sh.x_empty), (ti & 1u) ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
#pragma unroll 1
            for (uint32_t d = 1; d < (uint32_t)CS; ++d) {
                const uint32_t q = (crank + d) % CS;                  // destination CTA
                const uint32_t slot = (crank + CS - q - 1) % CS;      // this CTA's place in q's buffer
                const uint32_t dst = mapa_cluster(x_base + (slot * TC_BM + (uint32_t)r) * (uint32_t)(W * 4), q);
                const uint32_t src = taddr + q * (uint32_t)W;
                tmem_ld16_issue(src, ra);
                for (int c = 0; c < W; c += 32) {
                    tmem_ld_wait16(ra);
                    tmem_ld16_issue(src + (uint32_t)(c + 16), rb);
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        st_cluster_v4(dst + ((((uint32_t)(c >> 2) + v) ^ swz) << 4), ra[4 * v], ra[4 * v + 1], ra[4 * v + 2], ra[4 * v + 3]);
                    tmem_ld_wait16(rb);
                    if (c + 32 < W) tmem_ld16_issue(src + (uint32_t)(c + 32), ra);
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        st_cluster_v4(dst + ((((uint32_t)(c >> 2) + 4 + v) ^ swz) << 4), rb[4 * v], rb[4 * v + 1], rb[4 * v + 2], rb[4 * v + 3]);
                }
                // (no separate fence: __syncwarp orders the lanes, the arrival below releases at cluster scope)
                __syncwarp();
                if (lane == 0) mbar_arrive_release_cluster(mapa_cluster(smem_u32(&sh.x_full), q));
            }
            // ---- reduce: own centroid range, own partials plus the peers'
            if (!mbar_wait_cluster_warp(smem_u32(&sh.x_full), ti & 1u, abort_flag, p.ctl)) { ok = false; break; }
            float b1 = TC_KEY_INIT, b2 = TC_KEY_INIT, b3 = TC_KEY_INIT, b4 = TC_KEY_INIT;
            {
                const int k0 = (int)crank * W;
                const uint32_t src = taddr + (uint32_t)k0;
#pragma unroll 1
                for (int c = 0; c < W; c += 16) {
                    tmem_ld16_issue(src + (uint32_t)c, ra);
                    // the peers' partials of these 16 centroids, read while the TMEM load is in flight
                    float acc[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) acc[j] = 0.f;
#pragma unroll
                    for (int slot = 0; slot < CS - 1; ++slot) {
                        const unsigned char *xr = x_ptr + ((size_t)slot * TC_BM + r) * (size_t)(W * 4);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            const float4 t = *reinterpret_cast<const float4 *>(xr + ((((uint32_t)(c >> 2) + v) ^ swz) << 4));
                            acc[4 * v] += t.x;
                            acc[4 * v + 1] += t.y;
                            acc[4 * v + 2] += t.z;
                            acc[4 * v + 3] += t.w;
                        }
                    }
                    tmem_ld_wait16(ra);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        key_insert(make_key(fmaf(-2.f, acc[j] + __uint_as_float(ra[j]), sh.cn[k0 + c + j]), k0 + c + j), b1, b2, b3, b4);
                }
            }
            // accumulator buffer b and the exchange buffer are free from here on
            tc_fence_before();
            // (no separate fence: __syncwarp orders the lanes, the arrival below releases at cluster scope)
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.tmem_empty[b]));
#pragma unroll 1
                for (uint32_t d = 1; d < (uint32_t)CS; ++d)
                    mbar_arrive_release_cluster(mapa_cluster(smem_u32(&sh.x_empty), (crank + d) % CS));
            }
            // ---- the four smallest keys of a row go to its owner, which merges the CS lists
            if (owner != crank) {
                const uint32_t dst = mapa_cluster(smem_u32(&sh.peer_key[b][crank * RP + (uint32_t)(r - (int)owner * RP)]), owner);
                st_cluster_v4(dst, __float_as_uint(b1), __float_as_uint(b2), __float_as_uint(b3), __float_as_uint(b4));
                // (no separate fence: __syncwarp orders the lanes, the arrival below releases at cluster scope)
                __syncwarp();
                if (lane == 0) mbar_arrive_release_cluster(mapa_cluster(smem_u32(&sh.k_full[b]), owner));
            } else {
                if (!mbar_wait_cluster_warp(smem_u32(&sh.k_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
                const int rl = r - (int)crank * RP;
#pragma unroll
                for (int d = 1; d < CS; ++d) {
                    const float4 t = sh.peer_key[b][((crank + d) % CS) * RP + rl];
                    key_insert(t.x, b1, b2, b3, b4);
                    key_insert(t.y, b1, b2, b3, b4);
                    key_insert(t.z, b1, b2, b3, b4);
                    key_insert(t.w, b1, b2, b3, b4);
                }
                if (!mbar_wait_warp(smem_u32(&sh.lab_empty[b]), ph ^ 1u, abort_flag, p.ctl)) { ok = false; break; }
                if (ti >= 2) {
                    // tile ti - 2 (same buffer) is streamed out: its row norms are in, its keys still here
                    const int64_t row = (unit - 2 * unit_step) * TC_BM + (int64_t)crank * RP + rl;
                    if (row < p.N) {
                        const float4 keys = sh.top_key[b][rl];
                        p.labels[row] = key_label(keys.x, p.K);
                        tc_decide(p, row, keys, tc_error_bound(p.D, sh.row_norm[b][rl] * 1.0001f, cmax2));
                    }
                }
                sh.top_key[b][rl] = make_float4(b1, b2, b3, b4);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.lab_full[b]));
            }
        }
        // the last two tiles are decided once the streaming warps are through with them
        if (ok && owner == crank) {
            const int rl = r - (int)crank * RP;
            for (uint32_t t = (ti >= 2 ? ti - 2 : 0); t < ti; ++t) {
                const int b = t & 1;
                if (!mbar_wait_warp(smem_u32(&sh.lab_empty[b]), (t >> 1) & 1u, abort_flag, p.ctl)) break;
                const int64_t row = (unit_first + (int64_t)t * unit_step) * TC_BM + (int64_t)crank * RP + rl;
                if (row < p.N) {
                    const float4 keys = sh.top_key[b][rl];
                    p.labels[row] = key_label(keys.x, p.K);
                    tc_decide(p, row, keys, tc_error_bound(p.D, sh.row_norm[b][rl] * 1.0001f, cmax2));
                }
            }
        }
    } else {
        // ------------------------------------------------------------ streaming warps
        setmaxnreg_inc<TCS_REGS_STREAM>();
        const int ew = warp - TC_FIRST_STREAM_WARP;
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t unit = unit_first; unit < num_units && ok; unit += unit_step, ++ti) {
            const int b = ti & 1;
            const uint32_t ph = (ti >> 1) & 1u;
            const int64_t row0 = unit * TC_BM + (int64_t)crank * RP;
            if (!mbar_wait_warp(smem_u32(&sh.lab_full[b]), ph, abort_flag, p.ctl)) { ok = false; break; }
            for (int rl = ew; rl < RP; rl += TCS_STREAM_WARPS) {
                const int64_t row = row0 + rl;
                if (row < p.N) {
                    const float ysq = stream_row_affine(p, row, key_label(sh.top_key[b][rl].x, p.K), lane);
                    if (lane == 0) sh.row_norm[b][rl] = ysq;
                }
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
    cluster_sync();   // no CTA's shared memory goes away while a peer may still write to it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// Squared row norms (labels-only mode), slightly over-estimated to keep the error bound on the safe
// side; with amax_bits also the largest magnitude of the matrix (as the bits of a non-negative float,
// which order like unsigned integers).  A row is read by G lanes, G = the power of two >= D / 4
// capped at 32, so short rows share a warp.
__global__ void row_norms_kernel(const float *__restrict__ Y, int64_t N, int D, int G, float *__restrict__ out,
                                 unsigned int *__restrict__ amax_bits)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t row = t / G;
    const int c0 = (int)(t % G);
    float s = 0.f, m = 0.f;
    if (row < N) {
        const float4 *y4 = reinterpret_cast<const float4 *>(Y + (size_t)row * D);
        const int D4 = D >> 2;
        for (int c = c0; c < D4; c += 8 * G) {   // eight loads in flight per lane
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int cc = c + u * G;
                v[u] = (cc < D4) ? __ldg(y4 + cc) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                s = fmaf(v[u].x, v[u].x, s);
                s = fmaf(v[u].y, v[u].y, s);
                s = fmaf(v[u].z, v[u].z, s);
                s = fmaf(v[u].w, v[u].w, s);
                m = fmaxf(fmaxf(m, fmaxf(fabsf(v[u].x), fabsf(v[u].y))), fmaxf(fabsf(v[u].z), fabsf(v[u].w)));
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        if (o < G) {
            s += __shfl_xor_sync(0xffffffffu, s, o);
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        }
    }
    if (row < N && c0 == 0) {
        out[row] = s * 1.0001f;
        if (amax_bits && m == m && m < CUDART_INF_F) atomicMax(amax_bits, __float_as_uint(m));
    }
}

// scale[0] = s_c, the power of two that brings the largest magnitude of the matrix (the bits
// left in scale[0] by the shadow kernel) to [2^13, 2^14); scale[1] = -2 / s_c (times 1 / row scale
// it turns the fp16 accumulator into -2 y.c); scale[2] = 2^-25 / s_c.
__global__ void half_scale_kernel(float *scale)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const float amax = __uint_as_float(reinterpret_cast<unsigned int *>(scale)[0]);
    int e = 0;
    if (amax > 0.f) frexpf(amax, &e);    // amax = f * 2^e, f in [0.5, 1)
    int sh = 14 - e;
    if (sh > 100) sh = 100;
    if (sh < -100) sh = -100;
    const float sc = ldexpf(1.f, sh);
    scale[0] = sc;
    scale[1] = -2.f / sc;
    scale[2] = 2.9802322e-8f / sc;
}

// One sweep over the rows: squared norm (slightly over-estimated), the row's own power-of-two
// scale s_i (largest magnitude to [2^13, 2^14)), rinv[i] = 1 / s_i, Yh[i, :] = fp16(Y[i, :] * s_i)
// rounded to nearest, and the largest magnitude of the matrix (float bits, one atomicMax per CTA).
// A row is handled by G lanes and read twice; the second read comes out of L1/L2.
__global__ void __launch_bounds__(256) half_shadow_kernel(const float *__restrict__ Y, int64_t N, int D, int G,
                                                          float *__restrict__ ynorm2, float *__restrict__ rinv,
                                                          unsigned int *__restrict__ amax_bits, __half *__restrict__ Yh)
{
    __shared__ float wmax[8];
    const int D4 = D >> 2;
    const int rows_per_cta = 256 / G;
    const int sub = threadIdx.x / G, c0 = threadIdx.x % G;
    float cta_max = 0.f;
    // The trip count is the same for every thread of the CTA (the shuffles below name all 32
    // lanes); a thread whose row lies beyond N goes through the loop with loads and stores off.
    for (int64_t base = (int64_t)blockIdx.x * rows_per_cta; base < N; base += (int64_t)gridDim.x * rows_per_cta) {
        const int64_t row = base + sub;
        const bool live = row < N;
        const float4 *y4 = reinterpret_cast<const float4 *>(Y + (size_t)(live ? row : 0) * D);
        float s = 0.f, m = 0.f;
        for (int c = c0; c < D4; c += 8 * G) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int cc = c + u * G;
                v[u] = (live && cc < D4) ? __ldg(y4 + cc) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                s = fmaf(v[u].x, v[u].x, s);
                s = fmaf(v[u].y, v[u].y, s);
                s = fmaf(v[u].z, v[u].z, s);
                s = fmaf(v[u].w, v[u].w, s);
                m = fmaxf(fmaxf(m, fmaxf(fabsf(v[u].x), fabsf(v[u].y))), fmaxf(fabsf(v[u].z), fabsf(v[u].w)));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            if (o < G) {
                s += __shfl_xor_sync(0xffffffffu, s, o);
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            }
        }
        int e = 0;
        if (m > 0.f && m < CUDART_INF_F) frexpf(m, &e);
        int sh = 14 - e;
        if (sh > 100) sh = 100;
        if (sh < -100) sh = -100;
        const float sc = ldexpf(1.f, sh);
        if (!live) continue;
        if (c0 == 0) {
            ynorm2[row] = s * 1.0001f;
            rinv[row] = ldexpf(1.f, -sh);
        }
        if (m == m && m < CUDART_INF_F) cta_max = fmaxf(cta_max, m);
        uint2 *h4 = reinterpret_cast<uint2 *>(Yh + (size_t)row * D);
        for (int c = c0; c < D4; c += G) {
            const float4 v = __ldg(y4 + c);
            const __half2 lo = __floats2half2_rn(v.x * sc, v.y * sc);
            const __half2 hi = __floats2half2_rn(v.z * sc, v.w * sc);
            uint2 o2;
            o2.x = *reinterpret_cast<const unsigned int *>(&lo);
            o2.y = *reinterpret_cast<const unsigned int *>(&hi);
            h4[c] = o2;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cta_max = fmaxf(cta_max, __shfl_xor_sync(0xffffffffu, cta_max, o));
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = cta_max;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t = fmaxf(t, wmax[w]);
        atomicMax(amax_bits, __float_as_uint(t));
    }
}

// dst = fp16(src * scale[0]), round to nearest; n4 = number of float4 groups
__global__ void to_half_kernel(const float4 *__restrict__ src, size_t n4, const float *__restrict__ scale,
                               uint2 *__restrict__ dst)
{
    const float sc = scale[0];
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const float4 v = __ldcs(src + i);
        const __half2 lo = __floats2half2_rn(v.x * sc, v.y * sc);
        const __half2 hi = __floats2half2_rn(v.z * sc, v.w * sc);
        uint2 o;
        o.x = *reinterpret_cast<const unsigned int *>(&lo);
        o.y = *reinterpret_cast<const unsigned int *>(&hi);
        dst[i] = o;
    }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever completes, with
// the given limit; the wait gives up, records CAT_ERR_DEVICE_TIMEOUT and the kernel returns.
__global__ void wait_selftest_kernel(Control *ctl, uint64_t limit_ns)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    {
        const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, ctl, limit_ns);
        (void)ok;
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// 2-D row-major [rows, D] of fp32 (or fp16) viewed in boxes of box_rows x 128 bytes, 128-byte
// swizzle, zero fill outside the matrix.
bool make_map(CUtensorMap *map, const void *base, bool half, int64_t rows, int D, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const size_t esz = half ? 2 : 4;
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * esz};
    cuuint32_t box[2] = {(cuuint32_t)(TC_SLAB_BYTES / esz), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, half ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                    const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The affine kernel re-divides its registers among its warpgroups; a division larger than
// what the block was launched with would wait forever, so it is checked here before launch.
bool regs_ok(const void *kern)
{
    cudaFuncAttributes a{};
    if (cudaFuncGetAttributes(&a, kern) != cudaSuccess) return false;
    return (long)a.numRegs * TC_THREADS_AFFINE >= 128L * (TC_REGS_CONTROL + TC_REGS_SCORE + 3 * TC_REGS_STREAM);
}

int lanes_per_row(int D)
{
    int G = 1;
    while (G < (D >> 2) && G < 32) G <<= 1;
    return G;
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

bool tc_make_map(CUtensorMap *map, const void *base, bool half, int64_t rows, int D, int box_rows)
{
    return make_map(map, base, half, rows, D, box_rows);
}

int tc_sm_count() { return sm_count(); }

bool tc_supported(int64_t N, int D, int K)
{
    return (D % 4 == 0) && D >= 4 && K <= 256 && N >= 1 && encode_fn() != nullptr;
}

cudaError_t launch_row_norms(const float *Y, int64_t N, int D, float *out, cudaStream_t s)
{
    const int threads = 256;
    const int G = lanes_per_row(D);
    const int64_t blocks = (N * G + threads - 1) / threads;
    row_norms_kernel<<<(unsigned)blocks, threads, 0, s>>>(Y, N, D, G, out, nullptr);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_half_shadow(const float *Y, int64_t N, int D, float *ynorm2, float *scale, void *Yh,
                               cudaStream_t s, bool finish_scale)
{
    float *rinv = scale + 4;
    cudaError_t e = cudaMemsetAsync(scale, 0, 4 * sizeof(float), s);
    if (e != cudaSuccess) return e;
    const int G = lanes_per_row(D);
    const int rows_per_cta = 256 / G;
    int64_t blocks = (N + rows_per_cta - 1) / rows_per_cta;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    half_shadow_kernel<<<(unsigned)blocks, 256, 0, s>>>(Y, N, D, G, ynorm2, rinv, reinterpret_cast<unsigned int *>(scale),
                                                        reinterpret_cast<__half *>(Yh));
    if (finish_scale) half_scale_kernel<<<1, 32, 0, s>>>(scale);
    count_launch(finish_scale ? 2 : 1);
    return cudaGetLastError();
}

cudaError_t launch_to_half(const float *src, size_t n, const float *scale, void *dst, cudaStream_t s)
{
    const int threads = 256;
    const size_t n4 = n / 4;
    size_t cb = (n4 + threads - 1) / threads;
    if (cb > (size_t)sm_count() * 16) cb = (size_t)sm_count() * 16;
    if (cb < 1) cb = 1;
    to_half_kernel<<<(unsigned)cb, threads, 0, s>>>(reinterpret_cast<const float4 *>(src), n4, scale,
                                                    reinterpret_cast<uint2 *>(dst));
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_wait_selftest(Control *ctl, int limit_ms, cudaStream_t s)
{
    if (limit_ms < 1) limit_ms = 1;
    if (limit_ms > 1000) limit_ms = 1000;
    wait_selftest_kernel<<<1, 32, 0, s>>>(ctl, (uint64_t)limit_ms * 1000000ull);
    count_launch();
    return cudaGetLastError();
}

// ---- column-split inference kernel: selection and launch
static std::atomic<int> g_apply_split{0};   // 0 = chosen here (row tiles at present), 1 = never, 2 / 4 = that cluster size where it applies

void set_apply_column_split(int cs) { g_apply_split.store((cs == 1 || cs == 2 || cs == 4 || cs == 64) ? cs : 0, std::memory_order_relaxed); }
int get_apply_column_split() { return g_apply_split.load(std::memory_order_relaxed); }

namespace {

struct SplitGeometry {
    int npad, a_stages, b_stages;
    size_t smem;
};

// false if a cluster of cs CTAs cannot take this shape
bool split_geometry(int cs, int64_t N, int D, int K, SplitGeometry *g)
{
    if (N <= TC_BM || D < 128 || D % (32 * cs) != 0) return false;
    const int unit = 32 * cs;
    g->npad = (K + unit - 1) / unit * unit;
    if (g->npad > 256) return false;
    g->b_stages = TC_AFFINE_B_STAGES;
    const size_t b_bytes = (size_t)g->npad * 128;
    const size_t x_bytes = (size_t)(cs - 1) * TC_BM * (g->npad / cs) * 4;
    const size_t fixed = 1024 + g->b_stages * b_bytes + x_bytes + sizeof(TcSplitShared);
    const size_t budget = 227 * 1024;
    if (fixed + 2 * TC_A_BYTES > budget) return false;
    int a = (int)((budget - fixed) / TC_A_BYTES);
    if (a > TC_AFFINE_A_STAGES) a = TC_AFFINE_A_STAGES;
    // the streaming warps need the L1 that a carve-out above 196 KB takes away: give up a stage for it
    const size_t soft = 195 * 1024;
    while (a > 2 && fixed + (size_t)a * TC_A_BYTES > soft) --a;
    g->a_stages = a;
    g->smem = fixed + (size_t)a * TC_A_BYTES;
    return true;
}

int choose_column_split(int64_t N, int D, int K)
{
    const int mode = g_apply_split.load(std::memory_order_relaxed);
    if (mode == 1) return 1;
    if (mode == 64) return apply_h64_supported(N, D, K) ? 64 : 1;
    SplitGeometry g;
    if (mode > 1) return split_geometry(mode, N, D, K, &g) ? mode : 1;
    // chosen here: 64-row tiles on fp16 operands for rows of about 1024 columns (measured: ahead of
    // the TF32 row tiles from D = 640 to D = 2048, behind them for shorter and for much longer rows)
    if (D >= 640 && D <= 2048 && N >= 4096 && apply_h64_supported(N, D, K)) return 64;
    return 1;
}

cudaError_t launch_apply_split(int cs, TcParams p, const float *C, cudaStream_t s)
{
    SplitGeometry g;
    if (!split_geometry(cs, p.N, p.D, p.K, &g)) return cudaErrorInvalidValue;
    p.npad = g.npad;
    int cols = 32;
    while (cols < 2 * p.npad) cols <<= 1;
    p.tmem_cols = cols;
    p.a_stages = g.a_stages;
    p.b_stages = g.b_stages;
    CUtensorMap mapA, mapB;
    if (!make_map(&mapA, p.Y, false, p.N, p.D, TC_BM) || !make_map(&mapB, C, false, p.K, p.D, p.npad))
        return cudaErrorInvalidValue;
    const void *kern = cs == 2 ? reinterpret_cast<const void *>(apply_split_kernel<2>)
                               : reinterpret_cast<const void *>(apply_split_kernel<4>);
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem)) != cudaSuccess) return e;
    {
        cudaFuncAttributes fa{};
        if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return cudaErrorInvalidValue;
        if ((long)fa.numRegs * TCS_THREADS < 128L * (TC_REGS_CONTROL + TC_REGS_SCORE + (TCS_STREAM_WARPS / 4) * TCS_REGS_STREAM))
            return cudaErrorLaunchOutOfResources;
    }

    cudaLaunchConfig_t cfg{};
    cfg.blockDim = dim3(TCS_THREADS, 1, 1);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // one resident cluster per cs SMs, as many as the device can hold at once
    int64_t clusters = sm_count() / cs;
    {
        cfg.gridDim = dim3((unsigned)(clusters * cs), 1, 1);
        int resident = 0;
        if (cudaOccupancyMaxActiveClusters(&resident, kern, &cfg) == cudaSuccess && resident > 0 && resident < clusters)
            clusters = resident;
    }
    const int64_t units = (p.N + TC_BM - 1) / TC_BM;
    if (units < clusters) clusters = units;
    cfg.gridDim = dim3((unsigned)(clusters * cs), 1, 1);
    if (cs == 2) e = cudaLaunchKernelEx(&cfg, apply_split_kernel<2>, mapA, mapB, p);
    else e = cudaLaunchKernelEx(&cfg, apply_split_kernel<4>, mapA, mapB, p);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

}  // namespace

int choose_apply_form(int64_t N, int D, int K) { return choose_column_split(N, D, K); }

cudaError_t launch_half_scale(float *scale, cudaStream_t s)
{
    half_scale_kernel<<<1, 32, 0, s>>>(scale);
    count_launch();
    return cudaGetLastError();
}

bool tc_half_supported(int64_t N, int D, int K)
{
    return tc_supported(N, D, K) && (D % 8 == 0);
}

cudaError_t launch_assign_tc(const float *Y, int64_t N, int D, int K, const float *C, const float *cnorm,
                             const float *ynorm2, int32_t *labels, int32_t *refine_rows,
                             int32_t *cand_rows, uint64_t *cand_list, Control *ctl,
                             const float *gamma, const float *beta, float *out, cudaStream_t s,
                             const void *Yh, const void *Ch, const float *scale, const FastOut *fast)
{
    TcParams p{};
    if (fast) p.fast = *fast;
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
    p.npad = (K + 31) / 32 * 32;
    int cols = 32;
    while (cols < 2 * p.npad) cols <<= 1;
    p.tmem_cols = cols;

    const bool affine = out != nullptr;
    const bool half = (Yh != nullptr) && !affine;
    p.scale = scale;
    if (affine) {
        const int cs = choose_column_split(N, D, K);
        if (cs == 2 || cs == 4) return launch_apply_split(cs, p, C, s);
    }
    // Two CTAs per 256 rows whenever there is more than one tile of rows.
    const bool pair = N > TC_BM;
    const int nb_rows = pair ? p.npad / 2 : p.npad;
    CUtensorMap mapA, mapB;
    if (half) {
        if (!make_map(&mapA, Yh, true, N, D, TC_BM) || !make_map(&mapB, Ch, true, K, D, nb_rows))
            return cudaErrorInvalidValue;
    } else {
        if (!make_map(&mapA, Y, false, N, D, TC_BM) || !make_map(&mapB, C, false, K, D, nb_rows))
            return cudaErrorInvalidValue;
    }

    // ring depths: the centroid ring is shallow (its slabs come out of L2), the row ring takes the rest
    const size_t b_bytes = (size_t)nb_rows * 128;
    const size_t smem_budget = 227 * 1024;
    int b_stages = affine ? TC_AFFINE_B_STAGES : 3;
    int a_stages = (int)((smem_budget - 1024 - sizeof(TcShared) - b_stages * b_bytes) / TC_A_BYTES);
    if (a_stages > TC_MAX_A_STAGES) a_stages = TC_MAX_A_STAGES;
    if (affine && a_stages > TC_AFFINE_A_STAGES) a_stages = TC_AFFINE_A_STAGES;
    if (a_stages < 2) return cudaErrorInvalidValue;
    p.a_stages = a_stages;
    p.b_stages = b_stages;
    const size_t smem = 1024 + (size_t)a_stages * TC_A_BYTES + (size_t)b_stages * b_bytes + sizeof(TcShared);
    // ask for no more shared memory than the kernel uses (the rest of the array serves as L1)
    const int carveout = (int)((smem * 100 + smem_budget - 1) / smem_budget);
    const int sms = sm_count();
    const unsigned threads = affine ? TC_THREADS_AFFINE : TC_THREADS_LABELS;
    unsigned grid = 1;
    if (pair) {
        const int64_t units = (N + 2 * TC_BM - 1) / (2 * TC_BM);
        const int64_t clusters = units < sms / 2 ? units : sms / 2;
        grid = (unsigned)(2 * clusters);
    }

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = pair ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // (the kernel starts with pdl_enter)
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;

    cudaError_t e;
#define CAT_TC_LAUNCH(AFF, PR, HF, SH)                                                                                      \
    do {                                                                                                               \
        auto kern = assign_tc_kernel<AFF, PR, HF, SH>;                                                                      \
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)   \
            return e;                                                                                                  \
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, carveout)) != cudaSuccess) \
            return e;                                                                                                  \
        if (AFF && !regs_ok(reinterpret_cast<const void *>(kern))) return cudaErrorLaunchOutOfResources;               \
        e = cudaLaunchKernelEx(&cfg, kern, mapA, mapB, p);                                                             \
    } while (0)
    if (affine && D < 128) {
        if (pair) CAT_TC_LAUNCH(true, true, false, true); else CAT_TC_LAUNCH(true, false, false, true);
    } else if (affine) {
        if (pair) CAT_TC_LAUNCH(true, true, false, false); else CAT_TC_LAUNCH(true, false, false, false);
    } else if (half) {
        if (pair) CAT_TC_LAUNCH(false, true, true, false); else CAT_TC_LAUNCH(false, false, true, false);
    } else {
        if (pair) CAT_TC_LAUNCH(false, true, false, false); else CAT_TC_LAUNCH(false, false, false, false);
    }
#undef CAT_TC_LAUNCH
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

}  // namespace cat
