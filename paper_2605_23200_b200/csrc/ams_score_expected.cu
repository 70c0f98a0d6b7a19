// Expected-attention scorer on the sm_100a tensor path.  For every query head r of a KV head's GQA
// group the caller gives the mean mu_r and the covariance Sigma_r of the head's future queries; the
// expected attention weight of key k_t under q ~ N(mu_r, Sigma_r) is exp(l_{r,t}) with
//     l_{r,t} = mu_r . k_t / sqrt(d) + k_t^T Sigma_r k_t / (2 d),
// and the score is (mean_r softmax_t(l_{r,.}) + eps) * |v_t|.
//
// k_expected_tc reads K once: a 128-token tile is the A operand (tokens on the TMEM lanes) and the
// group's covariance matrices, resident in shared memory, are the B operands, so that one
// tcgen05.mma chain per head leaves (Sigma_r k_t) of token t in the 128 columns of TMEM lane t.  The
// thread that owns the lane dots them with k_t (read from the same shared-memory tile); the mean term
// mu_r . k_t of the tile comes from one more warp (mma.sync on the same tile); the logit is stored and a
// running (max, sum of 2^x) kept per head.  The block shape and the pipeline are those of
// the window scorer: warp 0 feeds K tiles by TMA, warp 2 computes the mean terms, warps 1 and 3 issue the MMAs for the two
// pairs of accumulator slots, warps 4-19 are four consumer warpgroups (each taking 32 of a head's 128
// columns of every tile).  k_expected_final then streams V and the stored logits (16 bytes per token and head
// group of four) and writes the scores.  Every wait is bounded; on expiry the block reports
// AMS_ERR_TIMEOUT, drains its copies, frees its TMEM and returns.
#include <cuda.h>

#include "ams_common.cuh"
#include "ams_tc_ptx.cuh"
#include "ams_tc_tiles.cuh"

namespace ams {

using namespace tc;

namespace {

constexpr int kExHeads = 4; // query heads per launch: 4 x 128 accumulator columns are the whole TMEM

struct ExShared {
    unsigned long long kfull[kMaxStages], kempty[kMaxStages], tfull[kSlots], tempty[kSlots];
    unsigned long long cfull, cempty, done[2];
    float pacc[kSlots][3][128];       // the parts of a logit that the three other warpgroups computed, per slot
    float2 red[4][kExHeads];          // per warp of warpgroup rb: (max, sum of 2^(x - max)) of head rb
    float2 stat[kExHeads][128];       // running (max, sum) of head rb in every thread of warpgroup rb
    unsigned long long linfull[2], linempty[2];
    float lin[2][128][kExHeads];      // mean term of the logits of a tile's tokens, per head (log2 units), two tiles deep
    uint32_t tmem_base;
    int abort_flag;
    int tiles_lh, tpc;
    long long n_tiles;
};

__global__ void __launch_bounds__(kTcThreads, 1) k_expected_tc(DevParams p, const __grid_constant__ CUtensorMap k_map,
                                                               const __grid_constant__ CUtensorMap c_map)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ ExShared sh;
    __shared__ int prefix[1025];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_rb = p.ex_gc, NS = p.tc_stages; // one 128-column accumulator block per query head
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *Cs = base;                                   // [n_rb][2 halves][128 rows][128 B]
    unsigned char *Ks = Cs + (size_t)n_rb * kTileBytes;         // [NS][8-row group][2 halves][8 rows][128 B]
    volatile int *abort_flag = &sh.abort_flag;

    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) {
            mbar_init(smem_u32(&sh.kfull[i]), 1);
            mbar_init(smem_u32(&sh.kempty[i]), 19); // both issuers' commits, the mean-term warp and the sixteen consumer warps
        }
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(smem_u32(&sh.tfull[i]), 1);
            mbar_init(smem_u32(&sh.tempty[i]), 16);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&sh.linfull[i]), 1); mbar_init(smem_u32(&sh.linempty[i]), (uint32_t)(4 * n_rb)); }
        mbar_init(smem_u32(&sh.cfull), 1);
        mbar_init(smem_u32(&sh.cempty), 2); // both MMA issuers release the covariance blocks
        mbar_init(smem_u32(&sh.done[0]), 1);
        mbar_init(smem_u32(&sh.done[1]), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    const int hpb = p.tc_hpb, my_hs = p.H / hpb;
    const int my_h0 = blockIdx.x % my_hs, my_group = blockIdx.x / my_hs;
    tc_partition(p, gridDim.x / my_hs, prefix, &sh.tiles_lh, &sh.n_tiles, &sh.tpc);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;
    const int tiles_lh = sh.tiles_lh, tpc = sh.tpc;
    const long long g_begin = (long long)my_group * tpc;
    const long long g_end = (g_begin + tpc < sh.n_tiles) ? g_begin + tpc : sh.n_tiles;
    const long long g_span = g_end - g_begin;
    const float c_lin = kLog2e * 0.08838834764831845f; // log2(e) / sqrt(128)
    const float c_quad = kLog2e * (1.0f / 256.0f);     // log2(e) / (2 * 128)

    if (tiles_lh > 0 && g_begin < g_end) {
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            int kit = 0, seg = 0, issued = 0;
            bool ok = true;
            for (long long gv = 0; gv < g_span * hpb && ok;) {
                const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                const long long g = g_begin + gv % g_span;
                const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                ok = mbar_wait(smem_u32(&sh.cempty), (uint32_t)((seg & 1) ^ 1), abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_expect_tx(smem_u32(&sh.cfull), (uint32_t)(n_rb * kTileBytes));
                    const int crow0 = ((((s.l * p.B + s.b) * p.H + s.h) * p.G) + p.ex_g0) * kHeadDim;
                    for (int rb = 0; rb < n_rb; ++rb)
                        for (int hf = 0; hf < 2; ++hf)
                            tma_load_2d(smem_u32(Cs + (size_t)rb * kTileBytes + hf * kHalfBytes), &c_map, smem_u32(&sh.cfull),
                                        hf * 64, crow0 + rb * kHeadDim);
                }
                const int *table = p.block_table + (size_t)s.b * p.bt_stride;
                const int last_page = (s.T - 1) >> 4;
                for (int i = 0; i < s.n && ok; ++i, ++kit) {
                    const int st = kit % NS;
                    ok = mbar_wait(smem_u32(&sh.kempty[st]), (uint32_t)(((kit / NS) & 1) ^ 1), abort_flag);
                    if (!ok) break;
                    if (lane == 0) mbar_expect_tx(smem_u32(&sh.kfull[st]), (uint32_t)kTileBytes);
                    __syncwarp();
                    if (lane < 8) {
                        const int pg = lane;
                        int pi = (s.tile0 + i) * 8 + pg;
                        if (pi > last_page) pi = last_page; // tokens past the end are dropped by position
                        tma_load_5d(smem_u32(Ks + (size_t)st * kTileBytes + pg * 4096), &k_map, smem_u32(&sh.kfull[st]), 0, 0, 2 * s.h, 0,
                                    s.l * (int)p.num_pages + table[pi]);
                    }
                    issued = kit + 1;
                }
                gv += s.n;
                ++seg;
            }
            if (!ok) { // drain: wait (bounded) for the copies that were issued and never consumed
                for (int k = max(0, issued - NS); k < issued; ++k) {
                    for (uint32_t i = 0; i < kWaitLimit; ++i)
                        if (mbar_try_wait(smem_u32(&sh.kfull[k % NS]), (uint32_t)((k / NS) & 1))) break;
                }
            }
        } else if (warp == 1 || warp == 3) {
            // ------------------------------------------------------------ MMA issuers (two heads of every tile each)
            if (lane == 0) {
                const int wg = warp >> 1;
                int kit = 0, seg = 0;
                bool ok = true;
                for (long long gv = 0; gv < g_span * hpb && ok;) {
                    const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                    const long long g = g_begin + gv % g_span;
                    const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                    ok = mbar_wait(smem_u32(&sh.cfull), (uint32_t)(seg & 1), abort_flag);
                    for (int i = 0; i < s.n && ok; ++i, ++kit) {
                        const int st = kit % NS;
                        ok = mbar_wait(smem_u32(&sh.kfull[st]), (uint32_t)((kit / NS) & 1), abort_flag);
                        // Head rb of every tile goes to accumulator slot rb; this issuer fills slots 2 wg and 2 wg + 1, so
                        // it sees every phase of their barriers in order (a parity wait must not skip a phase), and the
                        // tensor pipe may run a whole tile ahead of the consumers.
                        for (int rb = 2 * wg; rb < n_rb && rb < 2 * wg + 2 && ok; ++rb) {
                            const int slot = rb;
                            ok = mbar_wait(smem_u32(&sh.tempty[slot]), (uint32_t)((kit & 1) ^ 1), abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                            const uint32_t ca = smem_u32(Cs + (size_t)rb * kTileBytes), ka = smem_u32(Ks + (size_t)st * kTileBytes);
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const unsigned long long dc = smem_desc(ca + (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32), 1024);
                                const unsigned long long dk = smem_desc(ka + (uint32_t)((k >> 2) * 1024 + (k & 3) * 32), 2048);
                                tc_mma(tmem_base + (uint32_t)(slot * 128), dk, dc, kIdesc, k > 0); // D[t][j] = sum_i K[t][i] C[j][i]
                            }
                            tc_commit(smem_u32(&sh.tfull[slot]));
                        }
                        if (ok) tc_commit(smem_u32(&sh.kempty[st]));
                    }
                    if (ok) tc_commit(smem_u32(&sh.cempty));
                    gv += s.n;
                    ++seg;
                }
                tc_commit(smem_u32(&sh.done[wg]));
                for (uint32_t i = 0; i < kWaitLimit; ++i)
                    if (mbar_try_wait(smem_u32(&sh.done[wg]), 0)) break;
            }
            __syncwarp();
        } else if (warp == 2) {
            // ------------------------------------------------------------ mean-term warp
            // mu_r . k_t for the tile's 128 tokens and the launch's heads with mma.sync (m16n8k16, fp32 accumulate):
            // A = 16 token rows of the K tile (ldmatrix from the swizzled tile), B = eight columns, two per head:
            // mu_r rounded to bf16 and the bf16 of what the rounding lost, so that their sum carries mu_r to 2^-17.
            int kit = 0;
            bool ok = true;
            for (long long gv = 0; gv < g_span * hpb && ok;) {
                const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                const long long g = g_begin + gv % g_span;
                const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                unsigned breg[8][2];
                {
                    const int head = lane >> 3, lost = (lane >> 2) & 1; // column n = lane / 4 = 2 * head + lost
                    const float *mu_g = p.q_mean + ((size_t)s.uid * p.G + p.ex_g0 + head) * kHeadDim;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
#pragma unroll
                        for (int hb = 0; hb < 2; ++hb) {
                            const int k0 = ks * 16 + hb * 8 + (lane & 3) * 2;
                            const float x0 = head < n_rb ? mu_g[k0] : 0.0f, x1 = head < n_rb ? mu_g[k0 + 1] : 0.0f;
                            __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
                            if (lost) {
                                h0 = __float2bfloat16_rn(x0 - __bfloat162float(h0));
                                h1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
                            }
                            breg[ks][hb] = (unsigned)__bfloat16_as_ushort(h0) | ((unsigned)__bfloat16_as_ushort(h1) << 16);
                        }
                }
                for (int i = 0; i < s.n && ok; ++i, ++kit) {
                    const int st = kit % NS, lb = kit & 1;
                    ok = mbar_wait(smem_u32(&sh.kfull[st]), (uint32_t)((kit / NS) & 1), abort_flag);
                    if (ok) ok = mbar_wait(smem_u32(&sh.linempty[lb]), (uint32_t)(((kit >> 1) & 1) ^ 1), abort_flag);
                    ok = __all_sync(0xffffffffu, ok) != 0; // (also brings the lanes back together before ldmatrix)
                    if (!ok) break;
                    const uint32_t ka = smem_u32(Ks + (size_t)st * kTileBytes);
                    // eight blocks of 16 tokens, their accumulators independent of one another
                    float c[8][4];
#pragma unroll
                    for (int mb = 0; mb < 8; ++mb) c[mb][0] = c[mb][1] = c[mb][2] = c[mb][3] = 0.0f;
                    const int row = lane & 15; // row of the block whose address this lane supplies to ldmatrix
                    const uint32_t rbase = ka + (uint32_t)((row >> 3) * 2048 + (row & 7) * 128);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const int c16 = ks * 2 + (lane >> 4); // 16-byte chunk of the row: dims [8 c16, 8 c16 + 8)
                        const uint32_t coff = (uint32_t)((c16 >> 3) * 1024 + (((c16 & 7) ^ (row & 7)) << 4));
#pragma unroll
                        for (int mb = 0; mb < 8; ++mb) {
                            unsigned a0, a1, a2, a3;
                            asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(rbase + coff + (uint32_t)(mb * 4096)));
                            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                                         : "+f"(c[mb][0]), "+f"(c[mb][1]), "+f"(c[mb][2]), "+f"(c[mb][3])
                                         : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(breg[ks][0]), "r"(breg[ks][1]));
                        }
                    }
                    // this lane holds, for rows lane / 4 and lane / 4 + 8 of each block, both columns of head lane % 4
#pragma unroll
                    for (int mb = 0; mb < 8; ++mb) {
                        sh.lin[lb][mb * 16 + (lane >> 2)][lane & 3] = (c[mb][0] + c[mb][1]) * c_lin;
                        sh.lin[lb][mb * 16 + (lane >> 2) + 8][lane & 3] = (c[mb][2] + c[mb][3]) * c_lin;
                    }
                    __syncwarp();
                    if (lane == 0) { mbar_arrive(smem_u32(&sh.linfull[lb])); mbar_arrive(smem_u32(&sh.kempty[st])); }
                }
                gv += s.n;
            }
        } else if (warp >= 4) {
            // ------------------------------------------------------------ consumers
            // Four warpgroups work on every tile together: thread li of warpgroup q owns TMEM lane li (token
            // t0 + li) and columns [32 q, 32 q + 32) of each head's accumulator.  Its 32 key elements are widened
            // to fp32 once per tile and serve all heads.  Head rb of a tile is in accumulator slot rb.
            const int q4 = (warp - 4) >> 2, quad = warp & 3, li = quad * 32 + lane;
            int kit = 0, seg = 0;
            bool ok = true;
            for (long long gv = 0; gv < g_span * hpb;) {
                const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                const long long g = g_begin + gv % g_span;
                const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                const int T = s.T;
                if (q4 < kExHeads) sh.stat[q4][li] = make_float2(-INFINITY, 0.0f); // warpgroup rb keeps the statistics of head rb
                asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
                float *lg_out = p.ex_logits + ((size_t)s.uid * p.G + p.ex_g0) * p.T_cap;
                // A thread whose wait ran out keeps walking tiles and heads without touching the pipeline: the named
                // barriers below have no time limit, so every consumer thread must reach each of them.
                for (int i = 0; i < s.n; ++i, ++kit) {
                    const int t0 = (s.tile0 + i) * kTileTokens;
                    const int st = kit % NS, lb = kit & 1;
                    unsigned long long kf[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) kf[j] = 0ull;
                    if (ok) ok = mbar_wait(smem_u32(&sh.kfull[st]), (uint32_t)((kit / NS) & 1), abort_flag);
                    if (ok) {
                        // this thread's quarter of its token's key: four 16-byte chunks, un-swizzled by the row number
                        const uint32_t row = smem_u32(Ks) + (uint32_t)(st * kTileBytes + (li >> 3) * 2048 + (q4 >> 1) * 1024 + (li & 7) * 128);
#pragma unroll
                        for (int cch = 0; cch < 4; ++cch) {
                            uint4 v;
                            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                         : "r"(row + (uint32_t)((((q4 & 1) * 4 + cch) ^ (li & 7)) << 4)));
                            kf[4 * cch] = pack_f32x2(bf16_lo(v.x), bf16_hi(v.x));
                            kf[4 * cch + 1] = pack_f32x2(bf16_lo(v.y), bf16_hi(v.y));
                            kf[4 * cch + 2] = pack_f32x2(bf16_lo(v.z), bf16_hi(v.z));
                            kf[4 * cch + 3] = pack_f32x2(bf16_lo(v.w), bf16_hi(v.w));
                        }
                    }
                    __syncwarp();
                    if (ok && lane == 0) mbar_arrive(smem_u32(&sh.kempty[st]));
                    // the mean terms of this tile (warp 2); warpgroup rb reads those of head rb
                    if (ok && q4 < n_rb) ok = mbar_wait(smem_u32(&sh.linfull[lb]), (uint32_t)((kit >> 1) & 1), abort_flag);
                    float my_part = 0.0f; // this warpgroup's quarter of its own head (head q4), until the others' parts are in
                    for (int rb = 0; rb < n_rb; ++rb) {
                        const int slot = rb;
                        float val = 0.0f;
                        if (ok) ok = mbar_wait(smem_u32(&sh.tfull[slot]), (uint32_t)(kit & 1), abort_flag);
                        ok = __all_sync(0xffffffffu, ok) != 0; // one answer per warp: the accumulator loads below are warp-wide
                        if (ok) {
                            tc_fence_after();
                            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * 128 + q4 * 32);
                            uint32_t d[32];
                            tc_ld32_issue(taddr, d);
                            tc_ld_wait(d);
                            unsigned long long aq2 = 0ull;
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                aq2 = fma_f32x2(pack_f32x2(__uint_as_float(d[2 * j]), __uint_as_float(d[2 * j + 1])), kf[j], aq2);
                            val = sum_f32x2(aq2) * c_quad; // this quarter's part of the quadratic term, in log2 units
                        }
                        // The four quarters of the columns meet in warpgroup rb (the heads take turns, so that the extra work is
                        // spread): the others leave their parts in the slot's buffer and arrive at the slot's named barrier, warpgroup
                        // rb waits there, adds and stores, and releases the slot only after reading the buffer, so the next use of
                        // the slot cannot overwrite it early.  It does so one head late, after delivering its part of head rb + 1:
                        // otherwise every head would wait for the warpgroup that has just added up the one before.
                        if (q4 != rb) {
                            sh.pacc[slot][q4 < rb ? q4 : q4 - 1][li] = val;
                            tc_fence_before();
                            asm volatile("bar.arrive %0, %1;" ::"r"(2 + slot), "n"(kConsumerThreads) : "memory");
                            if (ok && lane == 0) mbar_arrive(smem_u32(&sh.tempty[slot]));
                        } else {
                            my_part = val;
                        }
                        if (q4 < n_rb && (rb == q4 + 1 || (rb == q4 && rb == n_rb - 1))) {
                            // this warpgroup's own head: slot q4
                            asm volatile("bar.sync %0, %1;" ::"r"(2 + q4), "n"(kConsumerThreads) : "memory");
                            if (ok) {
                                const float lg2 = my_part + (sh.pacc[q4][0][li] + sh.pacc[q4][1][li]) + (sh.pacc[q4][2][li] + sh.lin[lb][li][q4]);
                                const int t = t0 + li;
                                if (t < T) {
                                    lg_out[(size_t)q4 * p.T_cap + t] = lg2;
                                    const float2 mz = sh.stat[q4][li];
                                    const float mn = fmaxf(mz.x, lg2);
                                    sh.stat[q4][li] = make_float2(mn, mz.y * ex2(mz.x - mn) + ex2(lg2 - mn));
                                }
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) { mbar_arrive(smem_u32(&sh.tempty[q4])); mbar_arrive(smem_u32(&sh.linempty[lb])); }
                            }
                        }
                    }
                }
                // fold each head's statistics (warpgroup rb, its four warps in a fixed order) and store this block's part of the unit
                {
                    float mm = sh.stat[q4][li].x, zz = sh.stat[q4][li].y;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const float m2 = __shfl_xor_sync(0xffffffffu, mm, o), z2 = __shfl_xor_sync(0xffffffffu, zz, o);
                        lse_merge(mm, zz, m2, z2);
                    }
                    if (lane == 0) sh.red[quad][q4] = make_float2(mm, zz);
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
                if (warp == 4 && lane < n_rb && ok) {
                    float mm = -INFINITY, zz = 0.0f;
                    for (int w = 0; w < 4; ++w) lse_merge(mm, zz, sh.red[w][lane].x, sh.red[w][lane].y);
                    reinterpret_cast<float2 *>(p.part)[((size_t)s.uid * p.n_slices + s.part) * p.G + p.ex_g0 + lane] = make_float2(mm, zz);
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); // the buffer is free again
                gv += s.n;
                ++seg;
            }
        }
    }
    if (*abort_flag && tid == 0) set_status(p.status, AMS_ERR_TIMEOUT, blockIdx.x, 3, 0);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

constexpr int kFinThreads = 256; // 16 token rows x 16 lanes of 16 bytes
constexpr int kFinSlice = 2048;  // tokens per block: long enough to pay for merging the unit's statistics first

// score_t = (mean over the group's heads of 2^(l_{r,t} - b_r) + eps) * |v_t|, b_r = M_r + log2 Z_r merged from the
// parts the blocks of the first kernel left (an unused part is all zero).
__global__ void __launch_bounds__(kFinThreads) k_expected_final(DevParams p)
{
    __shared__ float b_s[16];
    wait_for_previous_kernel(); // logits and statistics
    const int uid = blockIdx.y, slice = blockIdx.x;
    const int h = uid % p.H, b = (uid / p.H) % p.B, l = uid / (p.H * p.B);
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int t_begin = slice * kFinSlice;
    if (t_begin >= T) return;
    const int t_end = min(T, t_begin + kFinSlice);
    // warp w merges the parts of heads w, w + 8, ...: one part per lane (their loads in flight together), then a
    // fixed tree over the lanes
    for (int hd = threadIdx.x >> 5; hd < p.G; hd += kFinThreads / 32) {
        float mm = -INFINITY, zz = 0.0f;
        for (int q = threadIdx.x & 31; q < p.n_slices; q += 32) {
            const float2 v = __ldcg(reinterpret_cast<const float2 *>(p.part) + ((size_t)uid * p.n_slices + q) * p.G + hd);
            if (v.y > 0.0f) tc::lse_merge(mm, zz, v.x, v.y);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mm, o), z2 = __shfl_xor_sync(0xffffffffu, zz, o);
            tc::lse_merge(mm, zz, m2, z2);
        }
        if ((threadIdx.x & 31) == 0) b_s[hd] = zz > 0.0f ? mm + log2f(zz) : INFINITY;
    }
    __syncthreads();
    const int lane = threadIdx.x & 15, r = threadIdx.x >> 4;
    const int *table = p.block_table + (size_t)b * p.bt_stride;
    const float *lg = p.ex_logits + (size_t)uid * p.G * p.T_cap;
    const float my_b = lane < p.G ? b_s[lane] : INFINITY;
    const float inv_g = 1.0f / (float)p.G;
    float *g_out = p.scores + (size_t)uid * p.T_cap;
    constexpr int kU = 4; // tokens per thread and round: their loads are issued together
    const int n_iter = (t_end - t_begin + 16 * kU - 1) / (16 * kU);
    for (int it = 0; it < n_iter; ++it) {
        uint4 v[kU];
        float e[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int t = t_begin + (it * kU + u) * 16 + r;
            v[u] = make_uint4(0, 0, 0, 0);
            e[u] = -INFINITY;
            if (t < t_end) {
                v[u] = ld_stream16(p.v_pages + row_offset(p, l, table[t >> 4], t & 15, h) + lane * 8);
                if (lane < p.G) e[u] = __ldcs(lg + (size_t)lane * p.T_cap + t);
            }
        }
        float a[2 * kU]; // a[2u]: this lane's part of |v|^2 of token u; a[2u + 1]: its head's attention weight
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            unsigned long long sq2 = 0ull;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const unsigned long long x2 = pack_f32x2(bf16_lo(w[i]), bf16_hi(w[i]));
                sq2 = fma_f32x2(x2, x2, sq2);
            }
            a[2 * u] = sum_f32x2(sq2);
            a[2 * u + 1] = tc::ex2(e[u] - my_b); // lanes beyond the group: 2^(-inf) = 0
        }
        // sums over the 16 lanes of a token row, all eight values at once: at each step a lane hands half of
        // its values to its partner and keeps the other half
#pragma unroll
        for (int o = 8, n = 2 * kU; o >= 2; o >>= 1, n >>= 1) {
            const bool up = (lane & o) != 0;
#pragma unroll
            for (int i = 0; i < n / 2; ++i) {
                const float send = up ? a[i] : a[i + n / 2];
                const float keep = up ? a[i + n / 2] : a[i];
                a[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
        }
        a[0] += __shfl_xor_sync(0xffffffffu, a[0], 1);
        // lane holds value index 4 * bit3 + 2 * bit2 + bit1: even = |v|^2 of token (index / 2), odd = its weight sum
        const float other = __shfl_xor_sync(0xffffffffu, a[0], 2);
        if ((lane & 3) == 0) {
            const int u = lane >> 2;
            const int t = t_begin + (it * kU + u) * 16 + r;
            if (t < t_end) g_out[t] = fmaf(other, inv_g, p.score_eps) * sqrtf(a[0]);
        }
    }
}

} // namespace

bool expected_supported(const DevParams &p) { return p.G >= 1 && p.G <= 16 && p.B <= 1024 && p.H <= 64; }

int launch_score_expected(const DevParams &p_in, LaunchCtx &ctx)
{
    DevParams p = p_in;
    if (!p.q_mean || !p.q_cov || !p.ex_logits) return AMS_ERR_INVALID_ARG;
    if (!expected_supported(p)) return AMS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return AMS_ERR_CUDA;
    CUtensorMap k_map, c_map;
    int rc = make_k_map(p, enc, &k_map);
    if (rc == AMS_OK) rc = make_rows_map(p.q_cov, (unsigned long long)p.L * p.B * p.H * p.G * kHeadDim, enc, &c_map);
    if (rc != AMS_OK) return rc;
    const int n_sm = sm_count();
    if (n_sm <= 0) return AMS_ERR_CUDA;
    const TcGrid tg = tc_grid(p, n_sm);
    p.tc_hpb = tg.hpb;
    // unused parts of the statistics must read as empty
    const size_t U = (size_t)p.L * p.B * p.H;
    if (cudaMemsetAsync(p.part, 0, U * p.n_slices * p.G * sizeof(float2), ctx.s) != cudaSuccess) return AMS_ERR_CUDA;
    static SmemGrant grant;
    for (int g0 = 0; g0 < p.G; g0 += kExHeads) {
        p.ex_g0 = g0;
        p.ex_gc = p.G - g0 < kExHeads ? p.G - g0 : kExHeads;
        // an even ring depth: each stage then belongs to one of the two MMA issuers
        p.tc_stages = p.ex_gc <= 2 ? 4 : 2;
        const size_t smem = 1024 + (size_t)(p.ex_gc + p.tc_stages) * kTileBytes + 256;
        if (!grant_dynamic_smem(k_expected_tc, smem, grant)) return AMS_ERR_CUDA;
        k_expected_tc<<<tg.grid, kTcThreads, smem, ctx.s>>>(p, k_map, c_map);
        ctx.mark(kKernScore1);
    }
    const dim3 grid((unsigned)((p.T_cap + kFinSlice - 1) / kFinSlice), (unsigned)U);
    if (launch_after(k_expected_final, grid, dim3(kFinThreads), 0, ctx.s, p) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernScore2);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

} // namespace ams
