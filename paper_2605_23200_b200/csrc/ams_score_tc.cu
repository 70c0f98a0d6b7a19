// TOVA-style scorer for wide observation windows (rows = G * W >= 64) on the sm_100a
// tensor path: tcgen05.mma with TMEM accumulators, operands staged by TMA.
//
// Work is the concatenation of all units' 128-token tiles; a group of blocks of a persistent grid
// takes the contiguous tile range [g * tpc, (g + 1) * tpc) for all KV heads (one or more heads per block).  Inside a block:
//   warp 0      TMA producer: query block of the current unit, then one 32 KB K tile per
//               stage (eight 16-token pages, one 4 KB copy each, 128-byte swizzle);
//   warps 1, 3  MMA issuers (one lane each, one per pair of consumer warpgroups, tiles in
//               turn): per (tile, 128-row query block) eight tcgen05.mma m128 n128 k16 into
//               one of four 128-column TMEM slots (two per pair, used in turn);
//   warps 4-19  four consumer warpgroups in two pairs, the pairs alternating tiles; thread i
//               of either warpgroup of a pair owns TMEM lane i of the pair's slots, the
//               first warpgroup taking columns [0, 64) and the second [64, 128).  (Two
//               warpgroups alone left each scheduler with two dependent instruction streams
//               and the accumulators waiting for them; four hide that latency.)
// Phase 1 puts query rows on the TMEM lanes (A = Q, B = K), so a thread folds its row's
// logits into a running (max, sum of 2^x) without leaving registers; phase 2 puts tokens
// on the lanes (A = K, B = Q), so a thread sums 2^(x - b_r) over the query rows of its
// token (the two halves of the rows meet through shared memory).  Both operands are K-major 128-byte-swizzled tiles, so the same shared-memory
// tiles serve either role.  Every wait is bounded; on expiry the block reports
// AMS_ERR_TIMEOUT, drains its copies, frees its TMEM and returns.
#include <cuda.h>

#include "ams_common.cuh"
#include "ams_tc_ptx.cuh"
#include "ams_tc_tiles.cuh"

namespace ams {

using namespace tc;

namespace {

struct TcShared {
    unsigned long long kfull[kMaxStages], kempty[kMaxStages], tfull[kSlots], tempty[kSlots];
    unsigned long long qfull, qempty, done[2];
    unsigned long long pfull[2][2];                  // usage pass: second half's partial sums are in pacc[pair][slot bit]
    float pacc[2][2][128];
    uint32_t tmem_base;
    int abort_flag;
    float wmax[2][16];
    int tiles_lh, tpc;
    long long n_tiles;
};

template <int PHASE>
__global__ void __launch_bounds__(kTcThreads, 1) k_tova_tc(DevParams p, const __grid_constant__ CUtensorMap k_map,
                                                           const __grid_constant__ CUtensorMap q_map)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ TcShared sh;
    __shared__ int prefix[1025];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_rb = p.rows_pad / 128, NS = p.tc_stages;
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *Qs = base;                                   // [n_rb][2 halves][128 rows][128 B]
    unsigned char *Ks = Qs + (size_t)n_rb * kTileBytes;         // [NS][2 halves][128 rows][128 B]
    float *fin_s = reinterpret_cast<float *>(Ks + (size_t)NS * kTileBytes);   // [2][rows_pad]
    float2 *red = reinterpret_cast<float2 *>(fin_s + 2 * p.rows_pad);         // [3][n_rb][128]
    volatile int *abort_flag = &sh.abort_flag;

    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(smem_u32(&sh.kfull[i]), 1); mbar_init(smem_u32(&sh.kempty[i]), 1); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(smem_u32(&sh.tfull[i]), 1); mbar_init(smem_u32(&sh.tempty[i]), 8); }
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&sh.pfull[i >> 1][i & 1]), 4);
        mbar_init(smem_u32(&sh.qfull), 1);
        mbar_init(smem_u32(&sh.qempty), 2); // both MMA issuers release the query block
        mbar_init(smem_u32(&sh.done[0]), 1);
        mbar_init(smem_u32(&sh.done[1]), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // A group of H / tc_hpb blocks walks one range of token tiles; block j of the group takes KV heads
    // j, j + H / tc_hpb, ... one after the other over that range (tc_hpb > 1 where H alone does not divide
    // the SM count well: 148 SMs and 8 heads give 18 groups of 8 blocks, or 37 groups of 4 with two heads each).
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
    const long long g_span = g_end - g_begin; // the loops below run over hpb * g_span tiles: head after head
    if (PHASE == 1 && blockIdx.x == 0 && tid == 0) {
        for (int b = 0; b < p.B; ++b) {
            const int T = p.seq_lens[b];
            if (T > p.Tk && T <= p.T_cap && p.W > T) set_status(p.status, AMS_ERR_INVALID_ARG, b, p.W, T);
        }
    }
    const float c = kLog2e * 0.08838834764831845f; // log2(e) / sqrt(128)

    if (tiles_lh > 0 && g_begin < g_end) {
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            int kit = 0, seg = 0, issued = 0;
            bool ok = true;
            for (long long gv = 0; gv < g_span * hpb && ok;) {
                const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                const long long g = g_begin + gv % g_span;
                const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                ok = mbar_wait(smem_u32(&sh.qempty), (uint32_t)((seg & 1) ^ 1), abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_expect_tx(smem_u32(&sh.qfull), (uint32_t)(n_rb * kTileBytes));
                    const int qrow0 = ((s.l * p.B + s.b) * p.H * p.G + s.h * p.G) * p.W;
                    for (int rb = 0; rb < n_rb; ++rb)
                        for (int hf = 0; hf < 2; ++hf)
                            tma_load_2d(smem_u32(Qs + (size_t)rb * kTileBytes + hf * kHalfBytes), &q_map, smem_u32(&sh.qfull),
                                        hf * 64, qrow0 + rb * 128);
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
                        // one copy per page: both 64-wide halves of this head's 16 rows (4 KB)
                        const int pg = lane;
                        int pi = (s.tile0 + i) * 8 + pg;
                        if (pi > last_page) pi = last_page;  // tokens past the end are masked by position
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
            // ------------------------------------------------------------ MMA issuers
            // One thread per consumer pair, taking the tiles in turn: a tile costs its issuer a
            // chain of long waits (two barriers, eight MMAs, two commits) that is longer than the
            // tile's share of the HBM stream, so a single issuer would be the bottleneck.
            if (lane == 0) {
                const int wg = warp >> 1; // issuer 0 feeds consumer pair 0 (even tiles), issuer 1 pair 1
                int kit = 0, seg = 0, wsit = 0; // wsit: accumulator slots handed to the warpgroup so far
                bool ok = true;
                for (long long gv = 0; gv < g_span * hpb && ok;) {
                const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                const long long g = g_begin + gv % g_span;
                    const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                    ok = mbar_wait(smem_u32(&sh.qfull), (uint32_t)(seg & 1), abort_flag);
                    for (int i = 0; i < s.n && ok; ++i, ++kit) {
                        if ((kit & 1) != wg) continue;
                        const int st = kit % NS;
                        ok = mbar_wait(smem_u32(&sh.kfull[st]), (uint32_t)((kit / NS) & 1), abort_flag);
                        for (int rb = 0; rb < n_rb && ok; ++rb, ++wsit) {
                            // warpgroup wg owns slots 2 wg and 2 wg + 1, used in turn
                            const int slot = 2 * wg + (wsit & 1);
                            ok = mbar_wait(smem_u32(&sh.tempty[slot]), (uint32_t)(((wsit >> 1) & 1) ^ 1), abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                            const uint32_t qa = smem_u32(Qs + (size_t)rb * kTileBytes), ka = smem_u32(Ks + (size_t)st * kTileBytes);
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                // Q tile: [half][128 rows][128 B]; K tile: [8-row group][half][8 rows][128 B]
                                const unsigned long long dq = smem_desc(qa + (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32), 1024);
                                const unsigned long long dk = smem_desc(ka + (uint32_t)((k >> 2) * 1024 + (k & 3) * 32), 2048);
                                tc_mma(tmem_base + (uint32_t)(slot * 128), PHASE == 1 ? dq : dk, PHASE == 1 ? dk : dq, kIdesc, k > 0);
                            }
                            tc_commit(smem_u32(&sh.tfull[slot]));
                        }
                        if (ok) tc_commit(smem_u32(&sh.kempty[st]));
                    }
                    if (ok) tc_commit(smem_u32(&sh.qempty));
                    gv += s.n;
                    ++seg;
                }
                // all tensor work issued by this thread has finished before TMEM is released
                tc_commit(smem_u32(&sh.done[wg]));
                for (uint32_t i = 0; i < kWaitLimit; ++i)
                    if (mbar_try_wait(smem_u32(&sh.done[wg]), 0)) break;
            }
            __syncwarp();
        } else if (warp >= 4) {
            // ------------------------------------------------------------ consumers
            // Four warpgroups.  Warpgroups (pair, 0) and (pair, 1) share the tiles of one pair (tiles in
            // turn between the two pairs): thread li of either owns TMEM lane li, the first takes
            // columns [0, 64) of the slot and the second columns [64, 128).
            const int wgq = (warp - 4) >> 2, pair = wgq & 1, half = wgq >> 1, quad = warp & 3, li = quad * 32 + lane;
            int kit = 0, wsit = 0, seg = 0, pc0 = 0, pc1 = 0; // pc*: uses so far of this pair's two hand-over barriers
            bool ok = true;
            // a thread whose wait ran out keeps walking the segments without touching the pipeline, so that
            // the consumers' named barriers stay matched
            for (long long gv = 0; gv < g_span * hpb;) {
                const int my_h = my_h0 + (int)(gv / g_span) * my_hs;
                const long long g = g_begin + gv % g_span;
                const Segment s = decode_segment(p, prefix, tiles_lh, tpc, g, g_end, my_h);
                const int T = s.T;
                float m[4], z[4];
                int lastv[4];
                float *fs = fin_s + (seg & 1) * p.rows_pad;
                float pmax = 0.0f;
                if (PHASE == 1) {
#pragma unroll
                    for (int rb = 0; rb < 4; ++rb) {
                        m[rb] = -INFINITY; z[rb] = 0.0f;
                        const int r = rb * 128 + li;
                        lastv[rb] = r < p.rows ? (p.causal ? T - p.W + (r % p.W) : T - 1) : -1;
                    }
                } else {
                    // merge the statistics the blocks of the first pass left for this unit, in block
                    // order: b_r = M_r + log2 Z_r per row, and the window maximum 1 / min_r Z_r.
                    // This pass is launched so that its blocks may start while the last blocks of the first
                    // pass are still running (its loads and MMAs depend on nothing the first pass writes);
                    // only here, before the statistics are read, must the first pass be complete.
                    if (seg == 0) wait_for_previous_kernel();
                    const int nt_u = prefix[s.b + 1] - prefix[s.b];
                    const long long ustart = g - s.tile0;
                    const int n_parts = (int)((ustart + nt_u - 1) / tpc) - (int)(ustart / tpc) + 1;
                    float best = 0.0f;
                    for (int r = (warp - 4) * 32 + lane; r < p.rows_pad; r += kConsumerThreads) {
                        float mm = -INFINITY, zz = 0.0f;
                        for (int q = 0; q < n_parts; ++q) {
                            const float2 v = __ldcg(reinterpret_cast<const float2 *>(p.part) + ((size_t)s.uid * p.n_slices + q) * p.rows_pad + r);
                            lse_merge(mm, zz, v.x, v.y);
                        }
                        const bool live = r < p.rows && zz > 0.0f;
                        fs[r] = live ? mm + log2f(zz) : INFINITY; // padding rows contribute nothing
                        if (live) best = fmaxf(best, 1.0f / zz);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
                    if (lane == 0) sh.wmax[seg & 1][warp - 4] = best;
                    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
#pragma unroll
                    for (int w = 0; w < kConsumerThreads / 32; ++w) pmax = fmaxf(pmax, sh.wmax[seg & 1][w]);
                }
                for (int i = 0; i < s.n && ok; ++i, ++kit) {
                    if ((kit & 1) != pair) continue;
                    const int t0 = (s.tile0 + i) * kTileTokens;
                    float acc = 0.0f;
                    int last_slot = 0;
                    for (int rb = 0; rb < n_rb && ok; ++rb, ++wsit) {
                        const int slot = 2 * pair + (wsit & 1);
                        last_slot = slot;
                        ok = mbar_wait(smem_u32(&sh.tfull[slot]), (uint32_t)((wsit >> 1) & 1), abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * 128 + half * 64);
                        if (PHASE == 1) {
                            // 32 columns at a time: one running-maximum update (one rescaling exponential) per 32 logits, and
                            // the maximum tree of one half can overlap the exponentials of the other
                            const int lv = min(lastv[rb], T - 1);
                            float mr = m[rb], zr = z[rb];
                            uint32_t d[32];
                            tc_ld32_issue(taddr, d);
#pragma unroll
                            for (int ch = 0; ch < 2; ++ch) {
                                tc_ld_wait(d);
                                float v[32];
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(d[j]);
                                if (ch == 0) tc_ld32_issue(taddr + 32, d);
                                const int tc0 = t0 + half * 64 + ch * 32;
                                if (tc0 <= lv) {
                                    if (tc0 + 31 > lv) {
#pragma unroll
                                        for (int j = 0; j < 32; ++j) if (tc0 + j > lv) v[j] = -INFINITY;
                                    }
                                    // tree of three-input maxima
                                    float a[11];
#pragma unroll
                                    for (int j = 0; j < 10; ++j) a[j] = max3(v[3 * j], v[3 * j + 1], v[3 * j + 2]);
                                    a[10] = fmaxf(v[30], v[31]);
                                    const float b0 = max3(a[0], a[1], a[2]), b1 = max3(a[3], a[4], a[5]), b2 = max3(a[6], a[7], a[8]);
                                    const float cm = fmaxf(max3(b0, b1, b2), fmaxf(a[9], a[10]));
                                    const float mn = fmaxf(mr, cm * c);
                                    zr *= ex2(mr - mn);
                                    mr = mn;
                                    float zs[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                                    for (int j = 0; j < 32; ++j) zs[j & 3] += ex2(fmaf(v[j], c, -mn));
                                    zr += (zs[0] + zs[1]) + (zs[2] + zs[3]);
                                }
                            }
                            m[rb] = mr; z[rb] = zr;
                        } else {
                            const int t = t0 + li;
                            const bool plain = !p.causal || t0 + kTileTokens - 1 <= T - p.W;
                            const float4 *fr4 = reinterpret_cast<const float4 *>(fs + rb * 128 + half * 64);
                            float ac[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                            uint32_t d[32];
                            tc_ld32_issue(taddr, d);
#pragma unroll
                            for (int ch = 0; ch < 2; ++ch) { // 32 columns (query rows) at a time
                                tc_ld_wait(d);
                                if (plain) {
#pragma unroll
                                    for (int j4 = 0; j4 < 8; ++j4) {
                                        const float4 f = fr4[ch * 8 + j4];
                                        ac[0] += ex2(fmaf(__uint_as_float(d[4 * j4]), c, -f.x));
                                        ac[1] += ex2(fmaf(__uint_as_float(d[4 * j4 + 1]), c, -f.y));
                                        ac[2] += ex2(fmaf(__uint_as_float(d[4 * j4 + 2]), c, -f.z));
                                        ac[3] += ex2(fmaf(__uint_as_float(d[4 * j4 + 3]), c, -f.w));
                                    }
                                } else {
                                    const int rbase = rb * 128 + half * 64 + ch * 32;
#pragma unroll
                                    for (int j = 0; j < 32; ++j) {
                                        const int r = rbase + j;
                                        const bool seen = t <= T - p.W + (r % p.W);
                                        ac[j & 3] += seen ? ex2(fmaf(__uint_as_float(d[j]), c, -fs[r])) : 0.0f;
                                    }
                                }
                                if (ch == 0) tc_ld32_issue(taddr + 32, d);
                            }
                            acc += (ac[0] + ac[1]) + (ac[2] + ac[3]);
                        }
                        if (PHASE == 2 && rb == n_rb - 1) break; // the slot of a tile's last query block is released below
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&sh.tempty[slot]));
                    }
                    if (PHASE == 2 && ok) {
                        // The two halves of the query rows meet here: the second warpgroup leaves its sum in shared
                        // memory, the first adds it and writes the token's usage.  The buffer is the one of the slot,
                        // and the first warpgroup releases the slot only after reading it, so the next tile that
                        // maps to this slot cannot overwrite it early.
                        ++wsit; // (the loop above left through its break)
                        const int bit = last_slot & 1;
                        float *pa = sh.pacc[pair][bit];
                        const uint32_t pbar = smem_u32(&sh.pfull[pair][bit]);
                        if (half == 1) {
                            pa[li] = acc;
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) { mbar_arrive(pbar); mbar_arrive(smem_u32(&sh.tempty[last_slot])); }
                        } else {
                            ok = mbar_wait(pbar, (uint32_t)((bit ? pc1 : pc0) & 1), abort_flag);
                            if (ok) {
                                acc += pa[li];
                                const int t = t0 + li;
                                // the slot is released before the usage goes to global memory: an arrive (a release) issued
                                // after the store would wait until the store has been performed
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(smem_u32(&sh.tempty[last_slot]));
                                if (t < T) {
                                    const int ninv = p.causal ? p.G * max(0, t - (T - p.W)) : 0;
                                    p.scores[(size_t)s.uid * p.T_cap + t] = (acc + (float)ninv * pmax) * (1.0f / (float)p.rows);
                                }
                            }
                        }
                        if (bit) ++pc1; else ++pc0;
                    }
                }
                if (PHASE == 1) {
                    // fold the four warpgroups' statistics (fixed order) and store this block's part of the unit
                    float2 *rd = red;
                    if (wgq > 0)
                        for (int rb = 0; rb < n_rb; ++rb) rd[((wgq - 1) * n_rb + rb) * 128 + li] = make_float2(m[rb], z[rb]);
                    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
                    if (wgq == 0 && ok) {
                        float2 *out = reinterpret_cast<float2 *>(p.part) + ((size_t)s.uid * p.n_slices + s.part) * p.rows_pad;
                        for (int rb = 0; rb < n_rb; ++rb) {
                            float mm = m[rb], zz = z[rb];
                            for (int w = 0; w < 3; ++w) {
                                const float2 o = rd[(w * n_rb + rb) * 128 + li];
                                lse_merge(mm, zz, o.x, o.y);
                            }
                            out[rb * 128 + li] = make_float2(mm, zz);
                        }
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); // the buffer is free again
                }
                gv += s.n;
                ++seg;
            }
        }
    }
    if (*abort_flag && tid == 0) set_status(p.status, AMS_ERR_TIMEOUT, blockIdx.x, PHASE, 0);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

} // namespace

bool tova_tc_supported(const DevParams &p) { return p.rows >= 64 && p.rows_pad % 128 == 0 && p.rows_pad <= 512 && p.B <= 1024 && p.H <= 64; }

size_t tova_tc_smem_bytes(const DevParams &p)
{
    return 1024 + (size_t)(p.rows_pad / 128 + p.tc_stages) * kTileBytes + (size_t)2 * p.rows_pad * 4 +
           (size_t)3 * (p.rows_pad / 128) * 128 * 8 + 256;
}

int launch_score_tova_tc(const DevParams &p_in, LaunchCtx &ctx)
{
    DevParams p = p_in; // the launcher fills in how the heads are spread over the blocks
    // With two MMA issuers taking tiles in turn, an even ring depth gives every stage to one issuer, which
    // then sees all phases of the stage's barrier in order (a parity wait must not skip a phase).
    if (p.tc_stages < 2 || (p.tc_stages & 1)) return AMS_ERR_UNSUPPORTED;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return AMS_ERR_CUDA;
    CUtensorMap k_map, q_map;
    int rc = make_k_map(p, enc, &k_map);
    if (rc == AMS_OK) rc = make_rows_map(p.q, (unsigned long long)p.L * p.B * p.H * p.G * p.W, enc, &q_map);
    if (rc != AMS_OK) return rc;
    const int n_sm = sm_count();
    if (n_sm <= 0) return AMS_ERR_CUDA;
    const size_t smem = tova_tc_smem_bytes(p);
    static SmemGrant grant1, grant2;
    if (!grant_dynamic_smem(k_tova_tc<1>, smem, grant1) || !grant_dynamic_smem(k_tova_tc<2>, smem, grant2)) return AMS_ERR_CUDA;
    const TcGrid tg = tc_grid(p, n_sm);
    const int hpb = tg.hpb, grid = tg.grid;
    p.tc_hpb = hpb;
    k_tova_tc<1><<<grid, kTcThreads, smem, ctx.s>>>(p, k_map, q_map);
    ctx.mark(kKernScore1);
    if (launch_after(k_tova_tc<2>, dim3((unsigned)grid), dim3(kTcThreads), smem, ctx.s, p, k_map, q_map) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernScore2);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

} // namespace ams
