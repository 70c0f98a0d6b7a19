// TOVA-style scorer that reads K once (rows = G * W padded to 128, sequences of at most one
// 128-token tile per block of the grid).
//
// All blocks of a cooperative grid work on the same (layer, sequence, KV head) at the same
// time, one 128-token tile each.  For its tile a block computes the logits with tcgen05.mma
// (query rows on the TMEM lanes), and a group of consumer threads turns them, in place in
// TMEM, into e = 2^(x - ref) with ref the maximum of the thread's 32-column chunk, summing e
// per row.  The per-row (max, sum) of the tile goes to global memory and a per-unit counter
// is raised.  When all tiles of a unit are in, every block merges the statistics of "its"
// query rows (row = tile index, a job of an otherwise idle warp) into
// b_r = log2 sum_t 2^(x_rt) and raises a second counter.  Two items later the consumer group
// comes back to the tile still sitting in TMEM, scales each chunk by 2^(ref - b_r) and adds
// up the rows: the usage of the tile's tokens.  K is read from HBM once and every
// exponential is taken once.
//
// Roles inside a block: warp 0 TMA producer (query block and K tile per item), warp 1 MMA
// issuer, warp 2 statistics merger, warps 4-11 and 12-19 two consumer groups that take items
// in turn (inside a group, half h owns columns [64 h, 64 h + 64) and a thread one query row).
// Four TMEM slots of 128 columns: one being filled, one or two in a group's first visit, the
// others waiting for their unit's statistics.  Every wait is bounded; on expiry the block
// reports AMS_ERR_TIMEOUT and leaves cleanly.
#include <cuda.h>
#include <stdlib.h>

#include "ams_common.cuh"
#include "ams_tc_ptx.cuh"

namespace ams {

using namespace tc;

namespace {

constexpr int kThreads = 640;
constexpr int kTileTokens = 128;
constexpr int kTileBytes = kTileTokens * kRowBytes; // 32 KB
constexpr int kHalfBytes = kTileBytes / 2;
constexpr int kKStages = 3, kQStages = 2, kSlots = 4;
constexpr uint32_t kFlagSpins = 1u << 20;

struct FusedShared {
    unsigned long long kfull[kKStages], kempty[kKStages], qfull[kQStages], qempty[kQStages], tfull[kSlots], tempty[kSlots], done;
    uint32_t tmem_base;
    int abort_flag;
    float wmax[2][2][4];
};

__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
                 ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
                   "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void named_bar(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }

__device__ __forceinline__ int ld_acquire(const int *ptr)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ int tiles_of(const DevParams &p, int b)
{
    const int T = p.seq_lens[b];
    return (T > p.Tk && T <= p.T_cap && p.W <= T) ? (T + kTileTokens - 1) / kTileTokens : 0;
}

// One work item of a block: its tile of the unit handled in round r (or nothing).
struct Item { int uid, l, b, h, T, nt; bool active; };

__device__ __forceinline__ Item item_of(const DevParams &p, int round, int unit_lanes, int my_lane, int my_tile)
{
    Item it;
    const int U = p.L * p.B * p.H;
    it.uid = round * unit_lanes + my_lane;
    it.active = false;
    if (it.uid >= U) return it;
    it.h = it.uid % p.H; it.b = (it.uid / p.H) % p.B; it.l = it.uid / (p.H * p.B);
    it.nt = tiles_of(p, it.b);
    it.T = p.seq_lens[it.b];
    it.active = my_tile < it.nt;
    return it;
}

// Sum over the 32 lanes of v[c] for every c: lane L returns the total of column L.
__device__ __forceinline__ float warp_transpose_sum(float (&v)[32], int lane)
{
#pragma unroll
    for (int s = 16, n = 32; s >= 1; s >>= 1, n >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < n / 2; ++i) {
            const float send = up ? v[i] : v[i + n / 2];
            const float keep = up ? v[i + n / 2] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    return v[0];
}

struct Pending { int uid, tile, T, slot, n; float ref0, ref1; bool valid; };

// Spins (bounded) until *ptr == want; false when the wait ran out or the block gave up.
__device__ __forceinline__ bool wait_count(const int *ptr, int want, volatile int *abort_flag)
{
    for (uint32_t i = 0; i < kFlagSpins; ++i) {
        if (ld_acquire(ptr) == want) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
        __nanosleep(64);
    }
    *abort_flag = 1;
    return false;
}

__global__ void __launch_bounds__(kThreads, 1) k_tova_fused(DevParams p, const __grid_constant__ CUtensorMap k_map,
                                                            const __grid_constant__ CUtensorMap q_map, int tiles_cap, int unit_lanes)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ FusedShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *Qs = base;                                          // [kQStages][2 halves][128 rows][128 B]
    unsigned char *Ks = Qs + (size_t)kQStages * kTileBytes;            // [kKStages][8-row group][half][8 rows][128 B]
    float2 *red_all = reinterpret_cast<float2 *>(Ks + (size_t)kKStages * kTileBytes); // [2 groups][128] statistics of half 1
    float *sred_all = reinterpret_cast<float *>(red_all + 256);        // [2 groups][2 halves][4 quads][64 columns]
    volatile int *abort_flag = &sh.abort_flag;

    if (tid == 0) {
        for (int i = 0; i < kKStages; ++i) { mbar_init(smem_u32(&sh.kfull[i]), 1); mbar_init(smem_u32(&sh.kempty[i]), 1); }
        for (int i = 0; i < kQStages; ++i) { mbar_init(smem_u32(&sh.qfull[i]), 1); mbar_init(smem_u32(&sh.qempty[i]), 1); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(smem_u32(&sh.tfull[i]), 1); mbar_init(smem_u32(&sh.tempty[i]), 8); }
        mbar_init(smem_u32(&sh.done), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;
    const int my_lane = blockIdx.x / tiles_cap, my_tile = blockIdx.x % tiles_cap;
    const int U = p.L * p.B * p.H;
    const int n_rounds = (U + unit_lanes - 1) / unit_lanes;
    if (blockIdx.x == 0 && tid == 0) {
        for (int b = 0; b < p.B; ++b) {
            const int T = p.seq_lens[b];
            if (T > p.Tk && T <= p.T_cap && p.W > T) set_status(p.status, AMS_ERR_INVALID_ARG, b, p.W, T);
        }
    }
    const float c = kLog2e * 0.08838834764831845f; // log2(e) / sqrt(128)

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        int j = 0, issued = 0;
        bool ok = true;
        for (int r = 0; r < n_rounds && ok; ++r) {
            const Item it = item_of(p, r, unit_lanes, my_lane, my_tile);
            if (!it.active) continue;
            const int kst = j % kKStages, qst = j % kQStages;
            ok = mbar_wait(smem_u32(&sh.kempty[kst]), (uint32_t)(((j / kKStages) & 1) ^ 1), abort_flag) &&
                 mbar_wait(smem_u32(&sh.qempty[qst]), (uint32_t)(((j / kQStages) & 1) ^ 1), abort_flag);
            if (!ok) break;
            if (lane == 0) {
                mbar_expect_tx(smem_u32(&sh.qfull[qst]), (uint32_t)kTileBytes);
                const int qrow0 = ((it.l * p.B + it.b) * p.H * p.G + it.h * p.G) * p.W;
                for (int hf = 0; hf < 2; ++hf)
                    tma_load_2d(smem_u32(Qs + (size_t)qst * kTileBytes + hf * kHalfBytes), &q_map, smem_u32(&sh.qfull[qst]), hf * 64, qrow0);
                mbar_expect_tx(smem_u32(&sh.kfull[kst]), (uint32_t)kTileBytes);
            }
            __syncwarp();
            if (lane < 8) {
                const int *table = p.block_table + (size_t)it.b * p.bt_stride;
                const int last_page = (it.T - 1) >> 4;
                int pi = my_tile * 8 + lane;
                if (pi > last_page) pi = last_page; // tokens past the end are masked by position
                tma_load_5d(smem_u32(Ks + (size_t)kst * kTileBytes + lane * 4096), &k_map, smem_u32(&sh.kfull[kst]), 0, 0, 2 * it.h, 0,
                            it.l * (int)p.num_pages + table[pi]);
            }
            ++j;
            issued = j;
        }
        if (!ok) { // drain: wait (bounded) for the copies that were issued and never consumed
            for (int k = max(0, issued - kKStages); k < issued; ++k)
                for (uint32_t i = 0; i < kWaitLimit; ++i)
                    if (mbar_try_wait(smem_u32(&sh.kfull[k % kKStages]), (uint32_t)((k / kKStages) & 1))) break;
            for (int k = max(0, issued - kQStages); k < issued; ++k)
                for (uint32_t i = 0; i < kWaitLimit; ++i)
                    if (mbar_try_wait(smem_u32(&sh.qfull[k % kQStages]), (uint32_t)((k / kQStages) & 1))) break;
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int j = 0;
            bool ok = true;
            for (int r = 0; r < n_rounds && ok; ++r) {
                const Item it = item_of(p, r, unit_lanes, my_lane, my_tile);
                if (!it.active) continue;
                const int kst = j % kKStages, qst = j % kQStages, slot = j % kSlots;
                ok = mbar_wait(smem_u32(&sh.qfull[qst]), (uint32_t)((j / kQStages) & 1), abort_flag) &&
                     mbar_wait(smem_u32(&sh.kfull[kst]), (uint32_t)((j / kKStages) & 1), abort_flag) &&
                     mbar_wait(smem_u32(&sh.tempty[slot]), (uint32_t)(((j / kSlots) & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t qa = smem_u32(Qs + (size_t)qst * kTileBytes), ka = smem_u32(Ks + (size_t)kst * kTileBytes);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const unsigned long long dq = smem_desc(qa + (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32), 1024);
                    const unsigned long long dk = smem_desc(ka + (uint32_t)((k >> 2) * 1024 + (k & 3) * 32), 2048);
                    tc_mma(tmem_base + (uint32_t)(slot * 128), dq, dk, kIdesc, k > 0);
                }
                tc_commit(smem_u32(&sh.tfull[slot]));
                tc_commit(smem_u32(&sh.kempty[kst]));
                tc_commit(smem_u32(&sh.qempty[qst]));
                ++j;
            }
            tc_commit(smem_u32(&sh.done));
            for (uint32_t i = 0; i < kWaitLimit; ++i)
                if (mbar_try_wait(smem_u32(&sh.done), 0)) break;
        }
        __syncwarp();
    } else if (warp == 2) {
        // ---------------------------------------------------------------- statistics merger
        // For every unit this block has a tile of: once all tiles' statistics are in, merge
        // those of query rows my_tile, my_tile + nt, ... and publish b_r and 1 / Z_r.
        bool ok = true;
        for (int r = 0; r < n_rounds && ok; ++r) {
            const Item it = item_of(p, r, unit_lanes, my_lane, my_tile);
            if (!it.active) continue;
            ok = wait_count(p.fcnt + it.uid, it.nt, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            int done_rows = 0;
            for (int row = my_tile; row < p.rows_pad; row += it.nt, ++done_rows) {
                const float2 *pp = reinterpret_cast<const float2 *>(p.part) + (size_t)it.uid * p.n_slices * p.rows_pad + row;
                float2 v[5];
#pragma unroll
                for (int k = 0; k < 5; ++k) {
                    const int tt = lane + 32 * k;
                    v[k] = tt < it.nt ? __ldcg(pp + (size_t)tt * p.rows_pad) : make_float2(-INFINITY, 0.0f);
                }
                float mm = v[0].x, zz = v[0].y;
#pragma unroll
                for (int k = 1; k < 5; ++k) lse_merge(mm, zz, v[k].x, v[k].y);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float m2 = __shfl_xor_sync(0xffffffffu, mm, o), z2 = __shfl_xor_sync(0xffffffffu, zz, o);
                    // same operands in the same order on both lanes of a pair
                    float ma = (lane & o) ? m2 : mm, za = (lane & o) ? z2 : zz, mb = (lane & o) ? mm : m2, zb = (lane & o) ? zz : z2;
                    lse_merge(ma, za, mb, zb);
                    mm = ma; zz = za;
                }
                if (lane == 0) {
                    const bool live = row < p.rows && zz > 0.0f;
                    p.fin[(size_t)it.uid * (p.rows_pad + 8) + row] = live ? mm + log2f(zz) : INFINITY; // padding rows contribute nothing
                    p.finz[(size_t)it.uid * p.rows_pad + row] = live ? 1.0f / zz : 0.0f;
                }
            }
            if (lane == 0) {
                __threadfence();
                atomicAdd(p.fflag + it.uid, done_rows);
            }
        }
    } else if (warp >= 4) {
        // ---------------------------------------------------------------- consumers
        const int grp = (warp - 4) >> 3, half = ((warp - 4) >> 2) & 1, quad = warp & 3, row = quad * 32 + lane;
        const int bar_grp = 1 + grp * 4, bar_half = 3 + grp * 4 + half; // named barriers: 256 threads / 128 threads
        float2 *red = red_all + grp * 128;
        float *sred = sred_all + (size_t)(grp * 2 + half) * 4 * 64;
        const float inv_rows = 1.0f / (float)p.rows;
        bool ok = true;
        Pending pend; // this group's previous item, waiting for its unit's statistics
        pend.valid = false;
        int j = 0;

        // second visit of a tile: scale by the unit's statistics and add up the rows
        auto finish_tile = [&](const Pending &pd) {
            if (ok) {
                // every lane polls: a loop run by one lane would leave the warp split in front of the
                // warp-aligned tcgen05 instructions below, which then do not act as one instruction
                wait_count(p.fflag + pd.uid, p.rows_pad, abort_flag);
                __syncwarp();
                ok = *abort_flag == 0;
            }
            float acc0 = 0.0f, acc1 = 0.0f, iz = 0.0f;
            if (ok) {
                const float br = __ldcg(p.fin + (size_t)pd.uid * (p.rows_pad + 8) + row);
                iz = __ldcg(p.finz + (size_t)pd.uid * p.rows_pad + row);
                const float w0 = (pd.ref0 == -INFINITY) ? 0.0f : ex2(pd.ref0 - br);
                const float w1 = (pd.ref1 == -INFINITY) ? 0.0f : ex2(pd.ref1 - br);
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(pd.slot * 128 + half * 64);
                uint32_t b0[32];
                float v[32];
                tc_ld32_issue(taddr, b0);
                tc_ld_wait(b0);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(b0[i]) * w0;
                acc0 = warp_transpose_sum(v, lane);
                tc_ld32_issue(taddr + 32, b0);
                tc_ld_wait(b0);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(b0[i]) * w1;
                acc1 = warp_transpose_sum(v, lane);
                tc_fence_before();
            }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(smem_u32(&sh.tempty[pd.slot]));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) iz = fmaxf(iz, __shfl_xor_sync(0xffffffffu, iz, o));
            if (lane == 0) sh.wmax[grp][half][quad] = iz;
            sred[quad * 64 + lane] = acc0;
            sred[quad * 64 + 32 + lane] = acc1;
            named_bar(bar_half, 128);
            if (ok && row < 64) {
                const float pmax = fmaxf(fmaxf(sh.wmax[grp][half][0], sh.wmax[grp][half][1]), fmaxf(sh.wmax[grp][half][2], sh.wmax[grp][half][3]));
                const float tot = (sred[row] + sred[64 + row]) + (sred[128 + row] + sred[192 + row]);
                const int t = pd.tile * kTileTokens + half * 64 + row;
                if (t < pd.T) {
                    const int ninv = p.causal ? p.G * max(0, t - (pd.T - p.W)) : 0;
                    p.scores[(size_t)pd.uid * p.T_cap + t] = (tot + (float)ninv * pmax) * inv_rows;
                }
            }
            named_bar(bar_half, 128); // the sums are read before the next visit overwrites them
        };

        for (int r = 0; r < n_rounds; ++r) {
            const Item it = item_of(p, r, unit_lanes, my_lane, my_tile);
            if (!it.active) continue;
            if ((j & 1) != grp) { ++j; continue; } // the other group's item
            const int slot = j % kSlots;
            // ---- first visit: logits -> e in place, per-row (max, sum) of this tile
            float m = -INFINITY, z = 0.0f, ref[2] = {-INFINITY, -INFINITY};
            if (ok) ok = mbar_wait(smem_u32(&sh.tfull[slot]), (uint32_t)((j / kSlots) & 1), abort_flag);
            if (ok) {
                tc_fence_after();
                const int lastv = row < p.rows ? (p.causal ? it.T - p.W + (row % p.W) : it.T - 1) : -1;
                const int lv = min(lastv, it.T - 1);
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(slot * 128 + half * 64);
                float zc[2] = {0.0f, 0.0f};
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t buf[32];
                    tc_ld32_issue(taddr + ch * 32, buf);
                    tc_ld_wait(buf);
                    const int tc0 = my_tile * kTileTokens + half * 64 + ch * 32;
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(buf[i]);
                    if (tc0 + 31 > lv) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) if (tc0 + i > lv) v[i] = -INFINITY;
                    }
                    float a8[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) a8[i] = fmaxf(max3(v[i], v[i + 8], v[i + 16]), v[i + 24]);
                    const float cm = fmaxf(max3(a8[0], a8[1], a8[2]), fmaxf(max3(a8[3], a8[4], a8[5]), fmaxf(a8[6], a8[7])));
                    if (cm != -INFINITY) {
                        const float rf = cm * c;
                        ref[ch] = rf;
                        float zs[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float e = ex2(fmaf(v[i], c, -rf)); // masked columns: 2^(-inf) = 0
                            zs[i & 3] += e;
                            buf[i] = __float_as_uint(e);
                        }
                        zc[ch] = (zs[0] + zs[1]) + (zs[2] + zs[3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) buf[i] = 0u;
                    }
                    __syncwarp(); // the branches above are per lane
                    tc_st32(taddr + ch * 32, buf);
                    tc_st_wait(); // the store reads its registers asynchronously: no reuse before it is done
                }
                m = ref[0]; z = zc[0];
                lse_merge(m, z, ref[1], zc[1]);
            }
            // ---- statistics of the tile to global memory, then the unit's tile counter
            if (half == 1) red[row] = make_float2(m, z);
            named_bar(bar_grp, 256);
            if (half == 0) {
                const float2 o = red[row];
                lse_merge(m, z, o.x, o.y);
                reinterpret_cast<float2 *>(p.part)[((size_t)it.uid * p.n_slices + my_tile) * p.rows_pad + row] = make_float2(m, z);
            }
            named_bar(bar_grp, 256);
            if (half == 0 && row == 0 && ok) {
                __threadfence(); // cumulative: orders the group's writes above before the count
                atomicAdd(p.fcnt + it.uid, 1);
            }
            // ---- second visit of this group's previous item
            if (pend.valid) finish_tile(pend);
            pend.valid = true; pend.uid = it.uid; pend.tile = my_tile; pend.T = it.T; pend.slot = slot; pend.n = j;
            pend.ref0 = ref[0]; pend.ref1 = ref[1];
            ++j;
        }
        if (pend.valid) finish_tile(pend);
    }
    if (*abort_flag && tid == 0) set_status(p.status, AMS_ERR_TIMEOUT, blockIdx.x, 3, 0);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

size_t fused_smem_bytes() { return 1024 + (size_t)(kQStages + kKStages) * kTileBytes + 256 * 8 + 2 * 2 * 4 * 64 * 4 + 256; }

} // namespace

// The single-pass scorer is opt-in (environment variable AMS_FUSED_SCORER=1): on B200 the
// hand-off of the per-tile statistics between blocks (publish, wait for the slowest block,
// merge) takes longer than the two items of look-ahead that TMEM's 512 columns allow, so the
// two-kernel scorer, which reads K twice, is the faster one at the benchmark sizes.
bool tova_fused_supported(const DevParams &p)
{
    const char *env = getenv("AMS_FUSED_SCORER");
    if (!env || env[0] != '1') return false;
    static int n_sm = 0;
    if (!n_sm) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    }
    const int tiles_cap = (p.T_cap + kTileTokens - 1) / kTileTokens;
    return p.rows >= 64 && p.rows_pad == 128 && tiles_cap <= n_sm && p.n_slices >= tiles_cap && p.fcnt && p.fflag && p.finz && p.B <= 1024 &&
           (long long)p.L * p.num_pages <= 0x7fffffffLL;
}

int launch_score_tova_fused(const DevParams &p, LaunchCtx &ctx)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return AMS_ERR_CUDA;
    CUtensorMap k_map, q_map;
    {
        // One page of one layer is [16 slots][H heads][2 halves][64]: seen as
        // (64, slot % 8, head * 2 + half, slot / 8, layer * num_pages + page), so that a box of
        // (64, 8, 2, 2, 1) is one head's 16 rows, stored as [slot / 8][half][slot % 8][64].
        const cuuint64_t dims[5] = {64, 8, (cuuint64_t)2 * p.H, 2, (cuuint64_t)p.L * (cuuint64_t)p.num_pages};
        const cuuint64_t strides[4] = {(cuuint64_t)p.H * kRowBytes, 128, (cuuint64_t)8 * p.H * kRowBytes, (cuuint64_t)kPage * p.H * kRowBytes};
        const cuuint32_t box[5] = {64, 8, 2, 2, 1};
        const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        if (enc(&k_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, p.k_pages, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return AMS_ERR_CUDA;
    }
    {
        const cuuint64_t dims[2] = {kHeadDim, (cuuint64_t)p.L * p.B * p.H * p.G * p.W};
        const cuuint64_t strides[1] = {kRowBytes};
        const cuuint32_t box[2] = {64, 128};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&q_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16 *>(p.q), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return AMS_ERR_CUDA;
    }
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return AMS_ERR_CUDA;
    const size_t smem = fused_smem_bytes();
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(k_tova_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return AMS_ERR_CUDA;
        configured = true;
    }
    int tiles_cap = (p.T_cap + kTileTokens - 1) / kTileTokens;
    int unit_lanes = n_sm / tiles_cap; // units worked on at the same time
    const int U = p.L * p.B * p.H;
    if (unit_lanes > U) unit_lanes = U;
    if (unit_lanes < 1) return AMS_ERR_UNSUPPORTED;
    DevParams pp = p;
    if (cudaMemsetAsync(p.fcnt, 0, (size_t)U * sizeof(int), ctx.s) != cudaSuccess ||
        cudaMemsetAsync(p.fflag, 0, (size_t)U * sizeof(int), ctx.s) != cudaSuccess)
        return AMS_ERR_CUDA;
    void *args[] = {&pp, &k_map, &q_map, &tiles_cap, &unit_lanes};
    // cooperative launch: all blocks are resident together, which the waits between blocks rely on
    if (cudaLaunchCooperativeKernel((const void *)k_tova_fused, dim3((unsigned)(tiles_cap * unit_lanes)), dim3(kThreads), args, smem, ctx.s) !=
        cudaSuccess)
        return AMS_ERR_CUDA;
    ctx.mark(kKernScore1);
    return AMS_OK;
}

} // namespace ams
