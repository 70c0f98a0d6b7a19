// Algorithm 1 steps 1-5 of the paper (mass, EMA credit, prefix scan, cuts, merge/split,
// quotas, per-segment top-q, must-keep, backfill, ordered index compaction) with every
// per-token array held on chip.
//
// One thread-block cluster handles one (layer, sequence, KV head).  Block r of the cluster
// owns tokens [r * TPC, (r + 1) * TPC); thread i of a block owns VPT consecutive tokens,
// whose fixed-point masses, sort keys and credits live in registers / thread-private shared
// memory.  Every per-token step is done by the owning thread on this block's shared memory;
// the blocks of a cluster meet only to add up per-block sums and per-segment counts through
// distributed shared memory.  Results are bit-identical to the one-block kernel: all
// decisions are integer, and integer sums do not depend on their order.
#include <cooperative_groups.h>
#include <string.h>

#include <type_traits>

#include "ams_common.cuh"
#include "ams_select.cuh"

namespace cg = cooperative_groups;

namespace ams {

using namespace sel;

namespace {

constexpr int kXch = 8; // ring of exchange slots (>= 2)
constexpr int kNT = 1024;

// Dynamic shared memory of one block (byte offsets).
struct SmemMap {
    size_t gs, flags, crs, cend, ms, bounds, quota, cap, give, raw, merged, poff, cand, cnt, take, ties, tps, qthr, total;
};

__host__ __device__ inline size_t up16(size_t x) { return (x + 15) & ~(size_t)15; }

__host__ __device__ inline SmemMap smem_map(int tpc, int sc, int S, bool ema_on)
{
    SmemMap m;
    size_t o = 0;
    m.gs = o;     o = up16(o + (size_t)tpc * 4);
    m.flags = o;  o = up16(o + (size_t)tpc);
    m.crs = o;    o = up16(o + (ema_on ? (size_t)tpc * 4 : 0));
    m.cend = o;   o = up16(o + (size_t)(sc + 1) * 8);
    m.ms = o;     o = up16(o + (size_t)sc * 8);
    m.bounds = o; o = up16(o + (size_t)(sc + 1) * 4);
    m.quota = o;  o = up16(o + (size_t)sc * 4);
    m.cap = o;    o = up16(o + (size_t)sc * 4);
    m.give = o;   o = up16(o + (size_t)sc * 4);
    m.raw = o;    o = up16(o + (size_t)(S + 1) * 4);
    m.merged = o; o = up16(o + (size_t)(S + 1) * 4);
    m.poff = o;   o = up16(o + (size_t)(S + 1) * 4);
    m.cand = o;   o = up16(o + (size_t)sc * 4);
    m.cnt = o;    o = up16(o + (size_t)2 * 3 * sc * 4);
    m.take = o;   o = up16(o + (size_t)sc * 4);
    m.ties = o;   o = up16(o + (size_t)sc * 4);
    m.tps = o;    o = up16(o + (size_t)sc * 4);
    m.qthr = o;   o = up16(o + (size_t)(S + 1) * 8);
    m.total = o;
    return m;
}

// CS (blocks per cluster) is a template parameter so that every loop over the ranks of the cluster
// unrolls into independent remote loads instead of a chain of dependent ones.
template <int NT, int VPT, int CS>
__device__ __forceinline__ void segment_unit(const DevParams &p, const int uid, const int cs_max)
{
    constexpr int nt = NT, TPC = NT * VPT, cs = CS;
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ Smem sm;
    __shared__ u64 xch[kXch];
    __shared__ int wcnt[64]; // per-warp counts of even / odd search rounds
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31;
    const int rank = cs > 1 ? (int)cluster.block_rank() : 0;
    const int h = uid % p.H, b = (uid / p.H) % p.B, l = uid / (p.H * p.B);
    const int T = p.seq_lens[b];
    // every exit below is taken by all blocks of the cluster together
    if (T <= p.Tk) return; // nothing to evict
    if (T > p.T_cap) { if (tid == 0 && rank == 0 && cs == cs_max) set_status(p.status, AMS_ERR_CAPACITY, uid, T, p.T_cap); return; }
    // one launch per cluster size: this one takes the sequences that need exactly cs blocks
    if (T > cs * TPC || (cs > 1 && T <= (cs / 2) * TPC)) return;

    const int sc = p.seg_cap;
    const bool ema_on = p.beta != 1.0f;
    const SmemMap mp = smem_map(TPC, sc, p.S, ema_on);
    float *gs = reinterpret_cast<float *>(dyn + mp.gs);
    unsigned char *flags = dyn + mp.flags;
    float *crs = reinterpret_cast<float *>(dyn + mp.crs);      // [VPT][nt], thread-private columns
    u64 *Cend = reinterpret_cast<u64 *>(dyn + mp.cend);
    u64 *Ms = reinterpret_cast<u64 *>(dyn + mp.ms);
    int *bounds = reinterpret_cast<int *>(dyn + mp.bounds);
    int *quota = reinterpret_cast<int *>(dyn + mp.quota);
    int *cap = reinterpret_cast<int *>(dyn + mp.cap);
    int *give = reinterpret_cast<int *>(dyn + mp.give);
    int *raw = reinterpret_cast<int *>(dyn + mp.raw);
    int *merged = reinterpret_cast<int *>(dyn + mp.merged);
    int *poff = reinterpret_cast<int *>(dyn + mp.poff);
    unsigned *cand = reinterpret_cast<unsigned *>(dyn + mp.cand);
    int *cnt = reinterpret_cast<int *>(dyn + mp.cnt);
    int *takev = reinterpret_cast<int *>(dyn + mp.take);
    int *tiesv = reinterpret_cast<int *>(dyn + mp.ties);
    int *tps = reinterpret_cast<int *>(dyn + mp.tps);
    u64 *qthr = reinterpret_cast<u64 *>(dyn + mp.qthr);

    const int t_base = rank * TPC;                       // first token of this block
    const int n_loc = max(0, min(TPC, T - t_base));      // tokens of this block
    const int my0 = tid * VPT;                           // local index of this thread's first token
    const size_t row = (size_t)uid * p.T_cap;
    float *credit = p.ema + (((size_t)l * p.Bmax + b) * p.H + h) * (size_t)p.T_cap;
    int *keep = p.keep_idx + (size_t)uid * p.Tk;
    const double two_f = (double)(1ull << kFixBits);
    int xn = 0; // exchanges done so far (same in every thread of the cluster)

    auto unit_barrier = [&]() { if (cs > 1) cluster.sync(); else __syncthreads(); };
    // Sum over the whole sequence; *prefix (optional) = sum over the blocks before this one.
    // A slot of the ring is rewritten only after kXch - 1 later cluster barriers, which every
    // block reaches only after it has read the slot.
    auto unit_sum = [&](u64 v, u64 *prefix) -> u64 {
        const u64 mine = block_sum_u64(v, sm.scratch);
        if (prefix) *prefix = 0;
        if (cs == 1) return mine;
        u64 *slot = &xch[xn++ % kXch];
        if (tid == 0) *slot = mine;
        cluster.sync();
        u64 tot = 0;
#pragma unroll
        for (int r = 0; r < cs; ++r) {
            const u64 x = *cluster.map_shared_rank(slot, r);
            if (prefix && r < rank) *prefix += x;
            tot += x;
        }
        return tot;
    };
    auto unit_max = [&](float v) -> float {
        const float mine = block_max_f32(v, sm.scratch);
        if (cs == 1) return mine;
        u64 *slot = &xch[xn++ % kXch];
        if (tid == 0) *slot = (u64)__float_as_uint(mine);
        cluster.sync();
        float m = mine;
#pragma unroll
        for (int r = 0; r < cs; ++r) m = fmaxf(m, __uint_as_float((unsigned)*cluster.map_shared_rank(slot, r)));
        return m;
    };

    // Score / flag of any token of the sequence, wherever it lives in the cluster (a short
    // segment may straddle two blocks).
    auto g_at = [&](int t) -> float {
        const int r = t / TPC;
        return r == rank ? gs[t - t_base] : *cluster.map_shared_rank(gs + (t - r * TPC), r);
    };
    auto flag_put = [&](int t, unsigned char f) {
        const int r = t / TPC;
        if (r == rank) flags[t - t_base] = f;
        else *cluster.map_shared_rank(flags + (t - r * TPC), r) = f;
    };

    // ---- scores into shared memory (token order); cut table starts at "no cut"
    {
        const float *g = p.scores + row + t_base;
        for (int i = tid * 4; i < n_loc; i += nt * 4)
            *reinterpret_cast<float4 *>(gs + i) = *reinterpret_cast<const float4 *>(g + i);
        for (int k = tid; k <= p.S; k += nt) raw[k] = T;
    }
    __syncthreads();

    // ---- Eq. 1 weights of this thread's tokens (re-read from shared memory where needed,
    //      so that they do not occupy registers across the reductions)
    // The usage the mass is built from is the score array itself unless it was smoothed or comes from
    // another signal; then it is read from global memory (L2) each time.
    const float *u_sep = p.usage != p.scores ? p.usage + row + t_base : nullptr;
    auto load_w = [&](float (&w)[VPT]) {
#pragma unroll
        for (int q = 0; q < VPT / 4; ++q) {
            float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (my0 + 4 * q < n_loc)
                v = u_sep ? __ldg(reinterpret_cast<const float4 *>(u_sep + my0 + 4 * q)) : *reinterpret_cast<const float4 *>(gs + my0 + 4 * q);
            w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) w[i] = (my0 + i < n_loc) ? weight_of(w[i], p.eps) : 0.0f;
    };
    if (ema_on) {
#pragma unroll
        for (int q = 0; q < VPT / 4; ++q) {
            float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (my0 + 4 * q < n_loc) v = *reinterpret_cast<const float4 *>(credit + t_base + my0 + 4 * q);
            crs[(4 * q) * nt + tid] = v.x; crs[(4 * q + 1) * nt + tid] = v.y;
            crs[(4 * q + 2) * nt + tid] = v.z; crs[(4 * q + 3) * nt + tid] = v.w;
        }
    }
    float wmax = 0.0f;
    {
        float w[VPT];
        load_w(w);
#pragma unroll
        for (int i = 0; i < VPT; ++i) wmax = fmaxf(wmax, w[i]);
    }
    wmax = unit_max(wmax);
    const int ew = fix_exponent(wmax);
    u64 sa = 0;
    {
        float w[VPT];
        load_w(w);
#pragma unroll
        for (int i = 0; i < VPT; ++i) sa += to_fixed_bits(w[i], ew);
    }
    const u64 SA = unit_sum(sa, nullptr);
    const double inv_sa = __ddiv_rn(1.0, (double)SA); // normalisations multiply by the rounded reciprocal

    // ---- EMA credit and the fixed-point mass used for segmentation
    float *mass_dbg = p.mass_dbg ? p.mass_dbg + row + t_base + my0 : nullptr;
    u64 Hm[VPT];
    if (ema_on) {
        const float oml = __fsub_rn(1.0f, p.lambda);
        float cmax = 0.0f;
        float w[VPT];
        load_w(w);
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            if (my0 + i < n_loc) {
                const float m = __double2float_rn(__dmul_rn(u52_to_double(to_fixed_bits(w[i], ew)), inv_sa));
                const float cn = __fadd_rn(__fmul_rn(p.lambda, crs[i * nt + tid]), __fmul_rn(oml, m));
                crs[i * nt + tid] = cn;
                if (mass_dbg) mass_dbg[i] = m;
                cmax = fmaxf(cmax, cn);
            }
        }
        cmax = unit_max(cmax);
        u64 scsum = 0;
        int ec = 0;
        if (cmax > 0.0f) {
            ec = fix_exponent(cmax);
#pragma unroll
            for (int i = 0; i < VPT; ++i)
                if (my0 + i < n_loc) scsum += to_fixed_bits(crs[i * nt + tid], ec);
        }
        const u64 SC = unit_sum(scsum, nullptr);
        const double bd = (double)p.beta, omb = __dsub_rn(1.0, (double)p.beta);
        const double inv_sc = SC > 0 ? __ddiv_rn(1.0, (double)SC) : 0.0;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            Hm[i] = 0;
            if (my0 + i < n_loc) {
                const double cur = __dmul_rn(bd, __dmul_rn(u52_to_double(to_fixed_bits(w[i], ew)), inv_sa));
                double hist_term = 0.0;
                if (SC > 0) hist_term = __dmul_rn(omb, __dmul_rn(u52_to_double(to_fixed_bits(crs[i * nt + tid], ec)), inv_sc));
                Hm[i] = floor_to_u64(__dmul_rn(__dadd_rn(cur, hist_term), two_f));
            }
        }
    } else {
        float w[VPT];
        load_w(w);
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            Hm[i] = 0;
            if (my0 + i < n_loc) {
                const double r = __dmul_rn(u52_to_double(to_fixed_bits(w[i], ew)), inv_sa);
                if (mass_dbg) mass_dbg[i] = __double2float_rn(r);
                Hm[i] = floor_to_u64(__dmul_rn(r, two_f));
            }
        }
    }
    u64 tt = 0;
#pragma unroll
    for (int i = 0; i < VPT; ++i) tt += Hm[i];
    u64 rank_prefix;
    const u64 SH = unit_sum(tt, &rank_prefix);

    // ---- prefix sum and mass-quantile cuts: the token that reaches quantile k closes its
    //      segment, so the boundary is (position + 1); every block receives every cut.
    //      C reaches quantile k when C * S >= k * SH, i.e. C >= ceil(k * SH / S)
    const u64 S = (u64)p.S;
    for (int k = tid + 1; k < p.S; k += nt) qthr[k] = ((u64)k * SH + S - 1) / S;
    u64 btot;
    const u64 exc = rank_prefix + block_excl_scan_u64(tt, sm.scratch, &btot); // (synchronises the block)
    auto quantile = [&](u64 C) -> int { // number of k in [1, S) with qthr[k] <= C
        int lo = 0, hi = p.S - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (qthr[mid] <= C) lo = mid; else hi = mid - 1;
        }
        return lo;
    };
    if (p.fixed_seg) { // component ablation: boundary k at floor(k T / S) whatever the mass (every block, own copy)
        for (int k = tid + 1; k < p.S; k += nt) raw[k] = (int)(((long long)k * T) / p.S);
    } else if (my0 < n_loc) {
        int kprev = quantile(exc);
        const int klast = quantile(exc + tt);
        if (klast != kprev) {
            u64 run = exc;
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                if (my0 + i < n_loc) {
                    run += Hm[i];
                    const int kc = quantile(run);
                    for (int k = kprev + 1; k <= kc; ++k) {
                        const int cut = t_base + my0 + i + 1;
                        if (cs == 1) raw[k] = cut;
                        else for (int r = 0; r < cs; ++r) *cluster.map_shared_rank(raw + k, r) = cut;
                    }
                    kprev = kc;
                }
            }
        }
    }
    unit_barrier();

    // ---- merge short raw segments forward, fold a short tail left, count split pieces
    //      (every block does this on its own copy of the cuts)
    if (tid == 0) {
        int nm = 0;
        merged[nm++] = 0;
        int last = 0;
        for (int k = 1; k < p.S; ++k) {
            const int e = raw[k];
            if (e <= last || e >= T) continue;
            last = e;
            if (e - merged[nm - 1] >= p.l_min) merged[nm++] = e;
        }
        merged[nm++] = T;
        if (nm > 2 && merged[nm - 1] - merged[nm - 2] < p.l_min) { merged[nm - 2] = T; --nm; }
        int off = 0;
        for (int i = 0; i + 1 < nm; ++i) {
            const int len = merged[i + 1] - merged[i];
            poff[i] = off;
            off += (p.l_max > 0 && len > p.l_max) ? (len + p.l_max - 1) / p.l_max : 1;
        }
        poff[nm - 1] = off;
        sm.bcast[0] = nm - 1;
        sm.bcast[1] = off;
    }
    __syncthreads();
    const int n_merged = sm.bcast[0], n_seg = sm.bcast[1];
    if (n_seg > sc) { if (tid == 0 && rank == 0) set_status(p.status, AMS_ERR_CAPACITY, uid, n_seg, sc); return; }
    if (tid == 0) bounds[0] = 0;
    for (int i = 0; i < n_merged; ++i) {
        const int a = merged[i], len = merged[i + 1] - a, pieces = poff[i + 1] - poff[i];
        const int bs = len / pieces, extra = len % pieces;
        for (int j = tid; j < pieces; j += nt) bounds[poff[i] + j + 1] = a + (j + 1) * bs + min(j + 1, extra);
    }
    __syncthreads();

    // ---- segment of each of this thread's tokens: s0 = segment of the first one, bit i of
    //      newseg = token i starts the next segment
    unsigned valid = 0;
#pragma unroll
    for (int i = 0; i < VPT; ++i) if (my0 + i < n_loc) valid |= 1u << i;
    int seg0 = n_seg - 1;
    unsigned newseg = 0;
    if (valid) {
        const int t0 = t_base + my0;
        int lo = 0, hi = n_seg; // bounds[lo] <= t0 < bounds[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (bounds[mid] <= t0) lo = mid; else hi = mid;
        }
        seg0 = lo;
        int s = lo, nb = bounds[lo + 1];
#pragma unroll
        for (int i = 1; i < VPT; ++i)
            if (((valid >> i) & 1u) && t0 + i == nb) { newseg |= 1u << i; ++s; nb = bounds[s + 1]; }
    }

    // ---- prefix of the mass at each segment end, written by the thread that owns the
    //      segment's last token; segment mass = difference of consecutive ends
    bool owns_end = false; // most threads lie strictly inside one segment and have nothing to write
    if (valid) {
        const int n_valid = __popc(valid);
        owns_end = (newseg >> 1) != 0u || t_base + my0 + n_valid == bounds[seg0 + __popc(newseg) + 1];
    }
    if (owns_end) {
        int s = seg0;
        u64 run = exc;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            if ((valid >> i) & 1u) {
                if (i > 0 && ((newseg >> i) & 1u)) ++s;
                run += Hm[i];
                const bool ends = (i + 1 < VPT && ((newseg >> (i + 1)) & 1u)) || t_base + my0 + i + 1 == bounds[s + 1];
                if (ends) {
                    if (cs == 1) Cend[s] = run;
                    else for (int r = 0; r < cs; ++r) *cluster.map_shared_rank(Cend + s, r) = run;
                }
            }
        }
    }
    unit_barrier();

    // ---- must-keep sizes and quotas (every block, same result)
    const int ns = max(0, min(p.n_sink, min(p.Tk, T)));
    const int nl = max(0, min(p.n_last, min(p.Tk - ns, T - ns)));
    const int Bq = p.Tk - ns - nl;
    const u64 SHq = p.uniform_q ? (u64)T : SH; // total of what the quotas are proportional to
    long long smin = 0;
    for (int i = tid; i < n_seg; i += nt) {
        Ms[i] = p.uniform_q ? (u64)(bounds[i + 1] - bounds[i]) : Cend[i] - (i > 0 ? Cend[i - 1] : 0ull); // ablation: share by length
        smin += max(0, min(p.q_min, bounds[i + 1] - bounds[i]));
    }
    smin = block_sum_i64(smin, sm.scratch);
    const long long Trem = (long long)Bq - smin;
    long long sq = 0;
    for (int i = tid; i < n_seg; i += nt) {
        const int L = bounds[i + 1] - bounds[i];
        long long qi = max(0, min(p.q_min, L));
        if (Trem >= 0) qi += (long long)((2ull * (u64)Trem * Ms[i] + SHq) / (2ull * SHq));
        if (qi > L) qi = L;
        quota[i] = (int)qi;
        sq += qi;
    }
    sq = block_sum_i64(sq, sm.scratch);
    const long long Dq = (long long)Bq - sq;
    if (Dq > 0) {
        for (int i = tid; i < n_seg; i += nt) cap[i] = bounds[i + 1] - bounds[i] - quota[i];
        __syncthreads();
        distribute<true>(Dq, cap, give, Ms, n_seg, sm);
        for (int i = tid; i < n_seg; i += nt) quota[i] += give[i];
    } else if (Dq < 0) {
        for (int i = tid; i < n_seg; i += nt)
            cap[i] = quota[i] - max(0, min(p.q_min, bounds[i + 1] - bounds[i]));
        __syncthreads();
        const long long left = distribute<false>(-Dq, cap, give, Ms, n_seg, sm);
        for (int i = tid; i < n_seg; i += nt) quota[i] -= give[i];
        if (left > 0) { // the budget cannot cover the minima: go below them
            __syncthreads();
            for (int i = tid; i < n_seg; i += nt) cap[i] = quota[i];
            __syncthreads();
            distribute<false>(left, cap, give, Ms, n_seg, sm);
            for (int i = tid; i < n_seg; i += nt) quota[i] -= give[i];
        }
    }
    __syncthreads();
    if (rank == 0) {
        if (tid == 0) p.n_seg[uid] = n_seg;
        for (int i = tid; i < n_seg; i += nt) {
            p.seg_bounds[(size_t)uid * (sc + 1) + i] = bounds[i];
            p.quotas[(size_t)uid * sc + i] = quota[i];
        }
        if (tid == 0) p.seg_bounds[(size_t)uid * (sc + 1) + n_seg] = T;
    }

    // ---- selection machinery.
    //      seg_search finds, for all segments at once, the q_s-th largest key of each segment
    //      by fixing two key bits per round from the top: in a round every thread counts, per
    //      segment it touches, its active tokens whose key is at least prefix | j << shift
    //      (j = 1, 2, 3); one thread per segment then keeps the largest j that still leaves q_s
    //      keys at or above.  A last round counts keys >= and > the final value, which gives
    //      how many of the keys equal to it belong to the top q_s.  The count tables of even
    //      and odd rounds alternate, so one cluster barrier per round is enough.
    unsigned key[VPT];
#pragma unroll
    for (int q = 0; q < VPT / 4; ++q) {
        float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (my0 + 4 * q < n_loc) v = *reinterpret_cast<const float4 *>(gs + my0 + 4 * q);
        key[4 * q] = score_key(v.x); key[4 * q + 1] = score_key(v.y);
        key[4 * q + 2] = score_key(v.z); key[4 * q + 3] = score_key(v.w);
    }
    auto seg_search = [&](const int *quo, int nsg, unsigned act, int s0, unsigned nsb) {
        for (int s = tid; s < nsg; s += nt) cand[s] = 0u;
        for (int i = tid; i < nsg * 3; i += nt) { cnt[i] = 0; cnt[sc * 3 + i] = 0; }
        if (tid == 0) sm.bcast[7] = 0;
        const int s0_first = __shfl_sync(0xffffffffu, s0, 0); // every lane takes part (no short-circuit around it)
        const bool wuni = __all_sync(0xffffffffu, nsb == 0 && s0 == s0_first);
        __syncthreads();
        int par = 0;
        for (int shift = 30; shift >= -2; shift -= 2, par ^= 1) {
            const bool fin = shift < 0;
            int *c = cnt + par * sc * 3;
            int s = s0, c1 = 0, c2 = 0, c3 = 0;
            auto flush = [&]() {
                if (c1) atomicAdd(&c[s * 3], c1);
                if (c2) atomicAdd(&c[s * 3 + 1], c2);
                if (c3) atomicAdd(&c[s * 3 + 2], c3);
            };
            if (act) {
                unsigned P = cand[s];
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    if (i > 0 && ((nsb >> i) & 1u)) {
                        flush();
                        ++s; c1 = c2 = c3 = 0;
                        P = cand[s];
                    }
                    if ((act >> i) & 1u) {
                        const unsigned k = key[i];
                        if (!fin) {
                            c1 += k >= (P | (1u << shift));
                            c2 += k >= (P | (2u << shift));
                            c3 += k >= (P | (3u << shift));
                        } else {
                            c1 += k >= P;
                            c2 += k > P;
                        }
                    }
                }
            }
            if (wuni) {
                c1 = __reduce_add_sync(0xffffffffu, c1);
                c2 = __reduce_add_sync(0xffffffffu, c2);
                c3 = __reduce_add_sync(0xffffffffu, c3);
                if (lane == 0) flush();
            } else if (act) {
                flush();
            }
            unit_barrier();
            for (int sg = tid; sg < nsg; sg += nt) {
                int a1 = c[sg * 3], a2 = c[sg * 3 + 1], a3 = c[sg * 3 + 2];
                if (cs > 1) {
                    a1 = a2 = a3 = 0;
#pragma unroll
                    for (int r = 0; r < cs; ++r) {
                        const int *rc = cluster.map_shared_rank(c + sg * 3, r);
                        a1 += rc[0]; a2 += rc[1]; a3 += rc[2];
                    }
                }
                const int q = quo[sg];
                if (!fin) {
                    const unsigned j = a3 >= q ? 3u : (a2 >= q ? 2u : (a1 >= q ? 1u : 0u));
                    cand[sg] |= j << shift;
                } else {
                    takev[sg] = q - a2;       // keys equal to the threshold that belong to the top q
                    tiesv[sg] = a1 - a2;      // keys equal to the threshold
                    if (q - a2 < a1 - a2) sm.bcast[7] = 1;
                }
                int *z = cnt + (par ^ 1) * sc * 3 + sg * 3;
                z[0] = 0; z[1] = 0; z[2] = 0;
            }
            __syncthreads();
        }
    };
    // Marks the winners of a seg_search among this thread's tokens: keys above the segment's
    // threshold, and of the keys equal to it the first take_s in position order.
    // raise_only: only sets flags (backfill); otherwise writes the flag of every active token.
    auto seg_mark = [&](const int *bnd, unsigned act, int s0, unsigned nsb, bool raise_only) {
        const bool need_rank = sm.bcast[7] != 0;
        unsigned keepb = 0, tieb = 0;
        int my_t = 0;
        if (act) {
            int s = s0;
            unsigned th = cand[s];
            bool all_ties = takev[s] >= tiesv[s];
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                if (i > 0 && ((nsb >> i) & 1u)) { ++s; th = cand[s]; all_ties = takev[s] >= tiesv[s]; }
                if ((act >> i) & 1u) {
                    const unsigned k = key[i];
                    if (k > th) keepb |= 1u << i;
                    else if (k == th) {
                        if (all_ties) keepb |= 1u << i;
                        else { tieb |= 1u << i; ++my_t; }
                    }
                }
            }
        }
        if (need_rank) { // same decision in every thread of the cluster
            u64 before_blocks, bt;
            unit_sum((u64)my_t, &before_blocks);
            const int run0 = (int)before_blocks + (int)block_excl_scan_u64((u64)my_t, sm.scratch, &bt);
            auto tp_put = [&](int sg, int v) {
                if (cs == 1) tps[sg] = v;
                else for (int r = 0; r < cs; ++r) *cluster.map_shared_rank(tps + sg, r) = v;
            };
            if (valid) { // number of tied keys before the first token of each segment
                int s = s0, run = run0;
                if (t_base + my0 == bnd[s0]) tp_put(s0, run);
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    if (i > 0 && ((nsb >> i) & 1u)) { ++s; tp_put(s, run); }
                    if ((tieb >> i) & 1u) ++run;
                }
            }
            unit_barrier();
            if (act) {
                int s = s0, run = run0, base = tps[s], tk = takev[s];
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    if (i > 0 && ((nsb >> i) & 1u)) { ++s; base = tps[s]; tk = takev[s]; }
                    if ((tieb >> i) & 1u) { if (run - base < tk) keepb |= 1u << i; ++run; }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            if ((act >> i) & 1u) {
                if ((keepb >> i) & 1u) flags[my0 + i] = 1;
                else if (!raise_only) flags[my0 + i] = 0;
            }
        }
    };

    // ---- per-segment top-q_i by (score desc, position asc).
    //      Segments of at most 1024 tokens (always, when 0 < l_max <= 1024): one warp per
    //      segment, in the block that owns the segment's first token, keys in registers; the
    //      q-th largest key is found bit by bit from the top (count of keys >= prefix | bit,
    //      one warp reduction per bit) and the search stops as soon as exactly q keys lie at
    //      or above the prefix.  Otherwise: all segments at once with seg_search.
    if (p.l_max > 0 && p.l_max <= 1024) {
        int s_lo, s_hi; // segments whose first token this block owns
        {
            int lo = 0, hi = n_seg;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (bounds[mid] < t_base) lo = mid + 1; else hi = mid; }
            s_lo = lo;
            hi = n_seg;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (bounds[mid] < t_base + TPC) lo = mid + 1; else hi = mid; }
            s_hi = lo;
        }
        auto warp_segment = [&](auto kpl_tag, int a, int e, int q) {
            constexpr int KPL = decltype(kpl_tag)::value;
            unsigned k[KPL];
#pragma unroll
            for (int j = 0; j < KPL; ++j) {
                const int t = a + j * 32 + lane;
                k[j] = t < e ? score_key(g_at(t)) : 0u; // keys that are 0 never count below (X >= 1)
            }
            unsigned P = 0;
            bool exact = false;
            for (int bit = 31; bit >= 0; --bit) {
                const unsigned X = P | (1u << bit);
                int c = 0;
#pragma unroll
                for (int j = 0; j < KPL; ++j) c += k[j] >= X;
                c = __reduce_add_sync(0xffffffffu, c);
                if (c >= q) {
                    P = X;
                    if (c == q) { exact = true; break; }
                }
            }
            int take = 0;
            if (!exact) { // P is the q-th largest key itself; some of the keys equal to it stay out
                int c = 0;
#pragma unroll
                for (int j = 0; j < KPL; ++j) c += k[j] > P;
                take = q - __reduce_add_sync(0xffffffffu, c);
            }
            int seen = 0;
#pragma unroll
            for (int j = 0; j < KPL; ++j) {
                const int t = a + j * 32 + lane;
                const bool in = t < e;
                bool keepit = in && k[j] > P;
                const bool tie = in && k[j] == P;
                if (exact) keepit |= tie;
                else {
                    const unsigned bal = __ballot_sync(0xffffffffu, tie);
                    keepit |= tie && seen + __popc(bal & ((1u << lane) - 1u)) < take;
                    seen += __popc(bal);
                }
                if (in) flag_put(t, keepit ? 1 : 0);
            }
        };
        const int warp = tid >> 5;
        for (int s = s_lo + warp; s < s_hi; s += nt / 32) {
            const int a = bounds[s], e = bounds[s + 1], q = quota[s], L = e - a;
            if (q <= 0 || q >= L) {
                const unsigned char f = q >= L ? 1 : 0;
                for (int t = a + lane; t < e; t += 32) flag_put(t, f);
            } else if (L <= 256) {
                warp_segment(std::integral_constant<int, 8>{}, a, e, q);
            } else if (L <= 512) {
                warp_segment(std::integral_constant<int, 16>{}, a, e, q);
            } else {
                warp_segment(std::integral_constant<int, 32>{}, a, e, q);
            }
        }
    } else {
        seg_search(quota, n_seg, valid, seg0, newseg);
        seg_mark(bounds, valid, seg0, newseg, false);
    }
    unit_barrier();

    // ---- must-keep prefix and suffix; every must-keep position a segment already chose
    //      frees one slot, refilled by the best positions not yet kept (one pseudo-segment
    //      [0, T) whose candidates are the tokens without a flag)
    long long already = 0;
    for (int i = tid; i < ns + nl; i += nt) {
        const int t = (i < ns ? i : T - nl + (i - ns)) - t_base;
        if (t >= 0 && t < n_loc) { already += flags[t]; flags[t] = 1; }
    }
    const int r_fill = (int)unit_sum((u64)already, nullptr);
    if (r_fill > 0) {
        // Bit-by-bit search for the r_fill-th largest key among the unflagged tokens of the
        // whole sequence: per round one count per warp, one barrier, and every thread adds up
        // the warps' (and blocks') counts itself.  Stops once exactly r_fill keys qualify.
        unsigned act = 0;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            if (((valid >> i) & 1u) && flags[my0 + i] == 0) act |= 1u << i;
            else key[i] = 0u; // never counted (X >= 1)
        }
        constexpr int nwarps = nt / 32;
        int *wc = wcnt;
        auto unit_count = [&](int c, int n) -> int {
            c = __reduce_add_sync(0xffffffffu, c);
            int *mine = wc + (n & 1) * 32;
            if (lane == 0) mine[tid >> 5] = c;
            unit_barrier();
            int v = 0;
            if (cs == 1) v = lane < nwarps ? mine[lane] : 0;
            else {
#pragma unroll
                for (int r = 0; r < cs; ++r) v += lane < nwarps ? cluster.map_shared_rank(mine, r)[lane] : 0;
            }
            return __reduce_add_sync(0xffffffffu, v);
        };
        unsigned P = 0;
        bool exact = false;
        int n = 0;
        for (int bit = 31; bit >= 0; --bit, ++n) {
            const unsigned X = P | (1u << bit);
            int c = 0;
#pragma unroll
            for (int i = 0; i < VPT; ++i) c += key[i] >= X;
            const int tot = unit_count(c, n);
            if (tot >= r_fill) {
                P = X;
                if (tot == r_fill) { exact = true; break; }
            }
        }
        unsigned keepb = 0, tieb = 0;
        int my_t = 0;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            if ((act >> i) & 1u) {
                if (key[i] > P || (exact && key[i] == P)) keepb |= 1u << i;
                else if (key[i] == P) { tieb |= 1u << i; ++my_t; }
            }
        }
        if (!exact) { // the first (r_fill - #keys above P) of the keys equal to P, in position order
            int c = 0;
#pragma unroll
            for (int i = 0; i < VPT; ++i) c += key[i] > P;
            const int take = r_fill - unit_count(c, n);
            u64 before_blocks, bt;
            unit_sum((u64)my_t, &before_blocks);
            int rk = (int)before_blocks + (int)block_excl_scan_u64((u64)my_t, sm.scratch, &bt);
#pragma unroll
            for (int i = 0; i < VPT; ++i)
                if ((tieb >> i) & 1u) { if (rk < take) keepb |= 1u << i; ++rk; }
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            if ((keepb >> i) & 1u) flags[my0 + i] = 1;
    }
    __syncthreads();

    // ---- ordered compaction of the kept positions; credit rows travel with their tokens
    //      and rows beyond the budget start from zero
    unsigned kept_bits = 0;
    int n_kept = 0;
#pragma unroll
    for (int i = 0; i < VPT; ++i)
        if (my0 + i < n_loc && flags[my0 + i]) { kept_bits |= 1u << i; ++n_kept; }
    u64 before_blocks, btot3;
    const int total = (int)unit_sum((u64)n_kept, &before_blocks);
    int pos = (int)before_blocks + (int)block_excl_scan_u64((u64)n_kept, sm.scratch, &btot3);
    if (total != p.Tk) {
        if (tid == 0 && rank == 0) set_status(p.status, AMS_ERR_INTERNAL, uid, total, p.Tk);
    } else {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            if (kept_bits & (1u << i)) {
                keep[pos] = t_base + my0 + i;
                if (ema_on) credit[pos] = crs[i * nt + tid];
                ++pos;
            }
        }
        if (ema_on) { // rows beyond the budget: whole groups of four with one store
#pragma unroll
            for (int q = 0; q < VPT / 4; ++q) {
                const int t = t_base + my0 + 4 * q;
                if (my0 + 4 * q + 3 < n_loc && t >= p.Tk) {
                    *reinterpret_cast<float4 *>(credit + t) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (my0 + 4 * q + k < n_loc && t + k >= p.Tk) credit[t + k] = 0.0f;
                }
            }
        }
    }
    if (cs > 1) cluster.sync(); // nobody leaves while a neighbour may still read its shared memory
}

template <int NT, int VPT, int CS>
__global__ void __launch_bounds__(NT, 1) k_segment_select_cluster(DevParams p, int cs_max)
{
    segment_unit<NT, VPT, CS>(p, blockIdx.x / CS, cs_max);
}

// Work-queue form for sequences that fit one block: a persistent grid (one block per SM) takes the units
// one by one.  Units rarely fill a whole number of waves, and their selection phases leave the memory
// system idle: a block that finds no unit left starts on the paged compaction (the two display
// equations of the paged-KV appendix: K_new[pi_new(b, j), h, :] <- K_old[pi_old(b, I_j), h, :], same
// for V), chunk by chunk in (layer, sequence) order, for as long as other blocks are still selecting.
// The gather kernel that follows moves the chunks that were not handed out (it has twice the threads
// per SM, hence twice the bytes in flight, and is the faster mover once every SM is free).
// ctrl: [0] next unit, [1] chunks handed out, [3] units finished, [4 + layer * B + b] heads of that
// pair finished; the table-update kernel puts them back to zero.  A chunk is only ever handed out after
// every unit has been handed out, so whoever it waits for is running; the wait is bounded all the same.
constexpr uint32_t kDoneSpins = 1u << 22;

template <int NT, int VPT>
__global__ void __launch_bounds__(NT, 1) k_segment_select_move(DevParams p, int *ctrl)
{
    __shared__ int item_s;
    const int tid = threadIdx.x;
    const int units = p.L * p.B * p.H;
    wait_for_previous_kernel(); // the scores
    for (;;) {
        __syncthreads(); // the previous unit's shared memory is no longer read
        if (tid == 0) item_s = atomicAdd(&ctrl[0], 1);
        __syncthreads();
        const int uid = item_s;
        if (uid >= units) break;
        segment_unit<NT, VPT, 1>(p, uid, 1);
        __syncthreads(); // every thread's writes of the unit (kept positions, credit) are issued
        if (tid == 0) {
            __threadfence();
            atomicAdd(&ctrl[4 + uid / p.H], 1);
            atomicAdd(&ctrl[3], 1);
        }
    }
    const int rows_lb = p.Tk * p.H, chunks = (rows_lb + kMoveRows - 1) / kMoveRows, n_items = p.L * p.B * chunks;
    for (;;) {
        __syncthreads();
        if (tid == 0) {
            int it = n_items;
            // once every unit is finished the rest is left to the gather kernel; the comparison and the
            // claim are not atomic together, which at worst hands out one more chunk per block
            if (*reinterpret_cast<const volatile int *>(ctrl + 3) < units) {
                it = atomicAdd(&ctrl[1], 1);
                if (it >= n_items) atomicSub(&ctrl[1], 1); // keep the count at the chunks really handed out
            }
            if (it < n_items) {
                const volatile int *done = ctrl + 4 + it / chunks;
                uint32_t spins = 0;
                while (*done < p.H && ++spins < kDoneSpins) __nanosleep(128);
                if (*done < p.H) { set_status(p.status, AMS_ERR_TIMEOUT, it, 0, 0); it = n_items; }
                __threadfence();
            }
            item_s = it;
        }
        __syncthreads();
        const int it = item_s;
        if (it >= n_items) break;
        const int lb = it / chunks, b = lb % p.B, l = lb / p.B;
        const int T = p.seq_lens[b];
        // sequences that were skipped or reported keep their rows
        if (T <= p.Tk || T > p.T_cap) continue;
        const int r_end = min(rows_lb, (it % chunks + 1) * kMoveRows);
        const int *table = p.block_table + (size_t)b * p.bt_stride;
        const int *dstp = p.dst_pages + (size_t)b * p.n_dst;
        const int *keep_base = p.keep_idx + (size_t)lb * p.H * p.Tk;
        const int l16 = tid & 15;
        constexpr int kUnroll = 4, kRowsPerIter = NT / 16, kStep = kRowsPerIter * kUnroll;
        // Rows are numbered r = j * H + h, so that consecutive rows are consecutive 256-byte pieces of the
        // destination page.  The source offsets of the next round (kept position, then its page: two
        // dependent loads) are fetched while this round's rows are in flight.
        auto source_of = [&](int r) -> size_t {
            const int j = r / p.H, h = r - j * p.H;
            const int pos = __ldcg(keep_base + (size_t)h * p.Tk + j);
            return row_offset(p, l, table[pos >> 4], pos & 15, h) + l16 * 8;
        };
        const int r_first = (it % chunks) * kMoveRows + (tid >> 4);
        size_t soff_next[kUnroll];
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const int r = r_first + i * kRowsPerIter;
            soff_next[i] = r < r_end ? source_of(r) : 0;
        }
        for (int r0 = r_first; r0 < r_end; r0 += kStep) {
            uint4 kv[kUnroll], vv[kUnroll];
#pragma unroll
            for (int i = 0; i < kUnroll; ++i) {
                if (r0 + i * kRowsPerIter < r_end) {
                    kv[i] = ld_stream16(p.k_pages + soff_next[i]);
                    vv[i] = ld_stream16(p.v_pages + soff_next[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < kUnroll; ++i) {
                const int r = r0 + kStep + i * kRowsPerIter;
                soff_next[i] = r < r_end ? source_of(r) : 0;
            }
#pragma unroll
            for (int i = 0; i < kUnroll; ++i) {
                const int r = r0 + i * kRowsPerIter;
                if (r < r_end) {
                    const int j = r / p.H, h = r - j * p.H;
                    const size_t doff = row_offset(p, l, dstp[j >> 4], j & 15, h) + l16 * 8;
                    st_stream16(p.k_pages + doff, kv[i]);
                    st_stream16(p.v_pages + doff, vv[i]);
                }
            }
        }
    }
}

template <int NT, int VPT, int CS>
int launch_cfg(const DevParams &p, LaunchCtx &ctx, int cs_max, size_t smem)
{
    static size_t configured = 0;
    if (smem > configured) {
        if (cudaFuncSetAttribute(k_segment_select_cluster<NT, VPT, CS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return AMS_ERR_CUDA;
        configured = smem;
    }
    const int units = p.L * p.B * p.H;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)(units * CS), 1, 1);
    cfg.blockDim = dim3(NT, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = ctx.s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, k_segment_select_cluster<NT, VPT, CS>, p, cs_max) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernSegmentSelect);
    return AMS_OK;
}

} // namespace

// True when the work-queue kernel takes the call: every sequence fits one block.  It also moves part of the kept rows.
static int sm_count()
{
    static int n_sm = 0;
    if (!n_sm) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n_sm = 0;
    }
    return n_sm;
}

// With more units than SMs there is a last, partial wave to fill; with fewer the plain kernel is quicker.
bool segment_moves_rows(const DevParams &p)
{
    return segment_cluster_supported(p) && p.T_cap <= kNT * 16 && sm_count() > 0 && p.L * p.B * p.H > sm_count();
}

template <int VPT>
int launch_move(const DevParams &p, LaunchCtx &ctx, size_t smem)
{
    static size_t configured = 0;
    const int n_sm = sm_count();
    if (n_sm <= 0) return AMS_ERR_CUDA;
    if (smem > configured) {
        if (cudaFuncSetAttribute(k_segment_select_move<kNT, VPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return AMS_ERR_CUDA;
        configured = smem;
    }
    const int units = p.L * p.B * p.H;
    const int chunks = (p.Tk * p.H + kMoveRows - 1) / kMoveRows;
    const int most = units > p.L * p.B * chunks ? units : p.L * p.B * chunks;
    const int grid = most < n_sm ? most : n_sm;
    if (launch_after(k_segment_select_move<kNT, VPT>, dim3((unsigned)grid), dim3(kNT), smem, ctx.s, p, p.qctrl) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernSegmentSelect);
    return AMS_OK;
}

// True when the on-chip kernel can take this call: the sequence capacity fits one cluster of
// at most eight blocks and the segment tables fit beside the per-token arrays.
bool segment_cluster_supported(const DevParams &p)
{
    if (p.T_cap > 8 * kNT * 16) return false;
    const int vpt = p.T_cap <= kNT * 4 ? 4 : (p.T_cap <= kNT * 8 ? 8 : 16);
    return smem_map(kNT * vpt, p.seg_cap, p.S, p.beta != 1.0f).total <= (size_t)200 * 1024;
}

int launch_segment_select_cluster(const DevParams &p, LaunchCtx &ctx)
{
    const bool ema_on = p.beta != 1.0f;
    if (segment_moves_rows(p)) {
        if (p.T_cap <= kNT * 4) return launch_move<4>(p, ctx, smem_map(kNT * 4, p.seg_cap, p.S, ema_on).total);
        if (p.T_cap <= kNT * 8) return launch_move<8>(p, ctx, smem_map(kNT * 8, p.seg_cap, p.S, ema_on).total);
        return launch_move<16>(p, ctx, smem_map(kNT * 16, p.seg_cap, p.S, ema_on).total);
    }
    if (p.T_cap <= kNT * 4) return launch_cfg<kNT, 4, 1>(p, ctx, 1, smem_map(kNT * 4, p.seg_cap, p.S, ema_on).total);
    if (p.T_cap <= kNT * 8) return launch_cfg<kNT, 8, 1>(p, ctx, 1, smem_map(kNT * 8, p.seg_cap, p.S, ema_on).total);
    const int tpc = kNT * 16;
    const int cs_need = (p.T_cap + tpc - 1) / tpc;
    int cs_max = 1;
    while (cs_max < cs_need) cs_max *= 2; // cluster sizes are powers of two
    // Sequence lengths are known on the device only: one launch per cluster size, each taking the
    // sequences that need exactly that many blocks (the blocks of the others leave at once), so that a
    // short sequence of a ragged batch does not pay for the cluster barriers of the longest one.
    const size_t smem = smem_map(tpc, p.seg_cap, p.S, ema_on).total;
    int rc = launch_cfg<kNT, 16, 1>(p, ctx, cs_max, smem);
    if (rc == AMS_OK && cs_max >= 2) rc = launch_cfg<kNT, 16, 2>(p, ctx, cs_max, smem);
    if (rc == AMS_OK && cs_max >= 4) rc = launch_cfg<kNT, 16, 4>(p, ctx, cs_max, smem);
    if (rc == AMS_OK && cs_max >= 8) rc = launch_cfg<kNT, 16, 8>(p, ctx, cs_max, smem);
    return rc;
}

} // namespace ams
