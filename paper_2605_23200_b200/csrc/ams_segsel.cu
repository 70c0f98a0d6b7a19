// Algorithm 1 steps 1-5 of the paper as three throughput-oriented kernels over all (layer, sequence,
// KV head) units of an event:
//
//   k_mass_scan        Eq. 1 on fixed-point weights, the EMA credit update and the history-aware mass
//                      (Section 3.3, "EMA credit"; Algorithm 1 steps 1-2), and the inclusive prefix sum of
//                      the integer mass with the mass-quantile cuts b_k = min{t : c(t) >= k / S} (Algorithm 1
//                      step 3).  One block per unit streams the unit's usage row from L2 once per reduction
//                      that the arithmetic needs.
//   k_segments_quotas  merge of short and split of long segments, quotas with their adjustment (Section
//                      3.3; Algorithm 1 steps 3-4).  One warp per unit: the work is a few dozen segments,
//                      serial in part, and running all units' warps side by side hides that latency.
//   k_select_compact   per-segment top-q_i, must-keep prefix and suffix, backfill, ordered kept positions
//                      and the credit rows that travel with them (Algorithm 1 step 5).  One block per
//                      unit; a warp per short segment, the block per long one; kept flags are one bit per
//                      token in shared memory.
//
// Every decision is integer arithmetic on fixed-point images of the mass (kFixBits fractional bits) and
// every floating-point step a single round-to-nearest operation, so results do not depend on the order in
// which a block adds things up.  Selection order is (score key descending, position ascending), a strict
// total order: the q-th element is found by fixing key bits from the top and, among keys equal to the
// threshold, position bits.
#include <type_traits>

#include "ams_common.cuh"
#include "ams_select.cuh"

namespace ams {

using namespace sel;

namespace {

constexpr int kScanVec = 8;                 // tokens per thread and round of the scan pass
constexpr int kListCap = 1024;              // backfill candidates kept in shared memory

struct UnitId { int l, b, h; };
__device__ __forceinline__ UnitId unit_of(const DevParams &p, int uid)
{
    UnitId u;
    u.h = uid % p.H; u.b = (uid / p.H) % p.B; u.l = uid / (p.H * p.B);
    return u;
}

// ------------------------------------------------------------------------------------------ k_mass_scan

// Walks the first `n` floats of a row (allocated to a multiple of 4) with float4 loads, four per thread in
// flight: f(t, v, full) gets the position of the group's first element and, as a compile-time flag, whether
// the whole group lies inside the row (then no per-element bound is needed).
template <int NT, typename F>
__device__ __forceinline__ void walk4(const float *row, int n, F f)
{
    const int n4 = (n + 3) & ~3;
    const int tid = threadIdx.x;
    for (int base = 0; base < n4; base += NT * 16) {
        float4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = base + (j * NT + tid) * 4;
            v[j] = t < n4 ? *reinterpret_cast<const float4 *>(row + t) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = base + (j * NT + tid) * 4;
            if (t + 3 < n) f(t, v[j], std::true_type{});
            else if (t < n) f(t, v[j], std::false_type{});
        }
    }
}

// The same over two rows at once (usage and credit).
template <int NT, typename F>
__device__ __forceinline__ void walk4x2(const float *row_a, const float *row_b, int n, F f)
{
    const int n4 = (n + 3) & ~3;
    const int tid = threadIdx.x;
    for (int base = 0; base < n4; base += NT * 16) {
        float4 va[4], vb[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = base + (j * NT + tid) * 4;
            va[j] = vb[j] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (t < n4) { va[j] = *reinterpret_cast<const float4 *>(row_a + t); vb[j] = *reinterpret_cast<const float4 *>(row_b + t); }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = base + (j * NT + tid) * 4;
            if (t + 3 < n) f(t, va[j], vb[j], std::true_type{});
            else if (t < n) f(t, va[j], vb[j], std::false_type{});
        }
    }
}

// Block-wide sum of doubles that are integers below 2^53 (exact, hence independent of the order).
__device__ __forceinline__ double block_sum_exact_f64(double v, u64 *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = (u64)__double_as_longlong(v);
    __syncthreads();
    if (warp == 0) {
        double x = lane < nw ? __longlong_as_double((long long)scratch[lane]) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        if (lane == 0) scratch[32] = (u64)__double_as_longlong(x);
    }
    __syncthreads();
    return __longlong_as_double((long long)scratch[32]);
}

// raw_cuts: [units][S + 1] cut positions of the mass quantiles (entry k: boundary after the token that
// reaches k / S; T where no token before the last one does).
template <int NT>
__global__ void __launch_bounds__(NT) k_mass_scan(DevParams p)
{
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ u64 scratch[40];
    u64 *qthr = reinterpret_cast<u64 *>(dyn); // [S]: prefix value at which quantile k is reached
    const int tid = threadIdx.x, uid = blockIdx.x;
    const UnitId un = unit_of(p, uid);
    const int T = p.seq_lens[un.b];
    if (T <= p.Tk || T > p.T_cap) return;
    const size_t row = (size_t)uid * p.T_cap;
    const float *u = p.usage + row;
    float *credit = p.ema + (((size_t)un.l * p.Bmax + un.b) * p.H + un.h) * (size_t)p.T_cap;
    u64 *C = p.cbuf + row;
    int *raw = p.raw_cuts + (size_t)uid * (p.S + 1);
    float *mass_dbg = p.mass_dbg ? p.mass_dbg + row : nullptr;
    const bool ema_on = p.beta != 1.0f;
    const double two_f = (double)(1ull << kFixBits);
    wait_for_previous_kernel(); // the usage scores
    for (int k = tid; k <= p.S; k += NT) raw[k] = T;

    // Rows are allocated to the capacity (a multiple of 16), so whole float4 groups may be read past the
    // sequence's end; what lies there is masked by position.
    // ---- largest Eq. 1 weight -> exponent of the fixed-point images
    float wmax = 0.0f;
    walk4<NT>(u, T, [&](int t, float4 v, auto full) {
        const float w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) if (decltype(full)::value || t + i < T) wmax = fmaxf(wmax, weight_of(w[i], p.eps));
    });
    wmax = block_max_f32(wmax, scratch);
    const int ew = fix_exponent(wmax);
    // ---- SA = sum of the images A_t = floor(w_t 2^(36 - ew)), held as doubles (integers below 2^53: exact)
    const double scale_w = fix_scale_of(ew);
    const float cut_w = fixed_trunc_threshold(ew); // weights below it lose their bits under the image's last one
    double sa = 0.0;
    walk4<NT>(u, T, [&](int t, float4 v, auto full) {
        const float w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (decltype(full)::value || t + i < T) sa = __dadd_rn(sa, __dmul_rn((double)fixed_trunc_by_add(weight_of(w[i], p.eps), cut_w), scale_w));
    });
    const double SA = block_sum_exact_f64(sa, scratch);
    const double inv_sa = __ddiv_rn(1.0, SA);          // normalisations multiply by the rounded reciprocal
    const double inv_sa_w = __dmul_rn(inv_sa, scale_w); // A_t / SA = trunc(w_t) * (2^(36 - ew) / SA): the scaling is exact

    // ---- EMA credit: c <- lambda c + (1 - lambda) m, updated in place (the block-wide reductions that follow
    //      make every thread's writes visible to the others before anybody reads them back)
    int ec = 0;
    float cut_c = 0.0f;
    double inv_sc_c = 0.0; // 2^(36 - ec) / SC
    bool have_credit = false;
    if (ema_on) {
        const float oml = __fsub_rn(1.0f, p.lambda);
        float cmax = 0.0f;
        walk4x2<NT>(u, credit, T, [&](int t, float4 v, float4 cv, auto full) {
            const float w[4] = {v.x, v.y, v.z, v.w};
            float c[4] = {cv.x, cv.y, cv.z, cv.w};
            float m[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                m[i] = __double2float_rn(__dmul_rn((double)fixed_trunc_by_add(weight_of(w[i], p.eps), cut_w), inv_sa_w));
                if (decltype(full)::value || t + i < T) {
                    c[i] = __fadd_rn(__fmul_rn(p.lambda, c[i]), __fmul_rn(oml, m[i]));
                    cmax = fmaxf(cmax, c[i]);
                }
            }
            if (decltype(full)::value) {
                *reinterpret_cast<float4 *>(credit + t) = make_float4(c[0], c[1], c[2], c[3]);
                if (mass_dbg) *reinterpret_cast<float4 *>(mass_dbg + t) = make_float4(m[0], m[1], m[2], m[3]);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (t + i < T) { credit[t + i] = c[i]; if (mass_dbg) mass_dbg[t + i] = m[i]; }
            }
        });
        cmax = block_max_f32(cmax, scratch);
        double scsum = 0.0;
        double scale_c = 0.0;
        if (cmax > 0.0f) {
            ec = fix_exponent(cmax);
            scale_c = fix_scale_of(ec);
            cut_c = fixed_trunc_threshold(ec);
            walk4<NT>(credit, T, [&](int t, float4 cv, auto full) {
                const float c[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (decltype(full)::value || t + i < T) scsum = __dadd_rn(scsum, __dmul_rn((double)fixed_trunc_by_add(c[i], cut_c), scale_c));
            });
        }
        const double SC = block_sum_exact_f64(scsum, scratch);
        have_credit = SC > 0.0;
        if (have_credit) inv_sc_c = __dmul_rn(__ddiv_rn(1.0, SC), scale_c);
    }

    // ---- history-aware integer mass Hm_t = floor((beta m + (1 - beta) normalize(c)) 2^36) and its inclusive
    //      prefix sum, kScanVec consecutive tokens per thread and round; the next round's inputs are fetched
    //      before this round's block-wide scan
    const double bd = (double)p.beta, omb = __dsub_rn(1.0, (double)p.beta);
    u64 carry = 0;
    constexpr int kRound = NT * kScanVec;
    float4 wn[kScanVec / 4], cn[kScanVec / 4];
    auto fetch = [&](int base) {
#pragma unroll
        for (int q = 0; q < kScanVec / 4; ++q) {
            const int t = base + tid * kScanVec + 4 * q;
            wn[q] = cn[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (t < T) {
                wn[q] = *reinterpret_cast<const float4 *>(u + t);
                if (have_credit) cn[q] = *reinterpret_cast<const float4 *>(credit + t);
            }
        }
    };
    fetch(0);
    for (int base = 0; base < T; base += kRound) {
        const int t0 = base + tid * kScanVec;
        u64 Hm[kScanVec];
        u64 tot8 = 0;
        float4 wv[kScanVec / 4], cv[kScanVec / 4];
#pragma unroll
        for (int q = 0; q < kScanVec / 4; ++q) { wv[q] = wn[q]; cv[q] = cn[q]; }
        if (base + kRound < T) fetch(base + kRound);
#pragma unroll
        for (int q = 0; q < kScanVec / 4; ++q) {
            const int t = t0 + 4 * q;
            const float w[4] = {wv[q].x, wv[q].y, wv[q].z, wv[q].w}, c[4] = {cv[q].x, cv[q].y, cv[q].z, cv[q].w};
            float m[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                u64 h = 0;
                m[i] = 0.0f;
                if (t + i < T) {
                    const double r = __dmul_rn((double)fixed_trunc_by_add(weight_of(w[i], p.eps), cut_w), inv_sa_w);
                    if (ema_on) {
                        double hist = 0.0;
                        if (have_credit) hist = __dmul_rn(omb, __dmul_rn((double)fixed_trunc_by_add(c[i], cut_c), inv_sc_c));
                        h = floor_to_u64(__dmul_rn(__dadd_rn(__dmul_rn(bd, r), hist), two_f));
                    } else {
                        m[i] = __double2float_rn(r);
                        h = floor_to_u64(__dmul_rn(r, two_f));
                    }
                }
                Hm[4 * q + i] = h;
                tot8 += h;
            }
            if (!ema_on && mass_dbg && t < T) {
                if (t + 3 < T) *reinterpret_cast<float4 *>(mass_dbg + t) = make_float4(m[0], m[1], m[2], m[3]);
                else
#pragma unroll
                    for (int i = 0; i < 4; ++i) if (t + i < T) mass_dbg[t + i] = m[i];
            }
        }
        u64 tot;
        u64 run = carry + block_excl_scan_u64(tot8, scratch, &tot);
        carry += tot;
        if (t0 < T) { // rows have the capacity's length: whole pairs are written, positions past T are never read
#pragma unroll
            for (int q = 0; q < kScanVec / 2; ++q) {
                ulonglong2 o;
                run += Hm[2 * q]; o.x = run;
                run += Hm[2 * q + 1]; o.y = run;
                if (t0 + 2 * q < T) *reinterpret_cast<ulonglong2 *>(C + t0 + 2 * q) = o;
            }
        }
    }
    if (p.fixed_seg) return; // component ablation: the cuts do not depend on the mass (the next kernel places them)

    // ---- mass-quantile cuts: the token that reaches quantile k closes its segment, so the boundary is
    //      (position + 1).  c(t) >= k / S  <=>  C(t) S >= k SH  <=>  C(t) >= ceil(k SH / S).  A thread looks at
    //      the prefix before its first and at its last token of a round and walks its tokens only if a
    //      quantile lies between the two.
    const u64 SH = carry, S = (u64)p.S;
    for (int k = tid + 1; k < p.S; k += NT) qthr[k] = ((u64)k * SH + S - 1) / S;
    __syncthreads(); // (also orders the prefix sums written above before the reads below)
    auto quantile = [&](u64 c) -> int { // number of k in [1, S) with qthr[k] <= c
        int lo = 0, hi = p.S - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (qthr[mid] <= c) lo = mid; else hi = mid - 1;
        }
        return lo;
    };
    for (int base = 0; base < T; base += 4 * kRound) {
        u64 before[4], last[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t0 = base + j * kRound + tid * kScanVec;
            before[j] = last[j] = 0;
            if (t0 < T) {
                before[j] = t0 > 0 ? C[t0 - 1] : 0ull;
                last[j] = C[min(t0 + kScanVec, T) - 1];
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t0 = base + j * kRound + tid * kScanVec;
            if (t0 >= T) continue;
            int kprev = quantile(before[j]);
            const int klast = quantile(last[j]);
            if (klast == kprev) continue;
            for (int i = 0; i < kScanVec && t0 + i < T; ++i) {
                const int kc = quantile(C[t0 + i]);
                for (int k = kprev + 1; k <= kc; ++k) raw[k] = t0 + i + 1;
                kprev = kc;
            }
        }
    }
}

// ------------------------------------------------------------------------------------ k_segments_quotas

__device__ __forceinline__ long long warp_sum_i64(long long v) { return (long long)warp_sum_u64((u64)v); }
__device__ __forceinline__ int warp_max_i32(int v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// The cycling quota adjustment in closed form, for one warp: `D` (> 0) tokens go to segments one per visit
// in the visiting order, segment i taking at most cap[i]; every segment receives min(cap, level) with
// `level` the largest whose total fits, and the first `rem` segments in visiting order that still have room
// receive one more.  kHeavyFirst: order (M desc, i asc); otherwise (M asc, i desc).  Returns what is left.
template <bool kHeavyFirst>
__device__ long long warp_distribute(long long D, const int *cap, int *give, const u64 *M, int n_seg)
{
    const int lane = threadIdx.x & 31;
    long long cnt1 = 0, tot = 0;
    int mx = 0;
    for (int i = lane; i < n_seg; i += 32) {
        cnt1 += cap[i] >= 1;
        tot += cap[i];
        mx = max(mx, cap[i]);
    }
    cnt1 = warp_sum_i64(cnt1);
    tot = warp_sum_i64(tot);
    mx = warp_max_i32(mx);
    long long level = 0, used = 0;
    if (tot <= D) {
        level = mx;
        used = tot;
    } else if (cnt1 <= D) {
        long long lo = 1, hi = mx; // F(lo) <= D < F(hi), F(k) = sum of min(cap, k)
        used = cnt1;
        while (hi - lo > 1) {
            const long long mid = (lo + hi) >> 1;
            long long f = 0;
            for (int i = lane; i < n_seg; i += 32) f += min((long long)cap[i], mid);
            f = warp_sum_i64(f);
            if (f <= D) { lo = mid; used = f; } else hi = mid;
        }
        level = lo;
    }
    const long long rem = D - used;
    for (int i = lane; i < n_seg; i += 32) {
        int g = (int)min((long long)cap[i], level);
        if (rem > 0 && cap[i] > level) {
            long long rank = 0;
            const u64 Mi = M[i];
            for (int j = 0; j < n_seg; ++j) {
                if (cap[j] <= level) continue;
                const u64 Mj = M[j];
                rank += kHeavyFirst ? (Mj > Mi || (Mj == Mi && j < i)) : (Mj < Mi || (Mj == Mi && j > i));
            }
            if (rank < rem) ++g;
        }
        give[i] = g;
    }
    __syncwarp();
    return tot <= D ? D - tot : 0;
}

struct QuotaSmem { size_t ms, bounds, quota, cap, give, raw, merged, poff, total; };
__host__ __device__ inline QuotaSmem quota_smem(int sc, int S)
{
    QuotaSmem m;
    size_t o = 0;
    m.ms = o;     o += (size_t)sc * 8;
    m.bounds = o; o += (size_t)(sc + 1) * 4;
    m.quota = o;  o += (size_t)sc * 4;
    m.cap = o;    o += (size_t)sc * 4;
    m.give = o;   o += (size_t)sc * 4;
    m.raw = o;    o += (size_t)(S + 1) * 4;
    m.merged = o; o += (size_t)(S + 1) * 4;
    m.poff = o;   o += (size_t)(S + 1) * 4;
    m.total = (o + 15) & ~(size_t)15;
    return m;
}

__global__ void __launch_bounds__(32) k_segments_quotas(DevParams p)
{
    extern __shared__ __align__(16) unsigned char dyn[];
    const int lane = threadIdx.x, uid = blockIdx.x;
    const UnitId un = unit_of(p, uid);
    const int T = p.seq_lens[un.b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int sc = p.seg_cap;
    const QuotaSmem mp = quota_smem(sc, p.S);
    u64 *Ms = reinterpret_cast<u64 *>(dyn + mp.ms);
    int *bounds = reinterpret_cast<int *>(dyn + mp.bounds);
    int *quota = reinterpret_cast<int *>(dyn + mp.quota);
    int *cap = reinterpret_cast<int *>(dyn + mp.cap);
    int *give = reinterpret_cast<int *>(dyn + mp.give);
    int *raw = reinterpret_cast<int *>(dyn + mp.raw);
    int *merged = reinterpret_cast<int *>(dyn + mp.merged);
    int *poff = reinterpret_cast<int *>(dyn + mp.poff);
    wait_for_previous_kernel(); // the prefix sums
    const u64 *C = p.cbuf + (size_t)uid * p.T_cap;
    const u64 SH = C[T - 1];
    // ---- raw cuts of the mass quantiles, found by the scan kernel (a cut at or beyond T means "none")
    for (int k = lane + 1; k < p.S; k += 32)
        raw[k] = p.fixed_seg ? (int)(((long long)k * T) / p.S)  // component ablation: boundary k at floor(k T / S)
                             : p.raw_cuts[(size_t)uid * (p.S + 1) + k];
    __syncwarp();

    // ---- merge short raw segments forward, fold a short tail left, count split pieces
    int n_merged = 0, n_seg = 0;
    if (lane == 0) {
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
        n_merged = nm - 1;
        n_seg = off;
    }
    __syncwarp(); // lane 0's tables are read by every lane below
    n_merged = __shfl_sync(0xffffffffu, n_merged, 0);
    n_seg = __shfl_sync(0xffffffffu, n_seg, 0);
    if (n_seg > sc) { // cannot happen with the capacity formula of the header; reported all the same
        if (lane == 0) { set_status(p.status, AMS_ERR_CAPACITY, uid, n_seg, sc); p.n_seg[uid] = -1; p.seq_bad[un.b] = 1; }
        return;
    }
    if (lane == 0) bounds[0] = 0;
    for (int i = 0; i < n_merged; ++i) {
        const int a = merged[i], len = merged[i + 1] - a, pieces = poff[i + 1] - poff[i];
        const int bs = len / pieces, extra = len % pieces;
        for (int j = lane; j < pieces; j += 32) bounds[poff[i] + j + 1] = a + (j + 1) * bs + min(j + 1, extra);
    }
    __syncwarp();

    // ---- must-keep sizes and quotas: q_i = q_i^min + round(T_rem M_i / sum M), clipped, then adjusted
    const int ns = max(0, min(p.n_sink, min(p.Tk, T)));
    const int nl = max(0, min(p.n_last, min(p.Tk - ns, T - ns)));
    const int Bq = p.Tk - ns - nl;
    const u64 SHq = p.uniform_q ? (u64)T : SH; // total of what the quotas are proportional to
    long long smin = 0;
    for (int i = lane; i < n_seg; i += 32) {
        const int a = bounds[i], e = bounds[i + 1];
        Ms[i] = p.uniform_q ? (u64)(e - a) : C[e - 1] - (a > 0 ? C[a - 1] : 0ull); // ablation: share by length
        smin += max(0, min(p.q_min, e - a));
    }
    smin = warp_sum_i64(smin);
    const long long Trem = (long long)Bq - smin;
    long long sq = 0;
    for (int i = lane; i < n_seg; i += 32) {
        const int L = bounds[i + 1] - bounds[i];
        long long qi = max(0, min(p.q_min, L));
        if (Trem >= 0) qi += (long long)((2ull * (u64)Trem * Ms[i] + SHq) / (2ull * SHq));
        if (qi > L) qi = L;
        quota[i] = (int)qi;
        sq += qi;
    }
    sq = warp_sum_i64(sq);
    const long long Dq = (long long)Bq - sq;
    if (Dq > 0) {
        for (int i = lane; i < n_seg; i += 32) cap[i] = bounds[i + 1] - bounds[i] - quota[i];
        __syncwarp();
        warp_distribute<true>(Dq, cap, give, Ms, n_seg);
        for (int i = lane; i < n_seg; i += 32) quota[i] += give[i];
    } else if (Dq < 0) {
        for (int i = lane; i < n_seg; i += 32) cap[i] = quota[i] - max(0, min(p.q_min, bounds[i + 1] - bounds[i]));
        __syncwarp();
        const long long left = warp_distribute<false>(-Dq, cap, give, Ms, n_seg);
        for (int i = lane; i < n_seg; i += 32) quota[i] -= give[i];
        if (left > 0) { // the budget cannot cover the minima: go below them
            __syncwarp();
            for (int i = lane; i < n_seg; i += 32) cap[i] = quota[i];
            __syncwarp();
            warp_distribute<false>(left, cap, give, Ms, n_seg);
            for (int i = lane; i < n_seg; i += 32) quota[i] -= give[i];
        }
    }
    __syncwarp();
    if (lane == 0) { p.n_seg[uid] = n_seg; p.seg_bounds[(size_t)uid * (sc + 1) + n_seg] = T; }
    for (int i = lane; i < n_seg; i += 32) {
        p.seg_bounds[(size_t)uid * (sc + 1) + i] = bounds[i];
        p.quotas[(size_t)uid * sc + i] = quota[i];
    }
}

// ------------------------------------------------------------------------------------- k_select_compact

struct SelSmem { size_t mask, bounds, quota, list, total; };
__host__ __device__ inline SelSmem sel_smem(int T_cap, int sc)
{
    SelSmem m;
    size_t o = 0;
    m.mask = o;   o += (size_t)((T_cap + 31) / 32 + 1) * 4;
    m.bounds = o; o += (size_t)(sc + 1) * 4;
    m.quota = o;  o += (size_t)sc * 4;
    o = (o + 7) & ~(size_t)7;
    m.list = o;   o += (size_t)kListCap * 8;
    m.total = (o + 15) & ~(size_t)15;
    return m;
}

struct SelShared {
    u64 scratch[40];
    int wc[2][32];   // per-warp counts of even / odd search rounds
    int n_list;
    unsigned bound;
    unsigned tmax[512];
};

// Sum of one count per thread over the block with one barrier per call: counts of consecutive calls land in
// alternating tables, so a table is rewritten only after every thread has passed the barrier that follows
// its last read.
template <int NT, int GT = NT>
__device__ __forceinline__ int block_count(int c, int round, SelShared &sh)
{
    // GT = NT: the whole block counts together; GT < NT: the block's teams of GT threads count on their own, each
    // behind its own named barrier (teams never share a warp's table entry)
    const int lane = threadIdx.x & 31, team = threadIdx.x / GT;
    c = __reduce_add_sync(0xffffffffu, c);
    int *mine = sh.wc[round & 1];
    if (lane == 0) mine[threadIdx.x >> 5] = c;
    if (GT == NT) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "n"(GT) : "memory");
    const int v = lane < GT / 32 ? mine[team * (GT / 32) + lane] : 0;
    return __reduce_add_sync(0xffffffffu, v);
}

// Sets the kept bit of 32 consecutive tokens starting at t0 (any alignment) from a warp ballot.
__device__ __forceinline__ void mask_or_ballot(unsigned *mask, int t0, unsigned bal)
{
    if (bal && (threadIdx.x & 31) == 0) {
        const int w = t0 >> 5, sft = t0 & 31;
        atomicOr(&mask[w], bal << sft);
        if (sft) atomicOr(&mask[w + 1], bal >> (32 - sft));
    }
}

// Top-q of one segment of at most 32 * KPL tokens by one warp, keys in registers: the q-th largest key is
// found bit by bit from the top (one warp-wide count per bit), stopping as soon as exactly q keys lie at or
// above the prefix; of the keys equal to the threshold the first ones in position order are taken.
template <int KPL>
__device__ __forceinline__ void warp_load_keys(const float *g, int a, int e, unsigned (&k)[KPL])
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        const int t = a + j * 32 + lane;
        k[j] = t < e ? score_key(g[t]) : 0u; // a key of 0 is never counted (X >= 1); real zeros are handled as ties of P = 0
    }
}

template <int KPL>
__device__ __forceinline__ void warp_segment(const unsigned (&k)[KPL], unsigned *mask, int a, int e, int q)
{
    const int lane = threadIdx.x & 31;
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
        for (int j = 0; j < KPL; ++j) c += (a + j * 32 + lane < e) && k[j] > P;
        take = q - __reduce_add_sync(0xffffffffu, c);
    }
    int seen = 0;
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        const int t0 = a + j * 32;
        if (t0 >= e) break;
        const bool in = t0 + lane < e;
        bool keepit = in && k[j] > P;
        const bool tie = in && k[j] == P;
        if (exact) keepit |= tie;
        else {
            const unsigned bal = __ballot_sync(0xffffffffu, tie);
            keepit |= tie && seen + __popc(bal & ((1u << lane) - 1u)) < take;
            seen += __popc(bal);
        }
        mask_or_ballot(mask, t0, __ballot_sync(0xffffffffu, keepit));
    }
}

// Top-q of the `n` items of a block-wide set, at most KPT per thread, item j of thread tid being number
// j * NT + tid (numbers ascend with position).  key_of(i) gives the score key, ok(i) whether the item
// takes part; keep(i) is called for every winner.  First the key bits, then (if more than q items lie at or
// above the q-th key) the item numbers of the tied items, smaller first.
template <int NT, int GT, int KPT, typename KeyOf, typename Ok, typename Keep>
__device__ __forceinline__ void block_select_reg(int n, int q, SelShared &sh, int &round, KeyOf key_of, Ok ok, Keep keep)
{
    const int tid = threadIdx.x % GT; // position inside the counting group
    unsigned k[KPT];
    unsigned elig = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const int i = j * GT + tid;
        k[j] = 0u;
        if (i < n && ok(i)) { elig |= 1u << j; k[j] = key_of(i); }
    }
    unsigned P = 0;
    bool exact = false;
    for (int bit = 31; bit >= 0; --bit) {
        const unsigned X = P | (1u << bit);
        int c = 0;
#pragma unroll
        for (int j = 0; j < KPT; ++j) c += k[j] >= X;
        const int tot = block_count<NT, GT>(c, round++, sh);
        if (tot >= q) {
            P = X;
            if (tot == q) { exact = true; break; }
        }
    }
    unsigned win = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j)
        if (((elig >> j) & 1u) && (k[j] > P || (exact && k[j] == P))) win |= 1u << j;
    if (!exact) {
        // ties at the threshold: the first (q - #above) of them by item number.  Search the item-number image
        // n - i (larger = earlier), unique per item, so the count ends exactly.
        const int above = block_count<NT, GT>(__popc(win), round++, sh);
        const int take = q - above;
        unsigned tie = 0;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int i = j * GT + tid;
            const bool is_tie = ((elig >> j) & 1u) && k[j] == P;
            if (is_tie) tie |= 1u << j;
            k[j] = is_tie ? (unsigned)(n - i) : 0u;
        }
        unsigned P2 = 0;
        for (int bit = 31 - __clz(n); bit >= 0; --bit) {
            const unsigned X = P2 | (1u << bit);
            int c = 0;
#pragma unroll
            for (int j = 0; j < KPT; ++j) c += k[j] >= X;
            const int tot = block_count<NT, GT>(c, round++, sh);
            if (tot >= take) {
                P2 = X;
                if (tot == take) break;
            }
        }
#pragma unroll
        for (int j = 0; j < KPT; ++j)
            if (((tie >> j) & 1u) && k[j] >= P2) win |= 1u << j;
    }
#pragma unroll
    for (int j = 0; j < KPT; ++j)
        if ((win >> j) & 1u) keep(j * GT + tid);
}

// The same selection for sets too large for registers: every round walks the items again (scores from L2).
template <int NT, typename KeyOf, typename Ok, typename Keep>
__device__ void block_select_stream(int n, int q, SelShared &sh, int &round, KeyOf key_of, Ok ok, Keep keep)
{
    const int tid = threadIdx.x;
    unsigned P = 0;
    bool exact = false;
    for (int bit = 31; bit >= 0; --bit) {
        const unsigned X = P | (1u << bit);
        int c = 0;
        for (int i = tid; i < n; i += NT) c += ok(i) && key_of(i) >= X;
        const int tot = block_count<NT>(c, round++, sh);
        if (tot >= q) {
            P = X;
            if (tot == q) { exact = true; break; }
        }
    }
    unsigned P2 = 0;
    if (!exact) {
        int c = 0;
        for (int i = tid; i < n; i += NT) c += ok(i) && key_of(i) > P;
        const int take = q - block_count<NT>(c, round++, sh);
        for (int bit = 31 - __clz(n); bit >= 0; --bit) {
            const unsigned X = P2 | (1u << bit);
            int c2 = 0;
            for (int i = tid; i < n; i += NT) c2 += ok(i) && key_of(i) == P && (unsigned)(n - i) >= X;
            const int tot = block_count<NT>(c2, round++, sh);
            if (tot >= take) {
                P2 = X;
                if (tot == take) break;
            }
        }
    }
    for (int i = tid; i < n; i += NT) {
        if (!ok(i)) continue;
        const unsigned key = key_of(i);
        if (key > P || (key == P && (exact || (unsigned)(n - i) >= P2))) keep(i);
    }
}

template <int NT, typename KeyOf, typename Ok, typename Keep>
__device__ __forceinline__ void block_select(int n, int q, SelShared &sh, int &round, KeyOf key_of, Ok ok, Keep keep)
{
    if (n <= NT * 4) block_select_reg<NT, NT, 4>(n, q, sh, round, key_of, ok, keep);
    else if (n <= NT * 8) block_select_reg<NT, NT, 8>(n, q, sh, round, key_of, ok, keep);
    else if (n <= NT * 16) block_select_reg<NT, NT, 16>(n, q, sh, round, key_of, ok, keep);
    else if (NT <= 256 && n <= NT * 32) block_select_reg<NT, NT, NT <= 256 ? 32 : 16>(n, q, sh, round, key_of, ok, keep);
    else block_select_stream<NT>(n, q, sh, round, key_of, ok, keep);
}

template <int NT>
__global__ void __launch_bounds__(NT, 1024 / NT) k_select_compact(DevParams p)
{
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ SelShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, uid = blockIdx.x;
    const UnitId un = unit_of(p, uid);
    const int T = p.seq_lens[un.b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int sc = p.seg_cap;
    const SelSmem mp = sel_smem(p.T_cap, sc);
    unsigned *mask = reinterpret_cast<unsigned *>(dyn + mp.mask);
    int *bounds = reinterpret_cast<int *>(dyn + mp.bounds);
    int *quota = reinterpret_cast<int *>(dyn + mp.quota);
    uint2 *list = reinterpret_cast<uint2 *>(dyn + mp.list);  // (key, position) of backfill candidates
    const size_t row = (size_t)uid * p.T_cap;
    const float *g = p.scores + row;
    int *keep = p.keep_idx + (size_t)uid * p.Tk;
    const bool ema_on = p.beta != 1.0f;
    const int n_words = (T + 31) >> 5;
    int round = 0;
    wait_for_previous_kernel(); // segments and quotas
    const int n_seg = p.n_seg[uid];
    if (n_seg < 0) return; // reported by the previous kernel
    for (int i = tid; i <= n_words; i += NT) mask[i] = 0u;
    for (int i = tid; i < n_seg; i += NT) {
        bounds[i] = p.seg_bounds[(size_t)uid * (sc + 1) + i];
        quota[i] = p.quotas[(size_t)uid * sc + i];
    }
    if (tid == 0) { bounds[n_seg] = T; sh.n_list = 0; }
    __syncthreads();

    // ---- per-segment top-q_i by (score desc, position asc): a warp per segment of at most 1024 tokens.  The keys of
    //      the warp's next segment (the common case of at most 256 tokens) are fetched before the current one is
    //      searched, so that their latency is hidden behind the search.
    bool any_long = false;
    {
        auto searched = [&](int sg) { // a segment that needs a search and fits eight keys per lane
            const int L = bounds[sg + 1] - bounds[sg], q = quota[sg];
            return q > 0 && q < L && L <= 256;
        };
        unsigned kn[8];
        bool have_next = false;
        if (warp < n_seg && searched(warp)) { warp_load_keys<8>(g, bounds[warp], bounds[warp + 1], kn); have_next = true; }
        for (int sg = warp; sg < n_seg; sg += (NT / 32)) {
            const int a = bounds[sg], e = bounds[sg + 1], q = quota[sg], L = e - a;
            unsigned kc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) kc[j] = kn[j];
            const bool have = have_next;
            const int nx = sg + (NT / 32);
            have_next = nx < n_seg && searched(nx);
            if (have_next) warp_load_keys<8>(g, bounds[nx], bounds[nx + 1], kn);
            if (q <= 0) continue;
            if (q >= L) {
                for (int t0 = a; t0 < e; t0 += 32) mask_or_ballot(mask, t0, __ballot_sync(0xffffffffu, t0 + lane < e));
            } else if (have) {
                warp_segment<8>(kc, mask, a, e, q);
            } else if (L <= 512) {
                unsigned k16[16];
                warp_load_keys<16>(g, a, e, k16);
                warp_segment<16>(k16, mask, a, e, q);
            } else if (L <= 1024) {
                unsigned k32[32];
                warp_load_keys<32>(g, a, e, k32);
                warp_segment<32>(k32, mask, a, e, q);
            } else {
                any_long = true;
            }
        }
    }
    // ---- longer segments: teams of four warps take those of up to 4096 tokens in turn, each team behind its own
    //      barrier (a count per key bit costs a team a fraction of a block-wide barrier, and the teams search
    //      different segments at the same time); the whole block then takes what is longer still
    if (__syncthreads_or(any_long)) {
        constexpr int GT = 128, kTeamMax = GT * 32;
        const int team = tid / GT;
        int k = 0;
        for (int sg = 0; sg < n_seg; ++sg) {
            const int a = bounds[sg], e = bounds[sg + 1], q = quota[sg], L = e - a;
            if (L <= 1024 || L > kTeamMax || q <= 0 || q >= L) continue;
            if (k++ % (NT / GT) != team) continue;
            auto key_of = [&](int i) { return score_key(g[a + i]); };
            auto all = [](int) { return true; };
            auto keepit = [&](int i) { atomicOr(&mask[(a + i) >> 5], 1u << ((a + i) & 31)); };
            if (L <= GT * 16) block_select_reg<NT, GT, 16>(L, q, sh, round, key_of, all, keepit);
            else block_select_reg<NT, GT, 32>(L, q, sh, round, key_of, all, keepit);
        }
        __syncthreads();
        round = 0; // the teams counted different numbers of rounds: everybody starts the block-wide counts on the same table
        for (int sg = 0; sg < n_seg; ++sg) {
            const int a = bounds[sg], e = bounds[sg + 1], q = quota[sg], L = e - a;
            if (L <= kTeamMax || q <= 0 || q >= L) continue;
            block_select<NT>(L, q, sh, round,
                             [&](int i) { return score_key(g[a + i]); },
                             [](int) { return true; },
                             [&](int i) { atomicOr(&mask[(a + i) >> 5], 1u << ((a + i) & 31)); });
        }
        __syncthreads();
    }

    // ---- must-keep prefix and suffix; every must-keep position a segment already chose frees one slot,
    //      refilled by the best positions not yet kept (top r_fill of the unflagged tokens of the sequence)
    const int ns = max(0, min(p.n_sink, min(p.Tk, T)));
    const int nl = max(0, min(p.n_last, min(p.Tk - ns, T - ns)));
    int already = 0;
    for (int i = tid; i < ns + nl; i += NT) {
        const int t = i < ns ? i : T - nl + (i - ns);
        already += (atomicOr(&mask[t >> 5], 1u << (t & 31)) >> (t & 31)) & 1u;
    }
    const int r_fill = (int)block_sum_u64((u64)already, sh.scratch);
    if (r_fill > 0) {
        auto key_at = [&](int t) { return score_key(g[t]); };
        auto unflagged = [&](int t) { return ((mask[t >> 5] >> (t & 31)) & 1u) == 0u; };
        auto raise = [&](int t) { atomicOr(&mask[t >> 5], 1u << (t & 31)); };
        if (T <= NT * 8) {
            // (winners are raised only after every thread has read its flags: the search ends with block-wide
            // counts before the first keep)
            block_select<NT>(T, r_fill, sh, round, key_at, unflagged, raise);
        } else {
            // Longer sequence: the r-th largest of the per-thread maxima is a lower bound of the r-th largest
            // key, so only tokens at or above it can win; they go to a short list.  Two walks over the scores
            // (float4 loads, four per thread in flight).
            const int T4 = (T + 3) & ~3;
            auto walk = [&](auto f) {
                for (int base = 0; base < T4; base += NT * 16) {
                    float4 v[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int t = base + (j * NT + tid) * 4;
                        v[j] = t < T4 ? *reinterpret_cast<const float4 *>(g + t) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int t = base + (j * NT + tid) * 4;
                        if (t >= T4) continue;
                        const unsigned taken = mask[t >> 5] >> (t & 31); // (t is a multiple of 4: the four bits share a word)
                        const float x[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (t + i < T && !((taken >> i) & 1u)) f(t + i, score_key(x[i]));
                    }
                }
            };
            unsigned tmax = 0;
            walk([&](int, unsigned key) { tmax = max(tmax, key); });
            // r-th largest of the per-thread maxima, found by one warp (a maximum of 0 counts for nothing: a thread
            // without candidates, or with NaN scores only, which then all qualify below)
            sh.tmax[tid] = tmax;
            __syncthreads();
            if (warp == 0) {
                unsigned tv[NT / 32];
#pragma unroll
                for (int j = 0; j < NT / 32; ++j) tv[j] = sh.tmax[j * 32 + lane];
                unsigned M = 0;
                for (int bit = 31; bit >= 0; --bit) {
                    const unsigned X = M | (1u << bit);
                    int c = 0;
#pragma unroll
                    for (int j = 0; j < NT / 32; ++j) c += tv[j] >= X;
                    if (__reduce_add_sync(0xffffffffu, c) >= r_fill) M = X;
                }
                if (lane == 0) sh.bound = M;
            }
            __syncthreads();
            const unsigned M = sh.bound;
            walk([&](int t, unsigned key) {
                if (key >= M) {
                    const int at = atomicAdd(&sh.n_list, 1);
                    if (at < kListCap) list[at] = make_uint2(key, (unsigned)t);
                }
            });
            __syncthreads();
            const int n_list = sh.n_list;
            if (n_list <= kListCap) {
                // Top r_fill of the list by (key desc, position asc), one warp, entries strided over the lanes.  The
                // list is in arrival order, so ties are ranked by position, not by list index.
                if (warp == 0) {
                    auto count = [&](auto pred) {
                        int c = 0;
                        for (int i = lane; i < n_list; i += 32) c += pred(list[i]);
                        return __reduce_add_sync(0xffffffffu, c);
                    };
                    unsigned P = 0;
                    bool exact = false;
                    for (int bit = 31; bit >= 0; --bit) {
                        const unsigned X = P | (1u << bit);
                        const int tot = count([&](uint2 v) { return v.x >= X; });
                        if (tot >= r_fill) { P = X; if (tot == r_fill) { exact = true; break; } }
                    }
                    unsigned P2 = 0;
                    if (!exact) {
                        const int take = r_fill - count([&](uint2 v) { return v.x > P; });
                        for (int bit = 31 - __clz(T); bit >= 0; --bit) {
                            const unsigned X = P2 | (1u << bit);
                            const int tot = count([&](uint2 v) { return v.x == P && (unsigned)T - v.y >= X; });
                            if (tot >= take) { P2 = X; if (tot == take) break; }
                        }
                    }
                    for (int i = lane; i < n_list; i += 32) {
                        const uint2 v = list[i];
                        if (v.x > P || (v.x == P && (exact || (unsigned)T - v.y >= P2))) raise((int)v.y);
                    }
                }
            } else {
                block_select_stream<NT>(T, r_fill, sh, round, key_at, unflagged, raise);
            }
        }
    }
    __syncthreads();

    // ---- ordered compaction of the kept positions: a thread takes a run of mask words
    const int wpt = (n_words + NT - 1) / NT;
    const int w0 = tid * wpt, w1 = min(n_words, w0 + wpt);
    int n_kept = 0;
    for (int w = w0; w < w1; ++w) n_kept += __popc(mask[w]);
    u64 total;
    int pos = (int)block_excl_scan_u64((u64)n_kept, sh.scratch, &total);
    if ((int)total != p.Tk) {
        if (tid == 0) { set_status(p.status, AMS_ERR_INTERNAL, uid, (int)total, p.Tk); p.seq_bad[un.b] = 1; }
        return;
    }
    for (int w = w0; w < w1; ++w) {
        unsigned m = mask[w];
        while (m) {
            const int bit = __ffs(m) - 1;
            m &= m - 1;
            keep[pos++] = w * 32 + bit;
        }
    }
    // ---- credit rows travel with their tokens; rows beyond the budget start from zero
    if (ema_on) {
        float *credit = p.ema + (((size_t)un.l * p.Bmax + un.b) * p.H + un.h) * (size_t)p.T_cap;
        float *tmp = reinterpret_cast<float *>(p.cbuf + row); // the prefix sums are no longer needed
        __syncthreads();
        for (int j = tid; j < p.Tk; j += NT) tmp[j] = credit[keep[j]];
        __syncthreads();
        for (int j = tid; j < T; j += NT) credit[j] = j < p.Tk ? tmp[j] : 0.0f;
    }
}

} // namespace

bool segsel_supported(const DevParams &p)
{
    return quota_smem(p.seg_cap, p.S).total <= (size_t)200 * 1024 && sel_smem(p.T_cap, p.seg_cap).total <= (size_t)200 * 1024;
}

int launch_segsel(const DevParams &p, LaunchCtx &ctx)
{
    const int units = p.L * p.B * p.H;
    const size_t smem_q = quota_smem(p.seg_cap, p.S).total, smem_s = sel_smem(p.T_cap, p.seg_cap).total;
    // Long segments (no split, or a split length above a warp's reach) are searched by the whole block, one
    // after the other, a barrier per key bit: four smaller blocks per SM hide that latency better; otherwise
    // twice the warps per unit shorten the warp-per-segment phase, unless there are many units per SM.
    const int n_sm = sm_count();
    if (n_sm <= 0) return AMS_ERR_CUDA;
    const bool many_units = units >= 6 * n_sm; // several blocks per SM anyway: the smaller ones overlap their serial parts better
    const bool small_blocks = p.l_max == 0 || p.l_max > 1024 || many_units;
    static SmemGrant grant_q, grant_s256, grant_s512;
    if (!grant_dynamic_smem(k_segments_quotas, smem_q, grant_q)) return AMS_ERR_CUDA;
    if (small_blocks ? !grant_dynamic_smem(k_select_compact<256>, smem_s, grant_s256) : !grant_dynamic_smem(k_select_compact<512>, smem_s, grant_s512))
        return AMS_ERR_CUDA;
    const size_t smem_a = (size_t)(p.S + 1) * 8;
    // A unit's pass is a chain of block-wide reductions: with many units per SM, blocks of 256 threads (four per SM
    // instead of two) overlap those chains better; with few units the wider block finishes its unit sooner.
    const bool narrow_scan = many_units;
    if (ctx.launches <= 1) {
        // nothing but the validation kernel ran before (caller-supplied scores): its effective lengths are read
        // before this kernel's first wait, so this launch is fully ordered after it
        if (narrow_scan) k_mass_scan<256><<<units, 256, smem_a, ctx.s>>>(p);
        else k_mass_scan<512><<<units, 512, smem_a, ctx.s>>>(p);
        if (cudaGetLastError() != cudaSuccess) return AMS_ERR_CUDA;
    } else if ((narrow_scan ? launch_after(k_mass_scan<256>, dim3((unsigned)units), dim3(256), smem_a, ctx.s, p)
                            : launch_after(k_mass_scan<512>, dim3((unsigned)units), dim3(512), smem_a, ctx.s, p)) != cudaSuccess) {
        return AMS_ERR_CUDA;
    }
    ctx.mark(kKernSegmentSelect);
    if (launch_after(k_segments_quotas, dim3((unsigned)units), dim3(32), smem_q, ctx.s, p) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernQuota);
    const cudaError_t e3 = small_blocks ? launch_after(k_select_compact<256>, dim3((unsigned)units), dim3(256), smem_s, ctx.s, p)
                                        : launch_after(k_select_compact<512>, dim3((unsigned)units), dim3(512), smem_s, ctx.s, p);
    if (e3 != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernSelect);
    return AMS_OK;
}

} // namespace ams
