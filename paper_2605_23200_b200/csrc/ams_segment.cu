// Mass, prefix scan, cuts, merge/split, quotas, segmented radix select, must-keep,
// backfill and ordered index compaction: Algorithm 1 steps 1-5 of the paper for one
// score row per thread block, with every per-token array in global scratch.  This
// one-kernel form serves the allocation-free entry point at the end of the file (its
// scratch is a fixed array); ams_compress uses the three kernels of ams_segsel.cu.
//
// Every decision is integer arithmetic on fixed-point images of the mass (kFixBits
// fractional bits) and every floating-point step is a single round-to-nearest
// operation, so the result does not depend on how the block orders its sums.
#include <string.h>

#include "ams_common.cuh"
#include "ams_select.cuh"

namespace ams {

using namespace sel;

__global__ void __launch_bounds__(1024) k_segment_select(DevParams p)
{
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ Smem sm;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int uid = blockIdx.x;
    const int h = uid % p.H, b = (uid / p.H) % p.B, l = uid / (p.H * p.B);
    const int T = p.seq_lens[b];
    if (T <= p.Tk) return; // nothing to evict
    if (T > p.T_cap) { if (tid == 0) set_status(p.status, AMS_ERR_CAPACITY, uid, T, p.T_cap); return; }

    // dynamic shared memory: bounds[seg_cap+1] | quota[seg_cap] | cap[seg_cap] | give[seg_cap] | M[seg_cap]
    //                        | raw[S+1] | merged[S+1] | pieces_off[S+1] | hist[nw*256]
    const int sc = p.seg_cap;
    u64 *Ms = reinterpret_cast<u64 *>(dyn);
    int *bounds = reinterpret_cast<int *>(Ms + sc);
    int *quota = bounds + sc + 1;
    int *cap = quota + sc;
    int *give = cap + sc;
    int *raw = give + sc;
    int *merged = raw + p.S + 1;
    int *poff = merged + p.S + 1;
    int *hist = poff + p.S + 1;

    const float *u = p.usage + (size_t)uid * p.T_cap;
    const float *g = p.scores + (size_t)uid * p.T_cap;
    float *credit = p.ema + (((size_t)l * p.Bmax + b) * p.H + h) * (size_t)p.T_cap;
    u64 *Cb = p.cbuf + (size_t)uid * p.T_cap;
    unsigned char *flags = p.flags + (size_t)uid * p.T_cap;
    int *keep = p.keep_idx + (size_t)uid * p.Tk;
    float *mass_dbg = p.mass_dbg ? p.mass_dbg + (size_t)uid * p.T_cap : nullptr;
    const bool ema_on = p.beta != 1.0f;
    const double two_f = (double)(1ull << kFixBits);

    // ---- Eq. 1 on fixed-point weights
    float wmax = 0.0f;
    for (int t = tid; t < T; t += nt) wmax = fmaxf(wmax, weight_of(u[t], p.eps));
    wmax = block_max_f32(wmax, sm.scratch);
    const double sw = fix_scale(wmax);
    u64 sa = 0;
    for (int t = tid; t < T; t += nt) sa += to_fixed(weight_of(u[t], p.eps), sw);
    const u64 SA = block_sum_u64(sa, sm.scratch);
    const double dSA = (double)SA;
    const double inv_sa = __ddiv_rn(1.0, dSA); // normalisations multiply by the rounded reciprocal of the total

    // ---- EMA credit and the mass used for segmentation
    u64 sh = 0;
    if (ema_on) {
        const float oml = __fsub_rn(1.0f, p.lambda);
        float cmax = 0.0f;
        for (int t = tid; t < T; t += nt) {
            const u64 A = to_fixed(weight_of(u[t], p.eps), sw);
            const float m = __double2float_rn(__dmul_rn((double)A, inv_sa));
            const float cn = __fadd_rn(__fmul_rn(p.lambda, credit[t]), __fmul_rn(oml, m));
            credit[t] = cn;
            if (mass_dbg) mass_dbg[t] = m;
            cmax = fmaxf(cmax, cn);
        }
        cmax = block_max_f32(cmax, sm.scratch);
        u64 scsum = 0;
        double scl = 0.0;
        if (cmax > 0.0f) {
            scl = fix_scale(cmax);
            for (int t = tid; t < T; t += nt) scsum += to_fixed(credit[t], scl);
        }
        const u64 SC = block_sum_u64(scsum, sm.scratch);
        const double dSC = (double)SC, bd = (double)p.beta, omb = __dsub_rn(1.0, (double)p.beta);
        const double inv_sc = SC > 0 ? __ddiv_rn(1.0, dSC) : 0.0;
        for (int t = tid; t < T; t += nt) {
            const u64 A = to_fixed(weight_of(u[t], p.eps), sw);
            const double cur = __dmul_rn(bd, __dmul_rn((double)A, inv_sa));
            double hist_term = 0.0;
            if (SC > 0) hist_term = __dmul_rn(omb, __dmul_rn((double)to_fixed(credit[t], scl), inv_sc));
            const u64 Hm = (u64)__double2ull_rd(__dmul_rn(__dadd_rn(cur, hist_term), two_f));
            Cb[t] = Hm;
            sh += Hm;
        }
    } else {
        for (int t = tid; t < T; t += nt) {
            const u64 A = to_fixed(weight_of(u[t], p.eps), sw);
            const double r = __dmul_rn((double)A, inv_sa);
            if (mass_dbg) mass_dbg[t] = __double2float_rn(r);
            const u64 Hm = (u64)__double2ull_rd(__dmul_rn(r, two_f));
            Cb[t] = Hm;
            sh += Hm;
        }
    }
    const u64 SH = block_sum_u64(sh, sm.scratch);

    // ---- inclusive prefix sum and mass-quantile cuts: the token that reaches quantile k
    //      closes its segment, so the boundary is (position + 1)
    const u64 S = (u64)p.S;
    for (int k = tid; k <= p.S; k += nt) raw[k] = T;
    __syncthreads();
    u64 carry = 0;
    for (int base = 0; base < T; base += nt * 4) {
        const int t0 = base + tid * 4;
        u64 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = (t0 + i < T) ? Cb[t0 + i] : 0ull;
        u64 tot;
        const u64 exc = carry + block_excl_scan_u64(v[0] + v[1] + v[2] + v[3], sm.scratch, &tot);
        carry += tot;
        if (t0 < T) {
            u64 run = exc;
            int kprev = quantile_of(exc, S, SH);
            const int klast = quantile_of(exc + v[0] + v[1] + v[2] + v[3], S, SH);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (t0 + i < T) {
                    run += v[i];
                    Cb[t0 + i] = run;
                    if (klast != kprev) {
                        const int kc = quantile_of(run, S, SH);
                        for (int k = kprev + 1; k <= kc; ++k) raw[k] = t0 + i + 1;
                        kprev = kc;
                    }
                }
            }
        }
    }
    __syncthreads();
    if (p.fixed_seg) { // component ablation: boundary k at floor(k T / S) whatever the mass
        for (int k = tid + 1; k < p.S; k += nt) raw[k] = (int)(((long long)k * T) / p.S);
        __syncthreads();
    }

    // ---- merge short raw segments forward, fold a short tail left, count split pieces
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
    if (n_seg > sc) { if (tid == 0) set_status(p.status, AMS_ERR_CAPACITY, uid, n_seg, sc); return; }
    if (tid == 0) bounds[0] = 0;
    for (int i = 0; i < n_merged; ++i) {
        const int a = merged[i], len = merged[i + 1] - a, pieces = poff[i + 1] - poff[i];
        const int bs = len / pieces, extra = len % pieces;
        for (int j = tid; j < pieces; j += nt) bounds[poff[i] + j + 1] = a + (j + 1) * bs + min(j + 1, extra);
    }
    __syncthreads();

    // ---- must-keep sizes and quotas
    const int ns = max(0, min(p.n_sink, min(p.Tk, T)));
    const int nl = max(0, min(p.n_last, min(p.Tk - ns, T - ns)));
    const int Bq = p.Tk - ns - nl;
    const u64 SHq = p.uniform_q ? (u64)T : SH; // total of what the quotas are proportional to
    long long smin = 0;
    for (int i = tid; i < n_seg; i += nt) {
        const int a = bounds[i], e = bounds[i + 1];
        Ms[i] = p.uniform_q ? (u64)(e - a) : Cb[e - 1] - (a > 0 ? Cb[a - 1] : 0ull); // ablation: share by length
        smin += max(0, min(p.q_min, e - a));
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
    long long Dq = (long long)Bq - sq;
    if (Dq > 0) {
        for (int i = tid; i < n_seg; i += nt) cap[i] = bounds[i + 1] - bounds[i] - quota[i];
        __syncthreads();
        distribute<true>(Dq, cap, give, Ms, n_seg, sm);
        for (int i = tid; i < n_seg; i += nt) quota[i] += give[i];
    } else if (Dq < 0) {
        for (int i = tid; i < n_seg; i += nt)
            cap[i] = quota[i] - max(0, min(p.q_min, bounds[i + 1] - bounds[i]));
        __syncthreads();
        long long left = distribute<false>(-Dq, cap, give, Ms, n_seg, sm);
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
    if (tid == 0) p.n_seg[uid] = n_seg;
    for (int i = tid; i < n_seg; i += nt) {
        p.seg_bounds[(size_t)uid * (sc + 1) + i] = bounds[i];
        p.quotas[(size_t)uid * sc + i] = quota[i];
    }
    if (tid == 0) p.seg_bounds[(size_t)uid * (sc + 1) + n_seg] = T;

    // ---- per-segment top-q_i by (score desc, position asc): one warp per segment
    int *whist = hist + warp * 256;
    int *wbc = hist + nw * 256 + warp * 4;
    for (int s = warp; s < n_seg; s += nw) {
        const int a = bounds[s], e = bounds[s + 1], q = quota[s], L = e - a;
        if (q <= 0 || q >= L) {
            const unsigned char f = q >= L ? 1 : 0;
            for (int t = a + lane; t < e; t += 32) flags[t] = f;
            continue;
        }
        unsigned thr; int take, ties;
        radix_select<false>(g, a, e, q, whist, wbc, [](int) { return true; }, &thr, &take, &ties);
        int seen = 0;
        for (int base = a; base < e; base += 32) {
            const int t = base + lane;
            const unsigned key = t < e ? score_key(g[t]) : 0u;
            bool keepit = t < e && key > thr;
            const bool tie = t < e && key == thr;
            if (take >= ties) keepit |= tie;
            else {
                const unsigned bal = __ballot_sync(0xffffffffu, tie);
                const int rank = seen + __popc(bal & ((1u << lane) - 1u));
                keepit |= tie && rank < take;
                seen += __popc(bal);
            }
            if (t < e) flags[t] = keepit ? 1 : 0;
        }
    }
    __syncthreads();

    // ---- must-keep prefix and suffix; every must-keep position a segment already chose
    //      frees one slot, refilled by the best positions not yet kept
    long long already = 0;
    for (int i = tid; i < ns + nl; i += nt) {
        const int t = i < ns ? i : T - nl + (i - ns);
        already += flags[t];
        flags[t] = 1;
    }
    const int r = (int)block_sum_i64(already, sm.scratch);
    if (r > 0) {
        unsigned thr; int take, ties;
        radix_select<true>(g, 0, T, r, hist, sm.bcast + 4, [flags](int t) { return flags[t] == 0; }, &thr, &take, &ties);
        int seen = 0;
        for (int base = 0; base < T; base += nt) {
            const int t = base + tid;
            const bool cand = t < T && flags[t] == 0;
            const unsigned key = cand ? score_key(g[t]) : 0u;
            bool keepit = cand && key > thr;
            const bool tie = cand && key == thr;
            if (take >= ties) keepit |= tie;
            else {
                if (seen >= take) { if (keepit) flags[t] = 1; continue; }
                u64 tot;
                const int rank = seen + (int)block_excl_scan_u64(tie ? 1ull : 0ull, sm.scratch, &tot);
                keepit |= tie && rank < take;
                seen += (int)tot;
            }
            if (keepit) flags[t] = 1;
        }
    }
    __syncthreads();

    // ---- ordered compaction of the kept positions
    int out = 0;
    for (int base = 0; base < T; base += nt * 16) {
        const int t0 = base + tid * 16;
        uint4 f = make_uint4(0, 0, 0, 0);
        if (t0 < T) f = *reinterpret_cast<const uint4 *>(flags + t0);
        unsigned wds[4] = {f.x, f.y, f.z, f.w};
        int cnt = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const bool on = (t0 + i < T) && ((wds[i >> 2] >> ((i & 3) * 8)) & 0xffu);
            cnt += on;
        }
        u64 tot;
        int pos = out + (int)block_excl_scan_u64((u64)cnt, sm.scratch, &tot);
        out += (int)tot;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const bool on = (t0 + i < T) && ((wds[i >> 2] >> ((i & 3) * 8)) & 0xffu);
            if (on) { if (pos < p.Tk) keep[pos] = t0 + i; ++pos; }
        }
    }
    if (out != p.Tk) { if (tid == 0) set_status(p.status, AMS_ERR_INTERNAL, uid, out, p.Tk); return; }
    __syncthreads();

    // ---- credit rows travel with their tokens; rows beyond the budget start from zero
    if (ema_on) {
        float *tmp = reinterpret_cast<float *>(Cb);
        for (int j = tid; j < p.Tk; j += nt) tmp[j] = credit[keep[j]];
        __syncthreads();
        for (int j = tid; j < T; j += nt) credit[j] = j < p.Tk ? tmp[j] : 0.0f;
    }
}

} // namespace ams

// ---------------------------------------------------------------------------------------
// Allocation-free selection entry point.
//
// Some callers cannot allocate device memory at all: code running while a stream is being
// captured into a CUDA graph (allocation calls are not permitted there), plug-ins loaded into
// a serving process whose memory pool is owned and fully reserved by the host framework, and
// callers on a hot path that must not take the allocator's locks.  For them the scratch the
// selection kernel needs lives in the fixed array below instead of a caller-supplied
// workspace.  Every GPU that loads the library holds the array (kStaticBytes, about 2.4 MB)
// until the process exits.
namespace ams {
namespace {

constexpr int kStaticMaxUnits = 8;       // score rows per call
constexpr int kStaticMaxTokens = 32768;  // tokens per score row
constexpr int kStaticSegCap = 1024;      // segments per row after merge and split
constexpr int kStaticMaxDevices = 64;

struct StaticLayout {
    static constexpr size_t status = 0;                                                   // 4 x int32
    static constexpr size_t lens = 256;                                                   // [units] int32
    static constexpr size_t n_seg = 512;                                                  // [units] int32
    static constexpr size_t bounds = 1024;                                                // [units][cap + 1] int32
    static constexpr size_t quotas = bounds + (size_t)kStaticMaxUnits * (kStaticSegCap + 1) * 4;
    static constexpr size_t flags = (quotas + (size_t)kStaticMaxUnits * kStaticSegCap * 4 + 255) / 256 * 256;
    static constexpr size_t cbuf = flags + (size_t)kStaticMaxUnits * kStaticMaxTokens;    // [units][tokens] u64
    static constexpr size_t total = cbuf + (size_t)kStaticMaxUnits * kStaticMaxTokens * 8;
};
constexpr size_t kStaticBytes = StaticLayout::total;

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

__global__ void k_static_prepare(int *lens, int n_units, int seq_len)
{
    if (threadIdx.x < n_units) lens[threadIdx.x] = seq_len;
}

struct PerDevice {
    bool ready;
    unsigned char *base;
};
PerDevice g_static_dev[kStaticMaxDevices];

} // namespace
} // namespace ams

extern "C" int ams_select_static(const ams_config *cfg, const float *scores, int32_t score_stride, int32_t n_units,
                                 int32_t seq_len, int32_t budget, int32_t n_segments, int32_t *keep_idx, void *stream)
{
    using namespace ams;
    if (!cfg || !scores || !keep_idx) return AMS_ERR_INVALID_ARG;
    if (n_units < 1 || n_units > kStaticMaxUnits) return AMS_ERR_CAPACITY;
    if (seq_len < 1 || seq_len > kStaticMaxTokens) return AMS_ERR_CAPACITY;
    if (score_stride < seq_len || score_stride > kStaticMaxTokens || score_stride % 16) return AMS_ERR_INVALID_ARG;
    if (budget < 1 || budget >= seq_len) return AMS_ERR_INVALID_ARG;
    if (n_segments < 1 || n_segments > 1024) return AMS_ERR_INVALID_ARG;
    if (cfg->l_min < 1 || cfg->l_max < 0 || cfg->q_min < 0 || cfg->n_sink < 0 || cfg->n_last < 0) return AMS_ERR_INVALID_ARG;
    if (!(cfg->eps > 0.0f) || !(cfg->eps < 1e30f)) return AMS_ERR_INVALID_ARG;
    const long long seg_cap = (long long)n_segments + (cfg->l_max > 0 ? 2LL * (seq_len / cfg->l_max) : 0) + 4;
    if (seg_cap > kStaticSegCap) return AMS_ERR_CAPACITY;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return AMS_ERR_CUDA;
    PerDevice &pd = g_static_dev[dev];
    const int nthreads = 1024;
    const size_t dyn = (size_t)kStaticSegCap * 8 + (size_t)(4 * kStaticSegCap + 1) * 4 + (size_t)3 * (1024 + 1) * 4 +
                       (size_t)(nthreads / 32) * (256 + 4) * 4 + 64;
    if (!pd.ready) {
        // once per device, with that device current: the array's address on this device
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return AMS_ERR_CUDA;
        pd.base = (unsigned char *)ptr;
        pd.ready = true;
    }
    // the kernel's dynamic shared-memory limit on this device is only ever raised here
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, k_segment_select) != cudaSuccess) return AMS_ERR_CUDA;
    if ((size_t)fa.maxDynamicSharedSizeBytes < dyn &&
        cudaFuncSetAttribute(k_segment_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return AMS_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    unsigned char *base = pd.base;

    DevParams p;
    memset(&p, 0, sizeof p);
    p.L = 1; p.B = n_units; p.Bmax = n_units; p.H = 1; p.G = 1; p.W = 0; p.rows = 1;
    p.T_cap = score_stride; p.seg_cap = kStaticSegCap; p.Tk = budget; p.S = n_segments; p.n_dst = (budget + kPage - 1) / kPage;
    p.l_min = cfg->l_min; p.l_max = cfg->l_max; p.q_min = cfg->q_min; p.n_sink = cfg->n_sink; p.n_last = cfg->n_last;
    p.lambda = 0.0f; p.beta = 1.0f; p.eps = cfg->eps; // no credit: the mass of the current scores alone
    p.seq_lens = (int *)(base + StaticLayout::lens);
    p.usage = scores;
    p.scores = const_cast<float *>(scores);
    p.cbuf = (u64 *)(base + StaticLayout::cbuf);
    p.flags = base + StaticLayout::flags;
    p.n_seg = (int *)(base + StaticLayout::n_seg);
    p.seg_bounds = (int *)(base + StaticLayout::bounds);
    p.quotas = (int *)(base + StaticLayout::quotas);
    p.keep_idx = keep_idx;
    p.status = (int *)(base + StaticLayout::status);

    k_static_prepare<<<1, 32, 0, s>>>((int *)(base + StaticLayout::lens), n_units, seq_len);
    k_segment_select<<<n_units, nthreads, dyn, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

// Device-side conditions of the calls above (a segment table that overflowed, a count that did not add up)
// land in a status word inside the same fixed array; this reads and clears it, like ams_get_status does
// for a handle.  Copies 16 bytes, allocates nothing, synchronises `stream`.
extern "C" int ams_select_static_status(int32_t *detail, void *stream)
{
    using namespace ams;
    int32_t host[4] = {0, 0, 0, 0};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return AMS_ERR_CUDA;
    const PerDevice &pd = g_static_dev[dev];
    if (pd.ready) {
        cudaStream_t s = (cudaStream_t)stream;
        if (cudaMemcpyAsync(host, pd.base + StaticLayout::status, sizeof host, cudaMemcpyDeviceToHost, s) != cudaSuccess) return AMS_ERR_CUDA;
        if (cudaMemsetAsync(pd.base + StaticLayout::status, 0, sizeof host, s) != cudaSuccess) return AMS_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return AMS_ERR_CUDA;
    }
    if (detail) memcpy(detail, host, sizeof host);
    return host[0];
}
