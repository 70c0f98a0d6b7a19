// Device helpers shared by the segmentation / selection kernels of libams: the Eq. 1
// weight, fixed-point images of the mass, quantile lookup, the closed form of the
// cycling quota adjustment, and the 8-bit radix select.  Not used by the CPU oracle.
#pragma once
#include <float.h>

#include "ams_common.cuh"

namespace ams {
namespace sel {

__device__ __forceinline__ float weight_of(float u, float eps)
{
    // Eq. 1 numerator: max(u, 0) + eps; NaN counts as 0, +inf as FLT_MAX.
    return fminf(__fadd_rn(fmaxf(u, 0.0f), eps), FLT_MAX); // (the sum is never NaN: fmaxf drops a NaN operand)
}

// 2^(kFixBits - (ilogb(mx) + 1)) as a double; mx > 0 (any fp32, subnormals included).
__device__ __forceinline__ double fix_scale(float mx)
{
    const long long bits = __double_as_longlong((double)mx);
    const int e = (int)((bits >> 52) & 0x7ff) - 1023 + 1;
    return __longlong_as_double((long long)(1023 + kFixBits - e) << 52);
}

__device__ __forceinline__ u64 to_fixed(float x, double scale)
{
    return (u64)__double2ull_rd(__dmul_rn((double)x, scale));
}

// min(floor(C * S / SH), S - 1): index of the last mass quantile reached at prefix C.
__device__ __forceinline__ int quantile_of(u64 C, u64 S, u64 SH)
{
    const u64 k = (C * S) / SH;
    return (int)(k < S - 1 ? k : S - 1);
}

struct Smem {
    u64 scratch[40];
    int bcast[8];
};

// Gives `D` (> 0) tokens to segments one per visit, cycling in the visiting order,
// where segment i can take at most cap[i].  Closed form of the cycle: every segment
// receives min(cap, k) with k the largest level whose total fits, and the first
// `rem` segments (in visiting order) that still have room receive one more.
// heavy_first: order (M desc, i asc); otherwise (M asc, i desc).  Returns what is left.
template <bool kHeavyFirst>
__device__ long long distribute(long long D, const int *cap, int *give, const u64 *M, int n_seg, Smem &sm)
{
    const int tid = threadIdx.x, nt = blockDim.x;
    long long cnt1 = 0, tot = 0;
    int mx = 0;
    for (int i = tid; i < n_seg; i += nt) {
        cnt1 += cap[i] >= 1;
        tot += cap[i];
        mx = max(mx, cap[i]);
    }
    cnt1 = block_sum_i64(cnt1, sm.scratch);
    tot = block_sum_i64(tot, sm.scratch);
    mx = (int)block_max_f32((float)mx, sm.scratch); // exact below 2^24; caps are <= 2^17
    long long level = 0, used = 0;
    if (tot <= D) {
        level = mx;
        used = tot;
    } else if (cnt1 <= D) {
        long long lo = 1, hi = mx; // F(lo) <= D < F(hi)
        used = cnt1;
        while (hi - lo > 1) {
            const long long mid = (lo + hi) >> 1;
            long long f = 0;
            for (int i = tid; i < n_seg; i += nt) f += min((long long)cap[i], mid);
            f = block_sum_i64(f, sm.scratch);
            if (f <= D) { lo = mid; used = f; } else hi = mid;
        }
        level = lo;
    }
    const long long rem = D - used;
    for (int i = tid; i < n_seg; i += nt) {
        int g = (int)min((long long)cap[i], level);
        if (rem > 0 && cap[i] > level) {
            long long rank = 0;
            const u64 Mi = M[i];
            for (int j = 0; j < n_seg; ++j) {
                if (cap[j] <= level) continue;
                const u64 Mj = M[j];
                const bool before = kHeavyFirst ? (Mj > Mi || (Mj == Mi && j < i)) : (Mj < Mi || (Mj == Mi && j > i));
                rank += before;
            }
            if (rank < rem) ++g;
        }
        give[i] = g;
    }
    __syncthreads();
    return tot <= D ? D - tot : 0;
}

// k-th largest (k >= 1) of the keys selected by `pred` among positions [a, b), found by
// a 4-pass, 8-bit radix select with a shared histogram.  The calling group is a warp
// (kBlock = false) or the whole block (kBlock = true).  On return *thr is that key,
// *take the number of positions equal to it that belong to the top k, and *ties the
// number of positions equal to it.
template <bool kBlock, typename Pred>
__device__ void radix_select(const float *g, int a, int b, int k, int *hist, int *bc, Pred pred,
                             unsigned *thr, int *take, int *ties)
{
    const int lane = threadIdx.x & 31;
    const int gid = kBlock ? threadIdx.x : lane;
    const int gsz = kBlock ? blockDim.x : 32;
    unsigned prefix = 0, mask = 0;
    int n_ties = 0;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int i = gid; i < 256; i += gsz) hist[i] = 0;
        if (kBlock) __syncthreads(); else __syncwarp();
        for (int t = a + gid; t < b; t += gsz) {
            if (!pred(t)) continue;
            const unsigned key = score_key(g[t]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        if (kBlock) __syncthreads(); else __syncwarp();
        if (!kBlock || threadIdx.x < 32) {
            // lane 0 owns the top eight bins; walk down until k positions are covered
            int c[8], lsum = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = hist[255 - 8 * lane - i]; lsum += c[i]; }
            int inc = lsum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += y;
            }
            const int exc = inc - lsum;
            const bool owner = exc < k && k <= inc;
            const unsigned who = __ballot_sync(0xffffffffu, owner);
            int digit = 0, knew = k, cnt = 0;
            if (owner) {
                int run = exc;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (run < k && k <= run + c[i]) { digit = 255 - 8 * lane - i; knew = k - run; cnt = c[i]; }
                    run += c[i];
                }
            }
            const int src = who ? __ffs(who) - 1 : 0;
            digit = __shfl_sync(0xffffffffu, digit, src);
            knew = __shfl_sync(0xffffffffu, knew, src);
            cnt = __shfl_sync(0xffffffffu, cnt, src);
            if (kBlock) { if (lane == 0) { bc[0] = digit; bc[1] = knew; bc[2] = cnt; } }
            else { bc[0] = digit; bc[1] = knew; bc[2] = cnt; }
            if (!kBlock) { k = knew; prefix |= (unsigned)digit << shift; n_ties = cnt; }
        }
        if (kBlock) {
            __syncthreads();
            k = bc[1];
            prefix |= (unsigned)bc[0] << shift;
            n_ties = bc[2];
            __syncthreads();
        }
        mask |= 0xffu << shift;
    }
    *thr = prefix;
    *take = k;
    *ties = n_ties;
}

// ---- fixed-point images through fp32 / fp64 arithmetic (the three-kernel form) -----------------
// Exponent e = ilogb(mx) + 1 of the largest weight mx > 0 (any fp32, subnormals included).
__device__ __forceinline__ int fix_exponent(float mx)
{
    const long long bits = __double_as_longlong((double)mx);
    return (int)((bits >> 52) & 0x7ff) - 1023 + 1;
}

// The fixed-point image A = floor(x * 2^(kFixBits - e)) (0 <= x < 2^e) equals trunc(x) * 2^(kFixBits - e), where
// trunc(x) is x with the mantissa bits below the image's last bit cleared: x = m * 2^(E - 23), and the image
// drops the lowest n = e - 13 - E bits of m when that is positive (all 24 of them from n = 24 on).  So the
// image is available as a double with one conversion and one exact multiplication by a power of two, and
// sums of images (integers below 2^53) can be added in fp64 in any order.
// The truncation takes two additions: below c = 2^(e - 13) a float is cut to a multiple of the image's
// last bit 2^(e - 36) by adding c rounded down (sums in [c, 2c) have exactly that spacing) and taking c off
// again (exact); from c upwards every float is such a multiple already.  c may be subnormal or zero for
// tiny e: then every float is a multiple of the last bit and both branches return x.
__device__ __forceinline__ float fixed_trunc_by_add(float x, float c)
{
    return x >= c ? x : __fsub_rn(__fadd_rd(x, c), c);
}
__device__ __forceinline__ float fixed_trunc_threshold(int e)
{
    const int k = e - (kFixBits - 23); // 2^k, any k in [-161, 115]
    return k >= -126 ? __uint_as_float((unsigned)(k + 127) << 23) : (k >= -149 ? __uint_as_float(1u << (k + 149)) : 0.0f);
}

// 2^(kFixBits - e) as a double (e = fix_exponent of a positive fp32, so the result is a normal double).
__device__ __forceinline__ double fix_scale_of(int e)
{
    return __longlong_as_double((long long)(1023 + kFixBits - e) << 52);
}

// floor(y) for 0 <= y < 2^51 as an integer: y + 2^52 rounded down lands on the integer grid.
__device__ __forceinline__ u64 floor_to_u64(double y)
{
    return (u64)__double_as_longlong(__dadd_rd(y, 4503599627370496.0)) & 0xfffffffffffffull;
}

} // namespace sel
} // namespace ams
