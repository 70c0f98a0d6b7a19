// Optional smoothing of the usage scores before Eq. 1 (Algorithm 1 step 1): zero-padded
// average pooling of width k (odd) along the sequence, written to a second array so that
// the base scores stay as they are.  The sum of a window runs left to right in fp32 with
// one rounding per addition and ends with one division by k: a fixed order, hence one
// result whatever the launch shape.  k = 1 copies (used when the usage comes from another
// scorer than the base scores).
#include "ams_common.cuh"

namespace ams {

namespace {

constexpr int kSmoothThreads = 256;

__global__ void __launch_bounds__(kSmoothThreads) k_smooth_usage(DevParams p, const float *src, float *dst, int k)
{
    const int uid = blockIdx.x;
    const int b = (uid / p.H) % p.B;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return; // the unit is skipped (or reported) by the kernels that follow
    const int t = blockIdx.y * kSmoothThreads + threadIdx.x;
    if (t >= T) return;
    const float *u = src + (size_t)uid * p.T_cap;
    float out;
    if (k <= 1) {
        out = u[t];
    } else {
        const int r = k >> 1;
        const int lo = max(t - r, 0), hi = min(t + r, T - 1);
        float s = 0.0f;
        for (int j = lo; j <= hi; ++j) s = __fadd_rn(s, u[j]);
        out = __fdiv_rn(s, (float)k);
    }
    dst[(size_t)uid * p.T_cap + t] = out;
}

// Retained-set IoU between the previous event and this one (mechanistic-diagnostics appendix of the
// paper), one thread per unit: the previous retained set occupies positions [0, prev) of the cache, the
// kept positions are ascending, so the intersection is the number of kept positions below prev.
__global__ void __launch_bounds__(128) k_retained_iou(DevParams p, const int *prev_kept, float *out)
{
    const int uid = blockIdx.x * 128 + threadIdx.x;
    if (uid >= p.L * p.B * p.H) return;
    const int b = (uid / p.H) % p.B;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int prev = max(0, min(prev_kept[b], T));
    const int *keep = p.keep_idx + (size_t)uid * p.Tk;
    int lo = 0, hi = p.Tk; // first kept position that is not below prev
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (keep[mid] < prev) lo = mid + 1; else hi = mid;
    }
    const int both = lo, either = prev + p.Tk - both;
    out[uid] = either > 0 ? __fdiv_rn((float)both, (float)either) : 0.0f;
}

} // namespace

int launch_retained_iou(const DevParams &p, const int *prev_kept, float *out, LaunchCtx &ctx)
{
    const int units = p.L * p.B * p.H;
    k_retained_iou<<<(units + 127) / 128, 128, 0, ctx.s>>>(p, prev_kept, out);
    ++ctx.launches;
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

int launch_smooth_usage(const DevParams &p, const float *src, float *dst, int k, LaunchCtx &ctx)
{
    const dim3 grid((unsigned)(p.L * p.B * p.H), (unsigned)((p.T_cap + kSmoothThreads - 1) / kSmoothThreads));
    k_smooth_usage<<<grid, kSmoothThreads, 0, ctx.s>>>(p, src, dst, k);
    ctx.mark(kKernUsage);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

} // namespace ams
