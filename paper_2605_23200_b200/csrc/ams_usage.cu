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

// First kernel of an event, one block per sequence: the effective length the other kernels work with.
// A sequence within the budget has nothing to evict (effective length 0: every kernel skips it).  A
// sequence over the configured capacity, shorter than the observation window, or whose block-table
// row or replacement pages name a page outside the pool is reported through the status word and
// skipped as well, so that no kernel ever forms an address from a bad page id.
__global__ void __launch_bounds__(256) k_prepare(DevParams p, const int *lens_in, int *eff_lens)
{
    const int b = blockIdx.x;
    const int T = lens_in[b];
    int eff = 0;
    if (T > p.Tk) {
        if (T > p.T_cap) {
            if (threadIdx.x == 0) set_status(p.status, AMS_ERR_CAPACITY, b, T, p.T_cap);
        } else if (p.W > T) {
            if (threadIdx.x == 0) set_status(p.status, AMS_ERR_INVALID_ARG, b, p.W, T);
        } else {
            const int n_src = (T + kPage - 1) / kPage;
            int bad = n_src > p.bt_stride ? 1 : 0;
            const int *row = p.block_table + (size_t)b * p.bt_stride;
            for (int i = threadIdx.x; i < n_src && !bad; i += blockDim.x) {
                const int pg = row[i];
                if (pg < 0 || (long long)pg >= p.num_pages) { bad = 1; set_status(p.status, AMS_ERR_INVALID_ARG, b, i, pg); }
            }
            for (int i = threadIdx.x; i < p.n_dst; i += blockDim.x) {
                const int pg = p.dst_pages[(size_t)b * p.n_dst + i];
                if (pg < 0 || (long long)pg >= p.num_pages) { bad = 1; set_status(p.status, AMS_ERR_INVALID_ARG, b, -1 - i, pg); }
            }
            if (!__syncthreads_or(bad)) eff = T;
        }
    }
    if (threadIdx.x == 0) { eff_lens[b] = eff; p.seq_bad[b] = 0; }
}

// Test hook: one thread waits on an mbarrier that nobody will ever arrive at, gives up after `polls`
// polls and reports AMS_ERR_TIMEOUT through the status word, exactly as the bounded waits of the
// tensor-core scorer do.  Nothing else is touched; the context stays usable.
__global__ void k_expire_wait(int *status, uint32_t polls)
{
    __shared__ unsigned long long bar;
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(&bar);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool done = false;
    for (uint32_t i = 0; i < polls && !done; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(addr), "r"(0) : "memory");
        done = ok != 0;
    }
    if (!done) set_status(status, AMS_ERR_TIMEOUT, -1, (int)polls, 0);
}

} // namespace

int launch_prepare(const DevParams &p, const int *lens_in, int *eff_lens, LaunchCtx &ctx)
{
    k_prepare<<<p.B, 256, 0, ctx.s>>>(p, lens_in, eff_lens);
    ctx.mark(kKernPrepare);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

int launch_expire_wait(int *status, uint32_t polls, cudaStream_t s)
{
    k_expire_wait<<<1, 1, 0, s>>>(status, polls);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

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
