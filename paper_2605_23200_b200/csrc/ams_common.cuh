// Shared device-side definitions of libams (sm_100a).  Nothing here is used by, or
// shared with, the CPU oracle.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ams.h"

namespace ams {

constexpr int kHeadDim = 128;
constexpr int kPage = 16;
constexpr int kFixBits = 36;          // fractional bits of the fixed-point mass images
constexpr int kRowBytes = kHeadDim * 2;

typedef unsigned long long u64;

// Everything a kernel of one ams_compress call needs; passed by value.
struct DevParams {
    // geometry of the call
    int L, B, Bmax, H, G, W, rows;    // rows = G * W query rows per KV head
    int T_cap, seg_cap, Tk, S, n_dst; // n_dst = ceil(Tk / 16)
    int l_min, l_max, q_min, n_sink, n_last, causal;
    int fixed_seg, uniform_q;         // component ablations: equal-length segments, quotas by segment length
    float lambda, beta, eps;
    // caller buffers
    __nv_bfloat16 *k_pages, *v_pages;
    long long num_pages;
    int *block_table;
    int bt_stride;
    const int *seq_lens;              // effective lengths of this call ([B], workspace): the caller's length where the
                                      // sequence is compressed, 0 where it is skipped (within the budget) or was
                                      // reported (over capacity, window longer than the sequence, bad page id)
    int *seq_lens_out;                // the caller's lengths, rewritten by the table update
    const __nv_bfloat16 *q;           // [L][B][H*G][W][128]
    float *ema;                       // [L][Bmax][H][T_cap]
    const int *dst_pages;             // [B][n_dst]
    // per-unit working arrays, [L*B*H][...]
    const float *usage;               // u: what the mass is built from
    float *scores;                    // g: what segments rank by (== usage unless external)
    u64 *cbuf;                        // [T_cap]  integer mass, then its inclusive prefix sum
    unsigned char *flags;             // [T_cap]  1 = kept
    int *n_seg;                       // [1]
    int *seg_bounds;                  // [seg_cap + 1]
    int *quotas;                      // [seg_cap]
    int *keep_idx;                    // [Tk]
    int *raw_cuts;                    // [S + 1]  cut after the token that reaches mass quantile k (T: none)
    float *mass_dbg;                  // [T_cap] or null
    // scorer scratch
    float *part;                      // per (unit, slice) partials
    float *fin;                       // per unit finals
    int slice_len, n_slices, rows_pad;
    int tc_tpc_min, tc_stages;        // tensor-core scorer: least tiles per block, K stages in shared memory
    int tc_hpb;                       // tensor-core scorer: KV heads a block takes one after the other (set by its launcher)
    int merge_in_usage;               // narrow query blocks: the pass over the stored logits merges the slices' statistics itself
                                      // (set by the launcher when there are too few units for a kernel of its own to pay)
    float *logits;                    // narrow query blocks (rows_pad <= 16): scaled logits [units][T_cap][rows_pad], or null
    // expected-attention scorer
    const float *q_mean;              // [L][B][H*G][128] mean of the future queries per query head
    const __nv_bfloat16 *q_cov;       // [L][B][H*G][128][128] their covariance
    float score_eps;                  // added to the group-mean attention weight before the value norm multiplies
    float *ex_logits;                 // [units][G][T_cap] logits in log2 units, or null
    int ex_g0, ex_gc;                 // query heads [g0, g0 + gc) of the group handled by one launch (set by the launcher)
    int *seq_bad;                     // [B]: set when a unit of the sequence reported a device-side error (its rows stay)
    int *status;                      // [4]: code, unit, a, b
};

__device__ __forceinline__ void set_status(int *status, int code, int unit, int a, int b)
{
    if (atomicCAS(status, 0, code) == 0) {
        status[1] = unit;
        status[2] = a;
        status[3] = b;
    }
}

// Element offset of the 128-wide row (layer, page, slot, head) in a page pool.
__device__ __forceinline__ size_t row_offset(const DevParams &p, int layer, int page, int slot, int h)
{
    return ((((size_t)layer * (size_t)p.num_pages + (size_t)page) * kPage + slot) * p.H + h) * kHeadDim;
}

// ------------------------------------------------------------------ block primitives
// All take a shared scratch array of at least 33 u64 and work for any block size
// that is a multiple of 32 (<= 1024).  Each ends with the result in every thread.

__device__ __forceinline__ u64 warp_sum_u64(u64 v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ u64 block_sum_u64(u64 v, u64 *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    v = warp_sum_u64(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (warp == 0) {
        u64 x = lane < nw ? scratch[lane] : 0ull;
        x = warp_sum_u64(x);
        if (lane == 0) scratch[32] = x;
    }
    __syncthreads();
    return scratch[32];
}

__device__ __forceinline__ long long block_sum_i64(long long v, u64 *scratch)
{
    return (long long)block_sum_u64((u64)v, scratch);
}

__device__ __forceinline__ float block_max_f32(float v, u64 *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if (lane == 0) scratch[warp] = (u64)__float_as_uint(v);
    __syncthreads();
    if (warp == 0) {
        float x = lane < nw ? __uint_as_float((unsigned)scratch[lane]) : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
        if (lane == 0) scratch[32] = (u64)__float_as_uint(x);
    }
    __syncthreads();
    return __uint_as_float((unsigned)scratch[32]);
}

// Exclusive prefix of v over the threads of the block; *total receives the block sum.
__device__ __forceinline__ u64 block_excl_scan_u64(u64 v, u64 *scratch, u64 *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    u64 inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        u64 y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        u64 x = lane < nw ? scratch[lane] : 0ull;
        u64 xi = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            u64 y = __shfl_up_sync(0xffffffffu, xi, o);
            if (lane >= o) xi += y;
        }
        scratch[lane] = xi - x; // exclusive prefix of the warp sums
        if (lane == 31) scratch[32] = xi;
    }
    __syncthreads();
    *total = scratch[32];
    return scratch[warp] + inc - v;
}

// Order-preserving image of an fp32 score; NaN ranks below everything.
__device__ __forceinline__ unsigned score_key(float x)
{
    const unsigned b = __float_as_uint(x);
    if ((b & 0x7fffffffu) > 0x7f800000u) return 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// bf16 pair -> two fp32 (exact).
__device__ __forceinline__ float bf16_lo(unsigned w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(unsigned w) { return __uint_as_float(w & 0xffff0000u); }

// Packed fp32 pairs (two floats in a 64-bit register) and their fused multiply-add.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c)
{
    unsigned long long r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ float sum_f32x2(unsigned long long a)
{
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a));
    return lo + hi;
}

// 16-byte global load that does not pollute L1 (streamed once per phase).
__device__ __forceinline__ uint4 ld_stream16(const void *ptr)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(ptr));
    return v;
}

// 16-byte global store that is not kept in the caches (written once, read by a later kernel or never).
__device__ __forceinline__ void st_stream16(void *ptr, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// A kernel launched with launch_after may start (prologue, loads that depend on nothing the previous kernel of
// the stream writes) while that kernel's last blocks are still running; it calls wait_for_previous_kernel() before
// it first touches anything the previous kernel wrote, or anything that kernel still reads and this one writes.
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Host-side launchers (one per translation unit).
int tova_rows_block(int rows); // query rows handled per pass of the TOVA kernel (8..128)
enum KernelId { kKernScore1 = 0, kKernScoreCombine, kKernScore2, kKernSegmentSelect, kKernGather, kKernTable, kKernUsage, kKernPrepare, kKernQuota, kKernSelect, kKernCount };

// Stream, launch counter and optional per-kernel timing events of one ams_compress call.
struct LaunchCtx {
    cudaStream_t s;
    int launches;
    cudaEvent_t *ev; // null unless profiling; ev[0] is recorded before the first launch
    int n_ev, max_ev;
    int ids[32];
    void begin()
    {
        launches = 0;
        n_ev = 0;
        if (ev) { cudaEventRecord(ev[0], s); n_ev = 1; }
    }
    void mark(int id) // call right after a launch
    {
        ++launches;
        if (ev && n_ev < max_ev) { cudaEventRecord(ev[n_ev], s); ids[n_ev] = id; ++n_ev; }
    }
};

int launch_score_tova(const DevParams &p, LaunchCtx &ctx);
bool tova_tc_supported(const DevParams &p);
size_t tova_tc_smem_bytes(const DevParams &p);
int launch_score_tova_tc(const DevParams &p, LaunchCtx &ctx);
int launch_score_keydiff(const DevParams &p, LaunchCtx &ctx);
bool expected_supported(const DevParams &p);
int launch_score_expected(const DevParams &p, LaunchCtx &ctx);
bool segsel_supported(const DevParams &p);   // shared-memory need of the selection kernels fits (always, within the configuration limits)
int launch_segsel(const DevParams &p, LaunchCtx &ctx); // Algorithm 1 steps 1-5: three kernels
int launch_gather(const DevParams &p, LaunchCtx &ctx);
int launch_smooth_usage(const DevParams &p, const float *src, float *dst, int k, LaunchCtx &ctx);
// First kernel of an event: validates lengths and page ids, writes the effective lengths (lens_in: the caller's).
int launch_prepare(const DevParams &p, const int *lens_in, int *eff_lens, LaunchCtx &ctx);
int launch_expire_wait(int *status, uint32_t polls, cudaStream_t s); // test hook: a bounded wait that runs out

// Launch state that differs per device (one process may drive several GPUs): SM count and, per kernel, the
// dynamic shared-memory limit already granted.
constexpr int kMaxDevices = 64;
inline int current_device()
{
    int d = -1;
    return (cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < kMaxDevices) ? d : -1;
}
inline int sm_count()
{
    static int n_sm[kMaxDevices];
    const int d = current_device();
    if (d < 0) return 0;
    if (!n_sm[d] && cudaDeviceGetAttribute(&n_sm[d], cudaDevAttrMultiProcessorCount, d) != cudaSuccess) n_sm[d] = 0;
    return n_sm[d];
}
struct SmemGrant { size_t bytes[kMaxDevices]; };
template <typename K>
inline bool grant_dynamic_smem(K kernel, size_t smem, SmemGrant &g)
{
    const int d = current_device();
    if (d < 0) return false;
    if (smem > g.bytes[d]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        g.bytes[d] = smem;
    }
    return true;
}
int launch_retained_iou(const DevParams &p, const int *prev_kept, float *out, LaunchCtx &ctx); // before the lengths are rewritten

} // namespace ams
