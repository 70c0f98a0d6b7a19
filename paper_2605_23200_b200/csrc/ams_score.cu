// Base scorers of the AMS compression step.
//
// TOVA-style usage (Section 3.2 / Algorithm 1 step 1 of the paper): every query row
// r = (head of the GQA group, window query j) is a softmax of q_r.k_t/sqrt(D) over the
// tokens the row can see; the usage of a token is the mean over rows, where a
// (row, token) pair the row cannot see counts as the largest probability in the
// window.  Two phases over K: phase 1 finds each row's (max, sum of exponentials),
// phase 2 recomputes the logits and sums the normalised probabilities over rows.
// The largest probability of a row is 1/Z_r (its arg-max token), so the window
// maximum is 1/min_r Z_r and needs no third pass.  With at most 16 (padded) query rows
// phase 1 also stores the scaled logits (at most 64 bytes per token against the 256
// bytes of its key), and phase 2 is a per-token kernel over those instead of K.
//
// KeyDiff-style score: negative cosine similarity of each key to the mean key of its
// (sequence, KV head) cache.
#include "ams_common.cuh"

namespace ams {

namespace {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (m, z) <- log-sum-exp merge of (m, z) and (m2, z2) in the base-2 domain.
__device__ __forceinline__ void lse_merge(float &m, float &z, float m2, float z2)
{
    const float mn = fmaxf(m, m2);
    if (mn == -INFINITY) return;
    z = z * ex2(m - mn) + z2 * ex2(m2 - mn);
    m = mn;
}

constexpr int kTovaThreads = 128;
constexpr int kQPitch = 136; // bf16 elements per staged query row: 272 bytes, conflict-free 16-byte reads

// One block = one (unit, token slice).  Each warp walks 16-token tiles; a tile is one
// page.  The tile is the M operand of m16n8k16 and eight query rows are the N
// operand, both read as 16-byte pieces along d: lane (g, tq) loads d = 32 j + 8 tq
// .. +7 of its rows, and those eight values feed k-steps 2j and 2j+1.  The same
// assignment of d to k on both operands leaves the dot product unchanged.
template <int NTB, int PHASE>
__global__ void __launch_bounds__(kTovaThreads) k_tova(DevParams p)
{
    __shared__ __align__(16) __nv_bfloat16 Qs[NTB > 1 ? NTB * 8 * kQPitch : 8];
    __shared__ float red[4][NTB * 8][2];
    if (PHASE == 2) wait_for_previous_kernel(); // merged statistics
    const int uid = blockIdx.y;
    const int h = uid % p.H, b = (uid / p.H) % p.B, l = uid / (p.H * p.B);
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return;
    if (p.W > T) { if (PHASE == 1 && blockIdx.x == 0 && threadIdx.x == 0) set_status(p.status, AMS_ERR_INVALID_ARG, uid, p.W, T); return; }
    const int slice = blockIdx.x;
    const int t_begin = slice * p.slice_len;
    if (t_begin >= T) return;
    const int t_end = min(T, t_begin + p.slice_len);
    const int n_tiles = (t_end - t_begin + 15) >> 4;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, tq = lane & 3;
    const int *table = p.block_table + (size_t)b * p.bt_stride;
    const __nv_bfloat16 *Q = p.q + ((((size_t)l * p.B + b) * p.H + h) * p.G) * (size_t)p.W * kHeadDim;
    const float c = kLog2e * 0.08838834764831845f; // log2(e) / sqrt(128)
    const float *fin = p.fin + (size_t)uid * (p.rows_pad + 8);
    float *u_out = p.scores + (size_t)uid * p.T_cap;
    const int n_rb = p.rows_pad / (NTB * 8);
    float *lg = (PHASE == 1 && p.logits && n_rb == 1) ? p.logits + (size_t)uid * p.T_cap * (NTB * 8) : nullptr;
    const float pmax = PHASE == 2 ? fin[p.rows_pad] : 0.0f;
    const float inv_rows = 1.0f / (float)p.rows;

    for (int rb = 0; rb < n_rb; ++rb) {
        const int row0 = rb * NTB * 8;
        uint4 zq[4];
        if (NTB > 1) {
            __syncthreads();
            for (int i = threadIdx.x; i < NTB * 8 * 16; i += kTovaThreads) {
                const int r = i >> 4, cpos = i & 15;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (row0 + r < p.rows) v = *reinterpret_cast<const uint4 *>(Q + (size_t)(row0 + r) * kHeadDim + cpos * 8);
                *reinterpret_cast<uint4 *>(Qs + r * kQPitch + cpos * 8) = v;
            }
            __syncthreads();
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                zq[j] = make_uint4(0, 0, 0, 0);
                if (row0 + g < p.rows) zq[j] = *reinterpret_cast<const uint4 *>(Q + (size_t)(row0 + g) * kHeadDim + 32 * j + 8 * tq);
            }
        }
        // per thread: rows (nt, e) = row0 + 8 nt + 2 tq + e
        int lastv[NTB][2];
        float st_a[NTB][2], st_b[NTB][2]; // phase 1: (m, z); phase 2: (b_r, unused)
#pragma unroll
        for (int nt = 0; nt < NTB; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int r = row0 + nt * 8 + 2 * tq + e;
                lastv[nt][e] = r < p.rows ? (p.causal ? T - p.W + (r % p.W) : T - 1) : -1;
                if (PHASE == 1) { st_a[nt][e] = -INFINITY; st_b[nt][e] = 0.0f; }
                else { st_a[nt][e] = fin[r]; st_b[nt][e] = 0.0f; }
            }

        for (int tile = warp; tile < n_tiles; tile += 4) {
            const int t0 = t_begin + tile * 16;
            const int page = table[t0 >> 4];
            const __nv_bfloat16 *ra = p.k_pages + row_offset(p, l, page, g, h) + 8 * tq;
            const __nv_bfloat16 *rbp = ra + (size_t)8 * p.H * kHeadDim;
            uint4 x[4], y[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) { x[j] = ld_stream16(ra + 32 * j); y[j] = ld_stream16(rbp + 32 * j); }
            const int ta = t0 + g, tb = t0 + g + 8;
            float acc_a = 0.0f, acc_b = 0.0f;
#pragma unroll
            for (int nt = 0; nt < NTB; ++nt) {
                if (NTB > 1) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        zq[j] = *reinterpret_cast<const uint4 *>(Qs + (nt * 8 + g) * kQPitch + 32 * j + 8 * tq);
                }
                float d[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    mma_bf16(d, x[j].x, y[j].x, x[j].y, y[j].y, zq[j].x, zq[j].y);
                    mma_bf16(d, x[j].z, y[j].z, x[j].w, y[j].w, zq[j].z, zq[j].w);
                }
                float keep_a[2], keep_b[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int lv = min(lastv[nt][e], t_end - 1);
                    const float va = ta <= lv ? d[e] * c : -INFINITY;
                    const float vb = tb <= lv ? d[2 + e] * c : -INFINITY;
                    if (PHASE == 1) {
                        if (NTB <= 2) { keep_a[e] = va; keep_b[e] = vb; }
                        const float mn = fmaxf(st_a[nt][e], fmaxf(va, vb));
                        if (mn != -INFINITY) {
                            st_b[nt][e] = st_b[nt][e] * ex2(st_a[nt][e] - mn) + ex2(va - mn) + ex2(vb - mn);
                            st_a[nt][e] = mn;
                        }
                    } else {
                        acc_a += ex2(va - st_a[nt][e]);
                        acc_b += ex2(vb - st_a[nt][e]);
                    }
                }
                if (PHASE == 1 && NTB <= 2 && lg) { // pairs the window hides are stored as -inf: they add nothing later
                    if (ta < t_end) *reinterpret_cast<float2 *>(lg + (size_t)ta * (NTB * 8) + nt * 8 + 2 * tq) = make_float2(keep_a[0], keep_a[1]);
                    if (tb < t_end) *reinterpret_cast<float2 *>(lg + (size_t)tb * (NTB * 8) + nt * 8 + 2 * tq) = make_float2(keep_b[0], keep_b[1]);
                }
            }
            if (PHASE == 2) {
                acc_a += __shfl_xor_sync(0xffffffffu, acc_a, 1);
                acc_a += __shfl_xor_sync(0xffffffffu, acc_a, 2);
                acc_b += __shfl_xor_sync(0xffffffffu, acc_b, 1);
                acc_b += __shfl_xor_sync(0xffffffffu, acc_b, 2);
                if (tq == 0) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int t = e ? tb : ta;
                        if (t < t_end) {
                            float v = e ? acc_b : acc_a;
                            if (rb > 0) v += u_out[t];
                            if (rb == n_rb - 1) {
                                const int ninv = p.causal ? p.G * max(0, t - (T - p.W)) : 0;
                                v = (v + (float)ninv * pmax) * inv_rows;
                            }
                            u_out[t] = v;
                        }
                    }
                }
            }
        }

        if (PHASE == 1) {
            // rows live in the quad index; fold the eight token groups, then the four warps
#pragma unroll
            for (int nt = 0; nt < NTB; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
#pragma unroll
                    for (int o = 4; o < 32; o <<= 1) {
                        const float m2 = __shfl_xor_sync(0xffffffffu, st_a[nt][e], o);
                        const float z2 = __shfl_xor_sync(0xffffffffu, st_b[nt][e], o);
                        lse_merge(st_a[nt][e], st_b[nt][e], m2, z2);
                    }
                    if (g == 0) {
                        red[warp][nt * 8 + 2 * tq + e][0] = st_a[nt][e];
                        red[warp][nt * 8 + 2 * tq + e][1] = st_b[nt][e];
                    }
                }
            __syncthreads();
            for (int r = threadIdx.x; r < NTB * 8; r += kTovaThreads) {
                float m = red[0][r][0], z = red[0][r][1];
#pragma unroll
                for (int w = 1; w < 4; ++w) lse_merge(m, z, red[w][r][0], red[w][r][1]);
                float2 *out = reinterpret_cast<float2 *>(p.part) + ((size_t)uid * p.n_slices + slice) * p.rows_pad + row0 + r;
                *out = make_float2(m, z);
            }
        }
    }
}

// Per unit: merge the slices' (max, sum) in slice order; b_r = M_r + log2 Z_r in the
// base-2 domain, and the window maximum 1 / min_r Z_r.
__global__ void __launch_bounds__(128) k_tova_combine(DevParams p)
{
    __shared__ u64 scratch[40];
    wait_for_previous_kernel(); // the slices' statistics
    const int uid = blockIdx.x;
    const int b = (uid / p.H) % p.B;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap || p.W > T) return;
    const int ns = (T + p.slice_len - 1) / p.slice_len;
    float *fin = p.fin + (size_t)uid * (p.rows_pad + 8);
    float best = 0.0f;
    for (int r = threadIdx.x; r < p.rows_pad; r += blockDim.x) {
        float m = -INFINITY, z = 0.0f;
        for (int s = 0; s < ns; ++s) {
            const float2 v = reinterpret_cast<const float2 *>(p.part)[((size_t)uid * p.n_slices + s) * p.rows_pad + r];
            lse_merge(m, z, v.x, v.y);
        }
        if (r < p.rows && z > 0.0f) {
            fin[r] = m + log2f(z);
            best = fmaxf(best, 1.0f / z);
        } else {
            fin[r] = INFINITY; // padding rows contribute nothing
        }
    }
    best = block_max_f32(best, scratch);
    if (threadIdx.x == 0) fin[p.rows_pad] = best;
}

// Usage pass over stored logits (RP = padded query rows, 8 or 16): one thread per token sums
// 2^(x_r - b_r) over the rows; pairs the window hides were stored as -inf, padding rows have
// b_r = +inf; the hidden pairs count as the window maximum.
template <int RP>
__global__ void __launch_bounds__(256) k_tova_usage_from_logits(DevParams p)
{
    __shared__ float bs[RP + 1], zinv[RP];
    wait_for_previous_kernel(); // the slices' statistics and the logits
    const int uid = blockIdx.x;
    const int b = (uid / p.H) % p.B;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap || p.W > T) return;
    if (!p.merge_in_usage) {
        const float *fin = p.fin + (size_t)uid * (p.rows_pad + 8);
        if (threadIdx.x <= RP) bs[threadIdx.x] = fin[threadIdx.x]; // b_r of the rows, then the window maximum
        __syncthreads();
    } else {
        // With few units (a launch-bound event) every block merges the slices' (max, sum) of its unit itself (a warp per
        // row, a slice per lane, then a fixed tree over the lanes: the same result in every block): b_r = M_r + log2 Z_r,
        // and the window maximum 1 / min_r Z_r.  With many units a kernel of its own does it once per unit.
        const int ns = (T + p.slice_len - 1) / p.slice_len, lane = threadIdx.x & 31;
        for (int r = threadIdx.x >> 5; r < RP; r += 8) {
            float m = -INFINITY, z = 0.0f;
            for (int sl = lane; sl < ns; sl += 32) {
                const float2 v = __ldcg(reinterpret_cast<const float2 *>(p.part) + ((size_t)uid * p.n_slices + sl) * RP + r);
                lse_merge(m, z, v.x, v.y);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float m2 = __shfl_xor_sync(0xffffffffu, m, o), z2 = __shfl_xor_sync(0xffffffffu, z, o);
                lse_merge(m, z, m2, z2);
            }
            if (lane == 0) {
                const bool live = r < p.rows && z > 0.0f;
                bs[r] = live ? m + log2f(z) : INFINITY; // padding rows contribute nothing
                zinv[r] = live ? 1.0f / z : 0.0f;
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float best = 0.0f;
#pragma unroll
            for (int r = 0; r < RP; ++r) best = fmaxf(best, zinv[r]);
            bs[RP] = best;
        }
        __syncthreads();
    }
    // a block takes several tiles of 256 tokens (up to eight at large capacities), so that the statistics above are
    // fetched once per 2048 tokens and a sequence far below the capacity costs few idle blocks
    const int tiles = ((p.T_cap + 255) / 256 + gridDim.y - 1) / gridDim.y;
    for (int tile = 0; tile < tiles; ++tile) {
        const int t = (blockIdx.y * tiles + tile) * 256 + threadIdx.x;
        if (t >= T) return;
        const float4 *x = reinterpret_cast<const float4 *>(p.logits + ((size_t)uid * p.T_cap + t) * RP);
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int q = 0; q < RP / 4; ++q) {
            const float4 v = __ldcs(x + q);
            acc[0] += ex2(v.x - bs[4 * q]);
            acc[1] += ex2(v.y - bs[4 * q + 1]);
            acc[2] += ex2(v.z - bs[4 * q + 2]);
            acc[3] += ex2(v.w - bs[4 * q + 3]);
        }
        const int ninv = p.causal ? p.G * max(0, t - (T - p.W)) : 0;
        p.scores[(size_t)uid * p.T_cap + t] = ((acc[0] + acc[1]) + (acc[2] + acc[3]) + (float)ninv * bs[RP]) * (1.0f / (float)p.rows);
    }
}

// ---------------------------------------------------------------------------- KeyDiff

constexpr int kKdThreads = 256; // 16 token rows x 16 lanes of 16 bytes

__global__ void __launch_bounds__(kKdThreads) k_keydiff_sum(DevParams p)
{
    __shared__ float red[16][kHeadDim];
    const int uid = blockIdx.y, slice = blockIdx.x;
    const int h = uid % p.H, b = (uid / p.H) % p.B, l = uid / (p.H * p.B);
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int t_begin = slice * p.slice_len;
    if (t_begin >= T) return;
    const int t_end = min(T, t_begin + p.slice_len);
    const int lane = threadIdx.x & 15, r = threadIdx.x >> 4;
    const int *table = p.block_table + (size_t)b * p.bt_stride;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int t = t_begin + r; t < t_end; t += 16) {
        const uint4 v = ld_stream16(p.k_pages + row_offset(p, l, table[t >> 4], t & 15, h) + lane * 8);
        acc[0] += bf16_lo(v.x); acc[1] += bf16_hi(v.x); acc[2] += bf16_lo(v.y); acc[3] += bf16_hi(v.y);
        acc[4] += bf16_lo(v.z); acc[5] += bf16_hi(v.z); acc[6] += bf16_lo(v.w); acc[7] += bf16_hi(v.w);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) red[r][lane * 8 + i] = acc[i];
    __syncthreads();
    if (threadIdx.x < kHeadDim) {
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < 16; ++i) s += red[i][threadIdx.x];
        p.part[((size_t)uid * p.n_slices + slice) * kHeadDim + threadIdx.x] = s;
    }
}

__global__ void __launch_bounds__(kHeadDim) k_keydiff_combine(DevParams p)
{
    __shared__ float sq[kHeadDim];
    wait_for_previous_kernel(); // the slices' sums
    const int uid = blockIdx.x;
    const int b = (uid / p.H) % p.B;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int ns = (T + p.slice_len - 1) / p.slice_len;
    float s = 0.0f;
    for (int i = 0; i < ns; ++i) s += p.part[((size_t)uid * p.n_slices + i) * kHeadDim + threadIdx.x];
    const float mu = s / (float)T;
    float *fin = p.fin + (size_t)uid * (p.rows_pad + 8);
    fin[threadIdx.x] = mu;
    sq[threadIdx.x] = mu * mu;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.0f;
        for (int i = 0; i < kHeadDim; ++i) tot += sq[i];
        fin[kHeadDim] = sqrtf(tot);
    }
}

__global__ void __launch_bounds__(kKdThreads) k_keydiff_score(DevParams p)
{
    wait_for_previous_kernel(); // the mean key
    const int uid = blockIdx.y, slice = blockIdx.x;
    const int h = uid % p.H, b = (uid / p.H) % p.B, l = uid / (p.H * p.B);
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap) return;
    const int t_begin = slice * p.slice_len;
    if (t_begin >= T) return;
    const int t_end = min(T, t_begin + p.slice_len);
    const int lane = threadIdx.x & 15, r = threadIdx.x >> 4;
    const int *table = p.block_table + (size_t)b * p.bt_stride;
    const float *fin = p.fin + (size_t)uid * (p.rows_pad + 8);
    unsigned long long mu2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) mu2[i] = pack_f32x2(fin[lane * 8 + 2 * i], fin[lane * 8 + 2 * i + 1]);
    const float mu_norm = fin[kHeadDim];
    float *g_out = p.scores + (size_t)uid * p.T_cap;
    // four tokens per thread and round: their loads are issued together, so that enough bytes are in flight
    constexpr int kU = 4;
    const int n_iter = (t_end - t_begin + 16 * kU - 1) / (16 * kU);
    for (int it = 0; it < n_iter; ++it) {
        uint4 v[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int t = t_begin + (it * kU + u) * 16 + r;
            v[u] = make_uint4(0, 0, 0, 0);
            if (t < t_end) v[u] = ld_stream16(p.k_pages + row_offset(p, l, table[t >> 4], t & 15, h) + lane * 8);
        }
        // a[2u] = this lane's part of k_t . mu, a[2u + 1] of |k_t|^2, for the four tokens u
        float a[2 * kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            // two dimensions per instruction: a bf16 pair widens to a packed fp32 pair (low half shifted up, high half
            // masked), and both running sums take packed multiply-adds
            const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
            unsigned long long dot2 = 0ull, sq2 = 0ull; // (0.0f, 0.0f)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const unsigned long long k2 = pack_f32x2(bf16_lo(w[i]), bf16_hi(w[i]));
                dot2 = fma_f32x2(k2, mu2[i], dot2);
                sq2 = fma_f32x2(k2, k2, sq2);
            }
            a[2 * u] = sum_f32x2(dot2); a[2 * u + 1] = sum_f32x2(sq2);
        }
        // sums over the 16 lanes of a token row, all eight values at once: at each step a lane hands half of
        // its values to its partner and keeps the other half (9 shuffles instead of 32)
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
        // lane holds value index 4 * bit3 + 2 * bit2 + bit1: even = dot of token (index / 2), odd = its |k|^2
        const float other = __shfl_xor_sync(0xffffffffu, a[0], 2);
        if ((lane & 3) == 0) {
            const int u = lane >> 2;
            const int t = t_begin + (it * kU + u) * 16 + r;
            if (t < t_end) g_out[t] = -a[0] / fmaxf(sqrtf(other) * mu_norm, 1e-30f);
        }
    }
}

template <int NTB>
void launch_tova_ntb(const DevParams &p_in, LaunchCtx &ctx)
{
    DevParams p = p_in;
    const dim3 grid(p.n_slices, p.L * p.B * p.H);
    k_tova<NTB, 1><<<grid, kTovaThreads, 0, ctx.s>>>(p);
    ctx.mark(kKernScore1);
    const bool from_logits = NTB <= 2 && p.logits && p.rows_pad == NTB * 8;
    p.merge_in_usage = from_logits && p.L * p.B * p.H <= 2 * sm_count();
    if (!p.merge_in_usage) {
        launch_after(k_tova_combine, dim3((unsigned)(p.L * p.B * p.H)), dim3(128), 0, ctx.s, p);
        ctx.mark(kKernScoreCombine);
    }
    if (from_logits) {
        const int n256 = (p.T_cap + 255) / 256, per = n256 >= 128 ? 8 : (n256 >= 32 ? n256 / 16 : 1); // tiles per block
        const dim3 g2(p.L * p.B * p.H, (n256 + per - 1) / per);
        launch_after(k_tova_usage_from_logits<NTB * 8>, g2, dim3(256), 0, ctx.s, p);
    } else {
        launch_after(k_tova<NTB, 2>, grid, dim3(kTovaThreads), 0, ctx.s, p);
    }
    ctx.mark(kKernScore2);
}

} // namespace

int tova_rows_block(int rows)
{
    int ntb = 1;
    while (ntb < 16 && ntb * 8 < rows) ntb *= 2;
    return ntb * 8;
}

int launch_score_tova(const DevParams &p, LaunchCtx &ctx)
{
    if (tova_tc_supported(p)) return launch_score_tova_tc(p, ctx);
    switch (tova_rows_block(p.rows) / 8) {
    case 1: launch_tova_ntb<1>(p, ctx); break;
    case 2: launch_tova_ntb<2>(p, ctx); break;
    case 4: launch_tova_ntb<4>(p, ctx); break;
    case 8: launch_tova_ntb<8>(p, ctx); break;
    default: launch_tova_ntb<16>(p, ctx); break;
    }
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

int launch_score_keydiff(const DevParams &p, LaunchCtx &ctx)
{
    const dim3 grid(p.n_slices, p.L * p.B * p.H);
    k_keydiff_sum<<<grid, kKdThreads, 0, ctx.s>>>(p);
    ctx.mark(kKernScore1);
    launch_after(k_keydiff_combine, dim3((unsigned)(p.L * p.B * p.H)), dim3(kHeadDim), 0, ctx.s, p);
    ctx.mark(kKernScoreCombine);
    launch_after(k_keydiff_score, grid, dim3(kKdThreads), 0, ctx.s, p);
    ctx.mark(kKernScore2);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

} // namespace ams
