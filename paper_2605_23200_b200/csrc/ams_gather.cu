// Paged head-wise compaction: K_new[pi_new(b, j), h, :] <- K_old[pi_old(b, I[b,h,j]), h, :]
// and the same for V (the two display equations of the paper's paged-KV appendix),
// followed by the block-table row and sequence-length rewrite of its runtime routine.
#include "ams_common.cuh"

namespace ams {

namespace {

constexpr int kGatherThreads = 256;          // 16 rows x 16 lanes of 16 bytes
constexpr int kRowsPerIter = kGatherThreads / 16;
constexpr int kUnroll = 4;                   // K and V of 4 rows in flight per thread
constexpr int kRowsPerBlock = kRowsPerIter * kUnroll;

// Rows of one (layer, sequence) are numbered r = j * H + h, so that consecutive rows
// are consecutive 256-byte pieces of the destination page.
__global__ void __launch_bounds__(kGatherThreads) k_gather(DevParams p)
{
    wait_for_previous_kernel(); // kept positions
    const int lb = blockIdx.y;
    const int b = lb % p.B, l = lb / p.B;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap || p.seq_bad[b]) return;
    const int n_rows = p.Tk * p.H;
    const int lane = threadIdx.x & 15, rsub = threadIdx.x >> 4;
    const int r0 = blockIdx.x * kRowsPerBlock + rsub;
    const int *table = p.block_table + (size_t)b * p.bt_stride;
    const int *dst = p.dst_pages + (size_t)b * p.n_dst;
    const int *keep_base = p.keep_idx + (size_t)(l * p.B + b) * p.H * p.Tk;

    uint4 kv[kUnroll], vv[kUnroll];
    size_t doff[kUnroll];
    bool ok[kUnroll];
#pragma unroll
    for (int i = 0; i < kUnroll; ++i) {
        const int r = r0 + i * kRowsPerIter;
        ok[i] = r < n_rows;
        if (ok[i]) {
            const int j = r / p.H, h = r - j * p.H;
            const int pos = keep_base[(size_t)h * p.Tk + j];
            const size_t soff = row_offset(p, l, table[pos >> 4], pos & 15, h) + lane * 8;
            doff[i] = row_offset(p, l, dst[j >> 4], j & 15, h) + lane * 8;
            kv[i] = ld_stream16(p.k_pages + soff);
            vv[i] = ld_stream16(p.v_pages + soff);
        }
    }
#pragma unroll
    for (int i = 0; i < kUnroll; ++i) {
        if (ok[i]) {
            st_stream16(p.k_pages + doff[i], kv[i]);
            st_stream16(p.v_pages + doff[i], vv[i]);
        }
    }
}

// Block-table row <- replacement pages followed by -1; length <- budget.  Runs after
// every kernel that reads the old table.
__global__ void k_table_update(DevParams p)
{
    wait_for_previous_kernel(); // the gather kernel reads the table this kernel rewrites
    const int b = blockIdx.x;
    const int T = p.seq_lens[b];
    if (T <= p.Tk || T > p.T_cap || p.seq_bad[b]) return;
    int *row = p.block_table + (size_t)b * p.bt_stride;
    for (int i = threadIdx.x; i < p.bt_stride; i += blockDim.x)
        row[i] = i < p.n_dst ? p.dst_pages[(size_t)b * p.n_dst + i] : -1;
    __syncthreads();
    if (threadIdx.x == 0) p.seq_lens_out[b] = p.Tk;
}

} // namespace

int launch_gather(const DevParams &p, LaunchCtx &ctx)
{
    const int n_rows = p.Tk * p.H;
    dim3 grid((n_rows + kRowsPerBlock - 1) / kRowsPerBlock, p.L * p.B);
    if (launch_after(k_gather, grid, dim3(kGatherThreads), 0, ctx.s, p) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernGather);
    if (launch_after(k_table_update, dim3((unsigned)p.B), dim3(128), 0, ctx.s, p) != cudaSuccess) return AMS_ERR_CUDA;
    ctx.mark(kKernTable);
    return cudaGetLastError() == cudaSuccess ? AMS_OK : AMS_ERR_CUDA;
}

} // namespace ams
