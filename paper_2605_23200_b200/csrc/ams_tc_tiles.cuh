// Tile bookkeeping shared by the tensor-core scorers of libams (sm_100a): the block shape, the
// partition of all units' 128-token tiles over a persistent grid, and the host-side choice of that grid.
#pragma once
#include <cuda.h>

#include "ams_common.cuh"
#include "ams_tc_ptx.cuh"

namespace ams {
namespace tc {

constexpr int kTcThreads = 640;
constexpr int kConsumerThreads = 512;                // warps 4-19
constexpr int kTileTokens = 128;
constexpr int kTileBytes = kTileTokens * kRowBytes;  // 32 KB
constexpr int kHalfBytes = kTileBytes / 2;           // one 64-wide half of a 128-row tile
constexpr int kSlots = 4;                            // TMEM accumulator slots of 128 columns
constexpr int kMaxStages = 6;

__device__ __forceinline__ int tiles_of(const DevParams &p, int b)
{
    const int T = p.seq_lens[b];
    return (T > p.Tk && T <= p.T_cap && p.W <= T) ? (T + kTileTokens - 1) / kTileTokens : 0;
}

// Prefix of tiles per sequence (shared by all layers and heads) and the partition of one head's
// tiles (all layers) over `grid` groups of blocks.  A group is H blocks, one per KV head, that
// walk the same token tiles at the same time: together they read whole pages (all heads of
// 16 tokens are contiguous), which DRAM serves far better than one head's 256-byte rows alone.
__device__ inline void tc_partition(const DevParams &p, int grid, int *prefix, int *tiles_lh, long long *n_tiles, int *tpc)
{
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int b = 0; b < p.B; ++b) { prefix[b] = acc; acc += tiles_of(p, b); }
        prefix[p.B] = acc;
        *tiles_lh = acc;
        const long long N = (long long)p.L * acc;
        *n_tiles = N;
        const long long per = (N + grid - 1) / grid;
        *tpc = (int)(per > p.tc_tpc_min ? per : p.tc_tpc_min);
    }
    __syncthreads();
}

struct Segment { int uid, l, b, h, tile0, n, T, part; };

// Decodes the segment that starts at global tile g and ends no later than `end`.
__device__ __forceinline__ Segment decode_segment(const DevParams &p, const int *prefix, int tiles_lh, int tpc, long long g, long long end, int h)
{
    Segment s;
    const int l = (int)(g / tiles_lh), rem = (int)(g % tiles_lh);
    int b = 0;
    while (prefix[b + 1] <= rem) ++b;
    s.l = l; s.h = h; s.b = b;
    s.uid = (s.l * p.B + b) * p.H + s.h;
    s.tile0 = rem - prefix[b];
    const int left = prefix[b + 1] - rem;
    s.n = (int)((end - g) < left ? (end - g) : left);
    s.T = p.seq_lens[b];
    const long long ustart = g - s.tile0;
    s.part = (int)(g / tpc) - (int)(ustart / tpc);
    return s;
}

// Host side: how many KV heads one block takes in turn and how many blocks to launch.  The divisor of H that
// fills most SMs wins (the smallest one on a tie); a group of H / hpb blocks walks one range of token tiles.
struct TcGrid { int hpb, grid; };
inline TcGrid tc_grid(const DevParams &p, int n_sm)
{
    const long long cap_tiles = (long long)p.L * p.B * ((p.T_cap + kTileTokens - 1) / kTileTokens); // per head
    const long long want = (cap_tiles + p.tc_tpc_min - 1) / p.tc_tpc_min;
    int hpb = 1;
    for (int d = 1, best = 0; d <= p.H; ++d) {
        if (p.H % d) continue;
        const int blocks = n_sm / (p.H / d) * (p.H / d);
        if (blocks > best) { best = blocks; hpb = d; }
    }
    const int nh = p.H / hpb;
    const int max_groups = n_sm / nh;
    const int groups = (int)(want < max_groups ? (want < 1 ? 1 : want) : max_groups);
    TcGrid g = {hpb, groups * nh};
    return g;
}

// Tensor map over the K pool.  One page of one layer is [16 slots][H heads][2 halves][64]: seen as
// (64, slot % 8, head * 2 + half, slot / 8, layer * num_pages + page), so that a box of (64, 8, 2, 2, 1)
// is one head's 16 rows, stored as [slot / 8][half][slot % 8][64] with the 128-byte swizzle.
inline int make_k_map(const DevParams &p, EncodeTiledFn enc, CUtensorMap *map)
{
    if ((long long)p.L * p.num_pages > 0x7fffffffLL) return AMS_ERR_UNSUPPORTED;
    const cuuint64_t dims[5] = {64, 8, (cuuint64_t)2 * p.H, 2, (cuuint64_t)p.L * (cuuint64_t)p.num_pages};
    const cuuint64_t strides[4] = {(cuuint64_t)p.H * kRowBytes, 128, (cuuint64_t)8 * p.H * kRowBytes,
                                   (cuuint64_t)kPage * p.H * kRowBytes};
    const cuuint32_t box[5] = {64, 8, 2, 2, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, p.k_pages, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS
               ? AMS_OK : AMS_ERR_CUDA;
}

// Tensor map over `rows` contiguous 128-wide bf16 rows; a box is one 64-wide half of 128 rows.
inline int make_rows_map(const void *ptr, unsigned long long rows, EncodeTiledFn enc, CUtensorMap *map)
{
    const cuuint64_t dims[2] = {kHeadDim, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {kRowBytes};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? AMS_OK : AMS_ERR_CUDA;
}

} // namespace tc
} // namespace ams
