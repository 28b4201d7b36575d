// Scale bytes in the tiled order that a block-scaled tensor-core matrix multiply reads (the step that
// follows the conversion path: W_t is consumed by a matmul, Sec. 3.5).  The [rows, kblocks] matrix of
// E8M0 bytes is cut into tiles of 128 rows x 4 block-columns; a tile is 512 consecutive bytes, and
// inside it the byte of row r, column c sits at (r mod 32) * 16 + (r div 32) * 4 + c.  Tiles follow
// one another row-tile by row-tile.  Rows and columns beyond the matrix are filled with byte 0.
#include "mxq_access.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kThreads = 128;

// One warp per tile: lane t assembles the 16 bytes of rows t, t + 32, t + 64, t + 96 (4 columns each)
// and writes them with one 16-byte store, so a warp's store covers the tile's 512 bytes in order.
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
tile_scales_kernel(const uint8_t* __restrict__ scales, size_t rows, size_t kblocks, size_t col_tiles, size_t ntiles,
                   uint8_t* __restrict__ out)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    pdl_acquire();
    if (tile >= ntiles) return;
    const size_t rt = tile / col_tiles, ct = tile % col_tiles;
    uint32_t w[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const size_t row = rt * 128 + (size_t)g * 32 + lane;
        uint32_t v = 0;
        if (row < rows) {
            const uint8_t* p = scales + row * kblocks + ct * 4;
            if constexpr (VEC) {
                v = *reinterpret_cast<const uint32_t*>(p);         // kblocks % 4 == 0: in range and aligned
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (ct * 4 + c < kblocks) v |= (uint32_t)p[c] << (8 * c);
            }
        }
        w[g] = v;
    }
    *reinterpret_cast<uint4*>(out + tile * 512 + (size_t)lane * 16) = make_uint4(w[0], w[1], w[2], w[3]);
}

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace
}  // namespace mxq

using namespace mxq;

#pragma GCC visibility push(default)
extern "C" {

size_t mxq_tiled_scales_bytes(size_t rows, size_t kblocks)
{
    return ((rows + 127) / 128) * ((kblocks + 3) / 4) * 512;
}

int mxq_tile_scales(const uint8_t* scales, size_t rows, size_t kblocks, uint8_t* tiled, mxq_stream stream)
{
    if (rows == 0 || kblocks == 0) return MXQ_OK;
    if (!scales || !tiled) return MXQ_ERR_NULL;
    if (!aligned(scales, 16) || !aligned(tiled, 16)) return MXQ_ERR_ALIGN;
    const size_t col_tiles = (kblocks + 3) / 4, ntiles = ((rows + 127) / 128) * col_tiles;
    const int grid = grid_for_tiles(ntiles, kThreads);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (kblocks % 4 == 0)
        return launch_kernel(tile_scales_kernel<true>, grid, kThreads, s, scales, rows, kblocks, col_tiles, ntiles, tiled);
    return launch_kernel(tile_scales_kernel<false>, grid, kThreads, s, scales, rows, kblocks, col_tiles, ntiles, tiled);
}

}  // extern "C"
#pragma GCC visibility pop
