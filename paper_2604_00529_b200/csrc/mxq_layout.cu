// Scale bytes in the tiled order that a block-scaled tensor-core matrix multiply reads (the step that
// follows the conversion path: W_t is consumed by a matmul, Sec. 3.5).  The [rows, kblocks] matrix of
// E8M0 bytes is cut into tiles of 128 rows x 4 block-columns; a tile is 512 consecutive bytes, and
// inside it the byte of row r, column c sits at (r mod 32) * 16 + (r div 32) * 4 + c.  Tiles follow
// one another row-tile by row-tile.  Rows and columns beyond the matrix are filled with byte 0.
//
// mxq_tile_scales re-orders stored scale bytes in a pass of its own; mxq_quantize_tiled and
// mxq_slice_scale_tiled are Q_f and Slice-and-Scale with the scale bytes written in that order by the
// producing kernel itself (put_scale in mxq_kernels.cuh), which saves the pass.
#include <vector>

#include "mxq_kernels.cuh"
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
                bool ok = true;
                MXQ_CHECKED(p, 4, ok = false)
                if (ok) v = *reinterpret_cast<const uint32_t*>(p); // kblocks % 4 == 0: in range and aligned
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (ct * 4 + c < kblocks) v |= ld_u8(p + c) << (8 * c);
            }
        }
        w[g] = v;
    }
    MXQ_CHECKED(out + tile * 512 + (size_t)lane * 16, 16, return)
    *reinterpret_cast<uint4*>(out + tile * 512 + (size_t)lane * 16) = make_uint4(w[0], w[1], w[2], w[3]);
}

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline size_t tiled_bytes(size_t rows, size_t kblocks) { return ((rows + 127) / 128) * ((kblocks + 3) / 4) * 512; }

// Checks shared by the fused entry points.  On MXQ_OK with *n == 0 there is nothing to do.
int check_tiled(size_t rows, size_t cols, int block, size_t* n, uint32_t* kblocks)
{
    *n = 0;
    if (block != 32) return MXQ_ERR_BLOCK;                 // the tiled order is defined for 32-element blocks
    if (cols % 32) return MXQ_ERR_SIZE;
    if (rows == 0 || cols == 0) return MXQ_OK;
    const size_t kb = cols / 32;
    if (kb > ((size_t)1 << 31) || rows > (((size_t)1 << 32) - 1) / kb) return MXQ_ERR_SIZE;   // block index in 32 bits
    *n = rows * cols;
    *kblocks = (uint32_t)kb;
    return MXQ_OK;
}

// Tiles that the matrix covers only in part keep byte 0 where no block lands: clear the buffer first.
int clear_partial_tiles(uint8_t* tiled, size_t rows, size_t kblocks, cudaStream_t s)
{
    if (rows % 128 == 0 && kblocks % 4 == 0) return MXQ_OK;
    if (cudaMemsetAsync(tiled, 0, tiled_bytes(rows, kblocks), s) != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    return MXQ_OK;
}

}  // namespace

}  // namespace mxq

using namespace mxq;

#pragma GCC visibility push(default)
extern "C" {

size_t mxq_tiled_scales_bytes(size_t rows, size_t kblocks) { return tiled_bytes(rows, kblocks); }

int mxq_tile_scales(const uint8_t* scales, size_t rows, size_t kblocks, uint8_t* tiled, mxq_stream stream)
{
    if (rows == 0 || kblocks == 0) return MXQ_OK;
    if (!scales || !tiled) return MXQ_ERR_NULL;
    if (!aligned(scales, 16) || !aligned(tiled, 16)) return MXQ_ERR_ALIGN;
    const size_t col_tiles = (kblocks + 3) / 4, ntiles = ((rows + 127) / 128) * col_tiles;
    const int grid = grid_for_tiles(ntiles, kThreads);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(scales, rows * kblocks);
    MXQ_DEBUG_EXPECT(tiled, tiled_bytes(rows, kblocks));
    if (kblocks % 4 == 0)
        return launch_kernel(tile_scales_kernel<true>, grid, kThreads, s, scales, rows, kblocks, col_tiles, ntiles, tiled);
    return launch_kernel(tile_scales_kernel<false>, grid, kThreads, s, scales, rows, kblocks, col_tiles, ntiles, tiled);
}

int mxq_quantize_tiled(const void* src, int src_dtype, size_t rows, size_t cols, int fmt, int block, void* codes,
                       uint8_t* tiled_scales, mxq_stream stream)
{
    if (fmt_info(fmt).kind != KIND_FP || (src_dtype != MXQ_F32 && src_dtype != MXQ_BF16)) return MXQ_ERR_FORMAT;
    size_t n;
    uint32_t kblocks = 0;
    if (int rc = check_tiled(rows, cols, block, &n, &kblocks)) return rc;
    if (n == 0) return MXQ_OK;
    if (!src || !codes || !tiled_scales) return MXQ_ERR_NULL;
    if (!aligned(src, 32) || !aligned(codes, 32) || !aligned(tiled_scales, 16)) return MXQ_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int rc = clear_partial_tiles(tiled_scales, rows, kblocks, s)) return rc;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(src, n * (src_dtype == MXQ_F32 ? 4u : 2u));
    MXQ_DEBUG_EXPECT(codes, n * (size_t)fmt_info(fmt).bits / 8);
    MXQ_DEBUG_EXPECT(tiled_scales, tiled_bytes(rows, kblocks));
    return launch_quantize_tiled(src, src_dtype, n, fmt, codes, tiled_scales, kblocks, s);
}

int mxq_slice_scale_tiled(const void* codes, const uint8_t* scales, size_t rows, size_t cols, int block, int src_fmt,
                          int dst_fmt, void* out_codes, uint8_t* out_tiled_scales, mxq_stream stream)
{
    if (fmt_info(src_fmt).kind != KIND_FP || fmt_info(dst_fmt).kind != KIND_FP) return MXQ_ERR_FORMAT;
    size_t n;
    uint32_t kblocks = 0;
    if (int rc = check_tiled(rows, cols, block, &n, &kblocks)) return rc;
    if (!ss_pair_ok(src_fmt, dst_fmt)) return MXQ_ERR_PAIR;
    if (n == 0) return MXQ_OK;
    if (!codes || !scales || !out_codes || !out_tiled_scales) return MXQ_ERR_NULL;
    if (!aligned(codes, 32) || !aligned(out_codes, 32) || !aligned(scales, 16) || !aligned(out_tiled_scales, 16))
        return MXQ_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (int rc = clear_partial_tiles(out_tiled_scales, rows, kblocks, s)) return rc;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(codes, n * (size_t)fmt_info(src_fmt).bits / 8);
    MXQ_DEBUG_EXPECT(scales, n / 32);
    MXQ_DEBUG_EXPECT(out_codes, n * (size_t)fmt_info(dst_fmt).bits / 8);
    MXQ_DEBUG_EXPECT(out_tiled_scales, tiled_bytes(rows, kblocks));
    return launch_slice_scale_tiled(codes, scales, n, src_fmt, dst_fmt, out_codes, out_tiled_scales, kblocks, s);
}

int mxq_slice_scale_tiled_batched(const mxq_ss_tiled_item* items, int count, int block, int src_fmt, int dst_fmt,
                                  mxq_stream stream)
{
    if (fmt_info(src_fmt).kind != KIND_FP || fmt_info(dst_fmt).kind != KIND_FP) return MXQ_ERR_FORMAT;
    if (block != 32) return MXQ_ERR_BLOCK;
    if (!ss_pair_ok(src_fmt, dst_fmt)) return MXQ_ERR_PAIR;
    if (count < 0) return MXQ_ERR_SIZE;
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;
    // every item is checked before anything is enqueued
    for (int i = 0; i < count; ++i) {
        const mxq_ss_tiled_item& it = items[i];
        size_t n;
        uint32_t kblocks = 0;
        if (int rc = check_tiled(it.rows, it.cols, block, &n, &kblocks)) return rc;
        if (n == 0) continue;
        if (!it.codes || !it.scales || !it.out_codes || !it.out_tiled_scales) return MXQ_ERR_NULL;
        if (!aligned(it.codes, 32) || !aligned(it.out_codes, 32) || !aligned(it.scales, 16) ||
            !aligned(it.out_tiled_scales, 16))
            return MXQ_ERR_ALIGN;
    }
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        const size_t n = items[i].rows * items[i].cols;
        MXQ_DEBUG_EXPECT(items[i].codes, n * (size_t)fmt_info(src_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].scales, n / 32);
        MXQ_DEBUG_EXPECT(items[i].out_codes, n * (size_t)fmt_info(dst_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].out_tiled_scales, tiled_bytes(items[i].rows, items[i].cols / 32));
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<SsTiledDeviceItem> chunk;
    chunk.reserve(kSsTiledItemsMax);
    size_t tiles = 0;
    auto flush = [&]() -> int {
        if (chunk.empty()) return MXQ_OK;
        const int rc = launch_slice_scale_tiled_batched(chunk.data(), (int)chunk.size(), tiles, src_fmt, dst_fmt, s);
        chunk.clear();
        tiles = 0;
        return rc;
    };
    for (int i = 0; i < count; ++i) {
        const mxq_ss_tiled_item& it = items[i];
        if (it.rows == 0 || it.cols == 0) continue;
        const uint32_t kblocks = (uint32_t)(it.cols / 32);
        if (int rc = clear_partial_tiles(it.out_tiled_scales, it.rows, kblocks, s)) return rc;
        SsTiledDeviceItem d;
        d.codes = static_cast<const uint8_t*>(it.codes);
        d.scales = it.scales;
        d.out_codes = static_cast<uint8_t*>(it.out_codes);
        d.out_scales = make_tiled_scales(it.out_tiled_scales, kblocks);
        d.nunits = it.rows * it.cols / 32;
        d.tile_begin = tiles;
        tiles += ss_batched_tiles(d.nunits);
        chunk.push_back(d);
        if ((int)chunk.size() == kSsTiledItemsMax)
            if (int rc = flush()) return rc;
    }
    return flush();
}

}  // extern "C"
#pragma GCC visibility pop
