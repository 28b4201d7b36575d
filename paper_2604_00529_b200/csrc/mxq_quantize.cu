// Launcher of Q_f (Eq. 1-3): instantiates quantize_kernel per source type, element format and
// block size.
#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kU = 2;   // lane units in flight per thread
constexpr int kThreads = 128;

template <class T, class F, int BLOCK>
int run(const void* src, size_t n, void* codes, uint8_t* scales, cudaStream_t stream)
{
    if constexpr (BLOCK < T::epl) {
        return MXQ_ERR_BLOCK;
    } else {
        constexpr int U = kU;
        auto kern = quantize_kernel<T, F, BLOCK, U, kThreads>;
        const size_t nunits = n / T::epl;
        const size_t ntiles = (nunits + 32 * U - 1) / (32 * U);
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream,
                             static_cast<const uint8_t*>(src), nunits, static_cast<uint8_t*>(codes), scales);
    }
}

template <class T, class F>
int by_block(int block, const void* src, size_t n, void* codes, uint8_t* scales, cudaStream_t stream)
{
    switch (block) {
    case 16: return run<T, F, 16>(src, n, codes, scales, stream);
    case 32: return run<T, F, 32>(src, n, codes, scales, stream);
    case 64: return run<T, F, 64>(src, n, codes, scales, stream);
    case 128: return run<T, F, 128>(src, n, codes, scales, stream);
    default: return MXQ_ERR_BLOCK;
    }
}

template <class T, class F, int BLOCK>
int run_batched(const QDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    if constexpr (BLOCK < T::epl) {
        return MXQ_ERR_BLOCK;
    } else {
        QItemBlock<kQBatchItemsMax> blk;
        for (int i = 0; i < count; ++i) blk.items[i] = items_host[i];
        for (int i = count; i < kQBatchItemsMax; ++i) blk.items[i] = QDeviceItem{};
        build_tile_index(blk.index, items_host, count, total_tiles);
        auto kern = quantize_batched_kernel<T, F, BLOCK, kU, kThreads, kQBatchItemsMax>;
        return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, blk, count, total_tiles);
    }
}

template <class T, class F>
int batched_by_block(int block, const QDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    switch (block) {
    case 16: return run_batched<T, F, 16>(items_host, count, total_tiles, stream);
    case 32: return run_batched<T, F, 32>(items_host, count, total_tiles, stream);
    case 64: return run_batched<T, F, 64>(items_host, count, total_tiles, stream);
    case 128: return run_batched<T, F, 128>(items_host, count, total_tiles, stream);
    default: return MXQ_ERR_BLOCK;
    }
}

template <class T, class F>
int run_tiled(const void* src, size_t n, void* codes, const TiledScales& tiled, cudaStream_t stream)
{
    if constexpr (F::kind == KIND_FP) {
        auto kern = quantize_kernel<T, F, 32, kU, kThreads, TiledScales>;
        const size_t nunits = n / T::epl;
        const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream,
                             static_cast<const uint8_t*>(src), nunits, static_cast<uint8_t*>(codes), tiled);
    } else {
        return MXQ_ERR_FORMAT;
    }
}

}  // namespace

int launch_quantize_tiled(const void* src, int dtype, size_t n, int fmt, void* codes, uint8_t* tiled,
                          uint32_t kblocks, cudaStream_t stream)
{
    const TiledScales sink = make_tiled_scales(tiled, kblocks);
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return run_tiled<F32, F>(src, n, codes, sink, stream);
        return run_tiled<BF16, F>(src, n, codes, sink, stream);
    });
    return MXQ_ERR_FORMAT;
}

size_t q_batched_tiles(size_t nunits) { return (nunits + 32 * kU - 1) / (32 * kU); }

int launch_quantize_batched(const QDeviceItem* items_host, int count, size_t total_tiles, int dtype, int fmt, int block,
                            cudaStream_t stream)
{
    if (count > kQBatchItemsMax) return MXQ_ERR_SIZE;
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return batched_by_block<F32, F>(block, items_host, count, total_tiles, stream);
        return batched_by_block<BF16, F>(block, items_host, count, total_tiles, stream);
    });
    return MXQ_ERR_FORMAT;
}

int launch_quantize(const void* src, int dtype, size_t n, int fmt, int block, void* codes, uint8_t* scales,
                    cudaStream_t stream)
{
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return by_block<F32, F>(block, src, n, codes, scales, stream);
        return by_block<BF16, F>(block, src, n, codes, scales, stream);
    });
    return MXQ_ERR_FORMAT;
}

}  // namespace mxq
