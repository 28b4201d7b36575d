// Launcher of the batched fused fake-quant (Eq. 6 over a whole set of tensors in one launch).
#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kU = 1;
// consecutive warp tiles of one tensor per warp: 2 amortises the tensor lookup (the whole weight set to
// MXINT4 through the anchor 4.29 -> 4.00 ms, to E2M1 4.17 -> 4.02 ms, to E2M3 unchanged); 4 is slower again
constexpr int kR = 2;
constexpr int kThreads = 128;

template <class T, class F, int BLOCK, int MODE>
int run(const FqDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    if constexpr (BLOCK < T::epl) {
        return MXQ_ERR_BLOCK;
    } else {
        FqItemBlock<kFqBatchItemsMax> blk;
        for (int i = 0; i < count; ++i) blk.items[i] = items_host[i];
        for (int i = count; i < kFqBatchItemsMax; ++i) blk.items[i] = FqDeviceItem{};
        build_tile_index(blk.index, items_host, count, total_tiles);
        auto kern = fake_quant_batched_kernel<T, F, BLOCK, MODE, kU, kR, kThreads, kFqBatchItemsMax>;
        return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, blk, count, total_tiles);
    }
}

template <class T, class F, int MODE>
int by_block(int block, const FqDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    switch (block) {
    case 16: return run<T, F, 16, MODE>(items_host, count, total_tiles, stream);
    case 32: return run<T, F, 32, MODE>(items_host, count, total_tiles, stream);
    case 64: return run<T, F, 64, MODE>(items_host, count, total_tiles, stream);
    case 128: return run<T, F, 128, MODE>(items_host, count, total_tiles, stream);
    default: return MXQ_ERR_BLOCK;
    }
}

template <class T, class F>
int by_mode(int mode, int block, const FqDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    constexpr bool anchor = F::id == MXQ_INT8 || F::id == MXQ_FP8_E4M3;
    if (mode == MXQ_FQ_DIRECT || anchor) return by_block<T, F, MXQ_FQ_DIRECT>(block, items_host, count, total_tiles, stream);
    if constexpr (!anchor) return by_block<T, F, MXQ_FQ_VIA_ANCHOR>(block, items_host, count, total_tiles, stream);
    return MXQ_ERR_FORMAT;
}

}  // namespace

size_t fq_batched_tiles(size_t nunits) { return (nunits + 32 * kU * kR - 1) / (32 * kU * kR); }

int launch_fake_quant_batched(const FqDeviceItem* items_host, int count, size_t total_tiles, int dtype, int fmt,
                              int block, int mode, cudaStream_t stream)
{
    if (count > kFqBatchItemsMax) return MXQ_ERR_SIZE;
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return by_mode<F32, F>(mode, block, items_host, count, total_tiles, stream);
        return by_mode<BF16, F>(mode, block, items_host, count, total_tiles, stream);
    });
    return MXQ_ERR_FORMAT;
}

}  // namespace mxq
