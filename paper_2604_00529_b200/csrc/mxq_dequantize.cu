// Launcher of the reconstruction V^ = X P (Sec. 3.3, Notation).
#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kU = 2;
constexpr int kThreads = 128;

template <class F, class T>
int run(const void* codes, const uint8_t* scales, size_t n, int block, void* dst, cudaStream_t stream)
{
    if constexpr (T::size == 4) {
        // FP32 output: lane units of 32 output bytes
        auto kern = dequantize_wide_kernel<F, T, kU, kThreads>;
        const size_t nunits = n / T::epl;
        const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
        int shift = 0;
        while ((T::epl << shift) < block) ++shift;        // units per scale = block / epl (block >= 16 >= epl)
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream,
                             static_cast<const uint8_t*>(codes), scales, nunits, shift, static_cast<uint8_t*>(dst));
    } else {
        // 16-bit output: lane units of 32 codes
        auto kern = dequantize_kernel<F, T, kU, kThreads>;
        const size_t nunits = n / 32;
        const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
        int shift = 0, per_unit = 1;
        if (block == 16) per_unit = 2;
        else while ((32 << shift) < block) ++shift;
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream,
                             static_cast<const uint8_t*>(codes), scales, nunits, shift, per_unit,
                             static_cast<uint8_t*>(dst));
    }
}

// shift / scales-per-unit of the kernel that writes T (see run above)
template <class T>
void scale_geometry(int block, int& shift, int& per_unit)
{
    shift = 0;
    per_unit = 1;
    if constexpr (T::size == 4) {
        while ((T::epl << shift) < block) ++shift;
    } else {
        if (block == 16) per_unit = 2;
        else while ((32 << shift) < block) ++shift;
    }
}

template <class F, class T>
int run_batched(const DqDeviceItem* items_host, int count, size_t total_tiles, int block, cudaStream_t stream)
{
    DqItemBlock<kDqBatchItemsMax> blk;
    for (int i = 0; i < count; ++i) blk.items[i] = items_host[i];
    for (int i = count; i < kDqBatchItemsMax; ++i) blk.items[i] = DqDeviceItem{};
    build_tile_index(blk.index, items_host, count, total_tiles);
    int shift, per_unit;
    scale_geometry<T>(block, shift, per_unit);
    auto kern = dequantize_batched_kernel<F, T, kU, kThreads, kDqBatchItemsMax>;
    return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, blk, count, total_tiles, shift,
                         per_unit);
}

}  // namespace

size_t dq_batched_tiles(size_t nunits) { return (nunits + 32 * kU - 1) / (32 * kU); }

int launch_dequantize_batched(const DqDeviceItem* items_host, int count, size_t total_tiles, int fmt, int block, int dtype,
                              cudaStream_t stream)
{
    if (count > kDqBatchItemsMax) return MXQ_ERR_SIZE;
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return run_batched<F, F32>(items_host, count, total_tiles, block, stream);
        return run_batched<F, BF16>(items_host, count, total_tiles, block, stream);
    });
    return MXQ_ERR_FORMAT;
}

int launch_dequantize(const void* codes, const uint8_t* scales, size_t n, int fmt, int block, void* dst, int dtype,
                      cudaStream_t stream)
{
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return run<F, F32>(codes, scales, n, block, dst, stream);
        return run<F, BF16>(codes, scales, n, block, dst, stream);
    });
    return MXQ_ERR_FORMAT;
}

}  // namespace mxq
