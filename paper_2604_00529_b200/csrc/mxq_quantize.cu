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
