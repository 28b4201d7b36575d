// Launcher of the fused fake-quant forward (Eq. 6 in reconstructed form) and of the
// straight-through backward copy.
#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kU = 1;
constexpr int kThreads = 128;

template <class T, class F, int BLOCK, int MODE>
int run(const void* src, size_t n, void* dst, cudaStream_t stream)
{
    if constexpr (BLOCK < T::epl) {
        return MXQ_ERR_BLOCK;
    } else {
        auto kern = fake_quant_kernel<T, F, BLOCK, MODE, kU, kThreads>;
        const size_t nunits = n / T::epl;
        const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream,
                             static_cast<const uint8_t*>(src), nunits, static_cast<uint8_t*>(dst));
    }
}

template <class T, class F, int MODE>
int by_block(int block, const void* src, size_t n, void* dst, cudaStream_t stream)
{
    switch (block) {
    case 16: return run<T, F, 16, MODE>(src, n, dst, stream);
    case 32: return run<T, F, 32, MODE>(src, n, dst, stream);
    case 64: return run<T, F, 64, MODE>(src, n, dst, stream);
    case 128: return run<T, F, 128, MODE>(src, n, dst, stream);
    default: return MXQ_ERR_BLOCK;
    }
}

template <class T, class F>
int by_mode(int mode, int block, const void* src, size_t n, void* dst, cudaStream_t stream)
{
    // for the anchors themselves the two modes coincide: one instantiation serves both
    constexpr bool anchor = F::id == MXQ_INT8 || F::id == MXQ_FP8_E4M3;
    if (mode == MXQ_FQ_DIRECT || anchor) return by_block<T, F, MXQ_FQ_DIRECT>(block, src, n, dst, stream);
    if constexpr (!anchor) return by_block<T, F, MXQ_FQ_VIA_ANCHOR>(block, src, n, dst, stream);
    return MXQ_ERR_FORMAT;
}

}  // namespace

int launch_fake_quant(const void* src, int dtype, size_t n, int fmt, int block, int mode, void* dst,
                      cudaStream_t stream)
{
    MXQ_DISPATCH_FORMAT(fmt, {
        if (dtype == MXQ_F32) return by_mode<F32, F>(mode, block, src, n, dst, stream);
        return by_mode<BF16, F>(mode, block, src, n, dst, stream);
    });
    return MXQ_ERR_FORMAT;
}

int launch_copy(const void* src, size_t nbytes, void* dst, cudaStream_t stream)
{
    constexpr int U = 1, kCopyThreads = 256;
    auto kern = copy_kernel<U, kCopyThreads>;
    const size_t ntiles = (nbytes / 32 + 32 * U - 1) / (32 * U);
    return launch_kernel(kern, grid_for_tiles(ntiles, kCopyThreads), kCopyThreads, stream,
                         static_cast<const uint8_t*>(src), nbytes, static_cast<uint8_t*>(dst));
}

}  // namespace mxq
