// Launcher of the two-target Slice-and-Scale (Eq. 4-5 applied twice to one read of the anchor).
// Fused instantiations exist for the 8-bit anchors and the main lower formats; every other legal
// combination is served by two single-target launches.
#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kU = 2;
constexpr int kThreads = 128;

template <class FH, class FL1, class FL2>
int run(const void* codes, const uint8_t* scales, size_t n, int block, void* oc1, uint8_t* os1, void* oc2, uint8_t* os2,
        cudaStream_t stream)
{
    auto kern = slice_scale2_kernel<FH, FL1, FL2, kU, kThreads>;
    const size_t nunits = n / 32, nscales = n / (size_t)block;
    const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
    return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream, static_cast<const uint8_t*>(codes),
                         scales, nunits, nscales, static_cast<uint8_t*>(oc1), os1, static_cast<uint8_t*>(oc2), os2);
}

}  // namespace

int launch_slice_scale2(const void* codes, const uint8_t* scales, size_t n, int block, int src_fmt, int dst_fmt1,
                        int dst_fmt2, void* oc1, uint8_t* os1, void* oc2, uint8_t* os2, cudaStream_t stream)
{
#define MXQ_TRY2(H, A, B)                                                                                     \
    if (src_fmt == H && dst_fmt1 == A && dst_fmt2 == B)                                                       \
        return run<Fmt<H>, Fmt<A>, Fmt<B>>(codes, scales, n, block, oc1, os1, oc2, os2, stream);              \
    if (src_fmt == H && dst_fmt1 == B && dst_fmt2 == A)                                                       \
        return run<Fmt<H>, Fmt<A>, Fmt<B>>(codes, scales, n, block, oc2, os2, oc1, os1, stream);
    MXQ_TRY2(MXQ_INT8, MXQ_INT6, MXQ_INT4)
    MXQ_TRY2(MXQ_FP8_E4M3, MXQ_FP6_E2M3, MXQ_FP4_E2M1)
    MXQ_TRY2(MXQ_FP8_E4M3, MXQ_FP6_E3M2, MXQ_FP4_E2M1)
    MXQ_TRY2(MXQ_FP8_E4M3, MXQ_FP6_E3M2, MXQ_FP6_E2M3)
#undef MXQ_TRY2
    return MXQ_ERR_PAIR;
}

}  // namespace mxq
