// Launcher of the two-target Slice-and-Scale (Eq. 4-5 applied twice to one read of the anchor).
// Fused instantiations exist for the 8-bit anchors and the main lower formats; every other legal
// combination is served by two single-target launches.
#include <utility>

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

template <class FH, class FL1, class FL2>
int run_batched(const Ss2DeviceItem* items_host, int count, size_t total_tiles, bool swap, cudaStream_t stream)
{
    Ss2ItemBlock<kSs2BatchItemsMax> blk;
    for (int i = 0; i < count; ++i) {
        blk.items[i] = items_host[i];
        if (swap) {                                   // the instantiation lists the targets the other way round
            std::swap(blk.items[i].out_codes1, blk.items[i].out_codes2);
            std::swap(blk.items[i].out_scales1, blk.items[i].out_scales2);
        }
    }
    for (int i = count; i < kSs2BatchItemsMax; ++i) blk.items[i] = Ss2DeviceItem{};
    build_tile_index(blk.index, items_host, count, total_tiles);
    auto kern = slice_scale2_batched_kernel<FH, FL1, FL2, kU, kThreads, kSs2BatchItemsMax>;
    return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, blk, count, total_tiles);
}

}  // namespace

size_t ss2_batched_tiles(size_t nunits) { return (nunits + 32 * kU - 1) / (32 * kU); }

int launch_slice_scale2_batched(const Ss2DeviceItem* items_host, int count, size_t total_tiles, int src_fmt, int dst_fmt1,
                                int dst_fmt2, cudaStream_t stream)
{
    if (count > kSs2BatchItemsMax) return MXQ_ERR_SIZE;
#define MXQ_TRY2B(H, A, B)                                                                                    \
    if (src_fmt == H && dst_fmt1 == A && dst_fmt2 == B)                                                       \
        return run_batched<Fmt<H>, Fmt<A>, Fmt<B>>(items_host, count, total_tiles, false, stream);            \
    if (src_fmt == H && dst_fmt1 == B && dst_fmt2 == A)                                                       \
        return run_batched<Fmt<H>, Fmt<A>, Fmt<B>>(items_host, count, total_tiles, true, stream);
    MXQ_TRY2B(MXQ_INT8, MXQ_INT6, MXQ_INT4)
    MXQ_TRY2B(MXQ_FP8_E4M3, MXQ_FP6_E2M3, MXQ_FP4_E2M1)
    MXQ_TRY2B(MXQ_FP8_E4M3, MXQ_FP6_E3M2, MXQ_FP4_E2M1)
    MXQ_TRY2B(MXQ_FP8_E4M3, MXQ_FP6_E3M2, MXQ_FP6_E2M3)
#undef MXQ_TRY2B
    return MXQ_ERR_PAIR;
}

bool slice_scale2_is_fused(int src_fmt, int dst_fmt1, int dst_fmt2)
{
    auto is = [&](int h, int a, int b) { return src_fmt == h && ((dst_fmt1 == a && dst_fmt2 == b) || (dst_fmt1 == b && dst_fmt2 == a)); };
    return is(MXQ_INT8, MXQ_INT6, MXQ_INT4) || is(MXQ_FP8_E4M3, MXQ_FP6_E2M3, MXQ_FP4_E2M1) ||
           is(MXQ_FP8_E4M3, MXQ_FP6_E3M2, MXQ_FP4_E2M1) || is(MXQ_FP8_E4M3, MXQ_FP6_E3M2, MXQ_FP6_E2M3);
}

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
