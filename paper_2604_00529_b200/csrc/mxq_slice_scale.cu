// Launchers of Slice-and-Scale (Eq. 4-5): one tensor per launch, and the batched form that
// converts a whole set of tensors in one launch.
#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kU = 2;
constexpr int kThreads = 128;

// One function template per operation: inside a template the branch that an illegal (source, target)
// pair would take is discarded, so kernels are instantiated for the legal pairs only.
template <class FH, class FL>
int run_single(const void* codes, const uint8_t* scales, size_t n, int block, void* out_codes, uint8_t* out_scales,
               cudaStream_t stream)
{
    if constexpr (ss_pair_ok(FH::id, FL::id)) {
        auto kern = slice_scale_kernel<FH, FL, kU, kThreads>;
        const size_t nunits = n / 32, nscales = n / (size_t)block;
        const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream, static_cast<const uint8_t*>(codes),
                             scales, nunits, nscales, static_cast<uint8_t*>(out_codes), out_scales);
    } else {
        return MXQ_ERR_PAIR;
    }
}

template <class FH, class FL>
int run_single_tiled(const void* codes, const uint8_t* scales, size_t n, void* out_codes, const TiledScales& out_tiled,
                     cudaStream_t stream)
{
    if constexpr (ss_pair_ok(FH::id, FL::id) && FL::kind == KIND_FP) {
        auto kern = slice_scale_kernel<FH, FL, kU, kThreads, TiledScales>;
        const size_t nunits = n / 32;
        const size_t ntiles = (nunits + 32 * kU - 1) / (32 * kU);
        return launch_kernel(kern, grid_for_tiles(ntiles, kThreads), kThreads, stream, static_cast<const uint8_t*>(codes),
                             scales, nunits, nunits, static_cast<uint8_t*>(out_codes), out_tiled);
    } else {
        return MXQ_ERR_PAIR;
    }
}

template <class FH, class FL>
int run_table(const SsDeviceItem* items_dev, const TileIndex* index_dev, int count, size_t total_tiles,
              cudaStream_t stream)
{
    if constexpr (ss_pair_ok(FH::id, FL::id)) {
        auto kern = slice_scale_batched_kernel<FH, FL, kU, kThreads>;
        return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, items_dev, index_dev, count,
                             total_tiles);
    } else {
        return MXQ_ERR_PAIR;
    }
}

template <class FH, class FL>
int run_params(const SsDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    if constexpr (ss_pair_ok(FH::id, FL::id)) {
        auto go = [&](auto k) {
            constexpr int K = decltype(k)::value;
            SsItemBlock<K> blk;
            for (int i = 0; i < count; ++i) blk.items[i] = items_host[i];
            for (int i = count; i < K; ++i) blk.items[i] = SsDeviceItem{};
            build_tile_index(blk.index, items_host, count, total_tiles);
            auto kern = slice_scale_batched_param_kernel<FH, FL, kU, kThreads, K>;
            return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, blk, count, total_tiles);
        };
        if (count <= 64) return go(std::integral_constant<int, 64>{});
        return go(std::integral_constant<int, kSsParamItemsMax>{});
    } else {
        return MXQ_ERR_PAIR;
    }
}

template <class FH, class FL>
int run_tiled_params(const SsTiledDeviceItem* items_host, int count, size_t total_tiles, cudaStream_t stream)
{
    if constexpr (ss_pair_ok(FH::id, FL::id) && FL::kind == KIND_FP) {
        SsTiledItemBlock<kSsTiledItemsMax> blk;
        for (int i = 0; i < count; ++i) blk.items[i] = items_host[i];
        for (int i = count; i < kSsTiledItemsMax; ++i) blk.items[i] = SsTiledDeviceItem{};
        build_tile_index(blk.index, items_host, count, total_tiles);
        auto kern = slice_scale_tiled_batched_kernel<FH, FL, kU, kThreads, kSsTiledItemsMax>;
        return launch_kernel(kern, grid_for_tiles(total_tiles, kThreads), kThreads, stream, blk, count, total_tiles);
    } else {
        return MXQ_ERR_PAIR;
    }
}

}  // namespace

size_t ss_batched_tiles(size_t nunits) { return (nunits + 32 * kU - 1) / (32 * kU); }

int launch_slice_scale(const void* codes, const uint8_t* scales, size_t n, int block, int src_fmt, int dst_fmt,
                       void* out_codes, uint8_t* out_scales, cudaStream_t stream)
{
    MXQ_DISPATCH_FORMAT_AS(src_fmt, FH, {
        MXQ_DISPATCH_FORMAT_AS(dst_fmt, FL, { return run_single<FH, FL>(codes, scales, n, block, out_codes, out_scales, stream); });
    });
    return MXQ_ERR_FORMAT;
}

int launch_slice_scale_tiled(const void* codes, const uint8_t* scales, size_t n, int src_fmt, int dst_fmt,
                             void* out_codes, uint8_t* out_tiled, uint32_t kblocks, cudaStream_t stream)
{
    const TiledScales sink = make_tiled_scales(out_tiled, kblocks);
    MXQ_DISPATCH_FORMAT_AS(src_fmt, FH, {
        MXQ_DISPATCH_FORMAT_AS(dst_fmt, FL, { return run_single_tiled<FH, FL>(codes, scales, n, out_codes, sink, stream); });
    });
    return MXQ_ERR_FORMAT;
}

int launch_slice_scale_tiled_batched(const SsTiledDeviceItem* items_host, int count, size_t total_tiles, int src_fmt,
                                     int dst_fmt, cudaStream_t stream)
{
    if (count > kSsTiledItemsMax) return MXQ_ERR_SIZE;
    MXQ_DISPATCH_FORMAT_AS(src_fmt, FH, {
        MXQ_DISPATCH_FORMAT_AS(dst_fmt, FL, { return run_tiled_params<FH, FL>(items_host, count, total_tiles, stream); });
    });
    return MXQ_ERR_FORMAT;
}

int launch_slice_scale_batched(const SsDeviceItem* items_dev, const TileIndex* index_dev, int count, size_t total_tiles,
                               int src_fmt, int dst_fmt, cudaStream_t stream)
{
    MXQ_DISPATCH_FORMAT_AS(src_fmt, FH, {
        MXQ_DISPATCH_FORMAT_AS(dst_fmt, FL, { return run_table<FH, FL>(items_dev, index_dev, count, total_tiles, stream); });
    });
    return MXQ_ERR_FORMAT;
}

int launch_slice_scale_batched_params(const SsDeviceItem* items_host, int count, size_t total_tiles, int src_fmt,
                                      int dst_fmt, cudaStream_t stream)
{
    if (count > kSsParamItemsMax) return MXQ_ERR_SIZE;
    MXQ_DISPATCH_FORMAT_AS(src_fmt, FH, {
        MXQ_DISPATCH_FORMAT_AS(dst_fmt, FL, { return run_params<FH, FL>(items_host, count, total_tiles, stream); });
    });
    return MXQ_ERR_FORMAT;
}

}  // namespace mxq
