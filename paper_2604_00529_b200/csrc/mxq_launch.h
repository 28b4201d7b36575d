// Internal interface between the C ABI (argument checks, mxq_api.cu) and the per-operation
// translation units that instantiate and launch the kernels.  Arguments are already validated.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/mxq.h"
#include "mxq_debug.cuh"

namespace mxq {

// Grid size that gives every warp tile a warp of its own (`threads` per CTA); 0 when the tensor
// would need more CTAs than a grid can hold (beyond 2^40 elements: reported as MXQ_ERR_SIZE).
inline int grid_for_tiles(size_t ntiles, int threads)
{
    const size_t warps = (size_t)threads / 32;
    const size_t need = (ntiles + warps - 1) / warps;
    if (need > (size_t)0x7FFFFFFF) return 0;
    return (int)(need ? need : 1);
}

int launch_quantize(const void* src, int dtype, size_t n, int fmt, int block, void* codes, uint8_t* scales,
                    cudaStream_t stream);
int launch_fake_quant(const void* src, int dtype, size_t n, int fmt, int block, int mode, void* dst,
                      cudaStream_t stream);
int launch_slice_scale(const void* codes, const uint8_t* scales, size_t n, int block, int src_fmt, int dst_fmt,
                       void* out_codes, uint8_t* out_scales, cudaStream_t stream);
// Anchor -> two lower formats in one pass.  Returns MXQ_ERR_PAIR when this pair of targets has no
// fused instantiation (the caller then falls back to two single-target launches).
int launch_slice_scale2(const void* codes, const uint8_t* scales, size_t n, int block, int src_fmt, int dst_fmt1,
                        int dst_fmt2, void* out_codes1, uint8_t* out_scales1, void* out_codes2, uint8_t* out_scales2,
                        cudaStream_t stream);
// The two-target conversion over up to kSs2BatchItemsMax tensors in one launch (items: a HOST array with
// tile_begin filled in); MXQ_ERR_PAIR when the pair of targets has no fused instantiation.
struct Ss2DeviceItem;
constexpr int kSs2BatchItemsMax = 256;
int launch_slice_scale2_batched(const Ss2DeviceItem* items_host, int count, size_t total_tiles, int src_fmt, int dst_fmt1,
                                int dst_fmt2, cudaStream_t stream);
bool slice_scale2_is_fused(int src_fmt, int dst_fmt1, int dst_fmt2);
size_t ss2_batched_tiles(size_t nunits);
// The same two operations with the scale bytes written in 128 x 4 tiles (block 32, kblocks block-columns
// per row); the caller has zeroed the tiled buffer when the matrix leaves part of a tile uncovered.
int launch_quantize_tiled(const void* src, int dtype, size_t n, int fmt, void* codes, uint8_t* tiled,
                          uint32_t kblocks, cudaStream_t stream);
int launch_slice_scale_tiled(const void* codes, const uint8_t* scales, size_t n, int src_fmt, int dst_fmt,
                             void* out_codes, uint8_t* out_tiled, uint32_t kblocks, cudaStream_t stream);
int launch_dequantize(const void* codes, const uint8_t* scales, size_t n, int fmt, int block, void* dst, int dtype,
                      cudaStream_t stream);
// Fused fake-quant over up to kFqBatchItemsMax tensors in one launch; `items_host` is a HOST array
// whose tile_begin fields are filled in.
struct FqDeviceItem;
constexpr int kFqBatchItemsMax = 512;
int launch_fake_quant_batched(const FqDeviceItem* items_host, int count, size_t total_tiles, int dtype, int fmt,
                              int block, int mode, cudaStream_t stream);
size_t fq_batched_tiles(size_t nunits);
int launch_copy(const void* src, size_t nbytes, void* dst, cudaStream_t stream);
// Q_f and the reconstruction over up to 512 tensors in one launch; `items_host` is a HOST array whose
// tile_begin fields are filled in (tiles counted by q_batched_tiles / dq_batched_tiles of each tensor's
// lane units: n / elements-per-32-bytes of the source for Q_f and for FP32 outputs, n / 32 for BF16 outputs).
struct QDeviceItem;
struct DqDeviceItem;
constexpr int kQBatchItemsMax = 512;
constexpr int kDqBatchItemsMax = 512;
int launch_quantize_batched(const QDeviceItem* items_host, int count, size_t total_tiles, int dtype, int fmt, int block,
                            cudaStream_t stream);
int launch_dequantize_batched(const DqDeviceItem* items_host, int count, size_t total_tiles, int fmt, int block, int dtype,
                              cudaStream_t stream);
size_t q_batched_tiles(size_t nunits);
size_t dq_batched_tiles(size_t nunits);

// Batched Slice-and-Scale over a device-resident item table and its coarse tile index (see
// mxq_kernels.cuh: SsDeviceItem, TileIndex); used by the fixed-table entry point.
struct SsDeviceItem;
struct TileIndex;
int launch_slice_scale_batched(const SsDeviceItem* items_dev, const TileIndex* index_dev, int count, size_t total_tiles,
                               int src_fmt, int dst_fmt, cudaStream_t stream);
// The same launch with the items (a HOST array here) passed in the kernel's parameter space; count
// must not exceed kSsParamItemsMax.
constexpr int kSsParamItemsMax = 512;
int launch_slice_scale_batched_params(const SsDeviceItem* items_host, int count, size_t total_tiles, int src_fmt,
                                      int dst_fmt, cudaStream_t stream);
// The batched launch with tiled scale outputs: up to kSsTiledItemsMax items (a HOST array, tile_begin
// filled in) in the kernel's parameter space.
struct SsTiledDeviceItem;
constexpr int kSsTiledItemsMax = 256;
int launch_slice_scale_tiled_batched(const SsTiledDeviceItem* items_host, int count, size_t total_tiles, int src_fmt,
                                     int dst_fmt, cudaStream_t stream);
// tiles one tensor of `nunits` lane units occupies in the batched kernel's tile space
size_t ss_batched_tiles(size_t nunits);

// Expands the body once per element format with NAME bound to mxq::Fmt<id>.
#define MXQ_DISPATCH_FORMAT_AS(fmt, NAME, ...)                                      \
    switch (fmt) {                                                                  \
    case MXQ_INT8: { using NAME = ::mxq::Fmt<MXQ_INT8>; __VA_ARGS__; } break;           \
    case MXQ_INT7: { using NAME = ::mxq::Fmt<MXQ_INT7>; __VA_ARGS__; } break;           \
    case MXQ_INT6: { using NAME = ::mxq::Fmt<MXQ_INT6>; __VA_ARGS__; } break;           \
    case MXQ_INT5: { using NAME = ::mxq::Fmt<MXQ_INT5>; __VA_ARGS__; } break;           \
    case MXQ_INT4: { using NAME = ::mxq::Fmt<MXQ_INT4>; __VA_ARGS__; } break;           \
    case MXQ_INT3: { using NAME = ::mxq::Fmt<MXQ_INT3>; __VA_ARGS__; } break;           \
    case MXQ_INT2: { using NAME = ::mxq::Fmt<MXQ_INT2>; __VA_ARGS__; } break;           \
    case MXQ_FP8_E4M3: { using NAME = ::mxq::Fmt<MXQ_FP8_E4M3>; __VA_ARGS__; } break;   \
    case MXQ_FP7_E3M3: { using NAME = ::mxq::Fmt<MXQ_FP7_E3M3>; __VA_ARGS__; } break;   \
    case MXQ_FP6_E3M2: { using NAME = ::mxq::Fmt<MXQ_FP6_E3M2>; __VA_ARGS__; } break;   \
    case MXQ_FP6_E2M3: { using NAME = ::mxq::Fmt<MXQ_FP6_E2M3>; __VA_ARGS__; } break;   \
    case MXQ_FP5_E2M2: { using NAME = ::mxq::Fmt<MXQ_FP5_E2M2>; __VA_ARGS__; } break;   \
    case MXQ_FP4_E2M1: { using NAME = ::mxq::Fmt<MXQ_FP4_E2M1>; __VA_ARGS__; } break;   \
    default: return MXQ_ERR_FORMAT;                                                 \
    }
#define MXQ_DISPATCH_FORMAT(fmt, ...) MXQ_DISPATCH_FORMAT_AS(fmt, F, __VA_ARGS__)

// Launches `kern` on `stream` with programmatic stream serialization allowed (see pdl_release /
// pdl_acquire in mxq_access.cuh).  Returns MXQ_OK or MXQ_ERR_CUDA.
template <class... KArgs, class... Args>
inline int launch_kernel(void (*kern)(KArgs...), int grid, int threads, cudaStream_t stream, Args... args)
{
    if (grid <= 0) return MXQ_ERR_SIZE;
#ifdef MXQ_DEBUG
    if (debug_upload(stream) != 0) {                      // the byte ranges this launch may touch
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
#endif
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...) != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    return MXQ_OK;
}

}  // namespace mxq
