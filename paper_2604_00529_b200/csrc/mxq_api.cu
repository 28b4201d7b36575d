// The C ABI of libmxq (declared in include/mxq.h): argument validation on the host, then the
// per-operation launchers.  Nothing here synchronises the device.
#include <vector>

#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {

namespace {

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline bool valid_format(int f) { return fmt_info(f).kind >= 0; }
inline bool valid_dtype(int t) { return t == MXQ_F32 || t == MXQ_BF16; }
inline bool valid_block(int b) { return b == 16 || b == 32 || b == 64 || b == 128; }

// Checks shared by the tensor entry points; returns MXQ_OK or the first violation.
int check_sizes(size_t n, int block)
{
    if (!valid_block(block)) return MXQ_ERR_BLOCK;
    if (n % (size_t)block) return MXQ_ERR_SIZE;
    return MXQ_OK;
}

}  // namespace

}  // namespace mxq

using namespace mxq;

#pragma GCC visibility push(default)
extern "C" {

const char* mxq_status_string(int status)
{
    switch (status) {
    case MXQ_OK: return "MXQ_OK";
    case MXQ_ERR_NULL: return "MXQ_ERR_NULL: a required pointer is null";
    case MXQ_ERR_FORMAT: return "MXQ_ERR_FORMAT: unknown format, dtype or mode";
    case MXQ_ERR_BLOCK: return "MXQ_ERR_BLOCK: unsupported block size";
    case MXQ_ERR_SIZE: return "MXQ_ERR_SIZE: element count is not a multiple of the block size, or a count is out of range";
    case MXQ_ERR_ALIGN: return "MXQ_ERR_ALIGN: a pointer is not aligned (32 bytes for tensors and codes, 16 for scales)";
    case MXQ_ERR_PAIR: return "MXQ_ERR_PAIR: not a same-family high-to-low format pair";
    case MXQ_ERR_CUDA: return "MXQ_ERR_CUDA: a CUDA call or kernel launch failed";
    case MXQ_ERR_TIMEOUT: return "MXQ_ERR_TIMEOUT: a bounded device-side wait gave up";
    default: return "unknown mxq status";
    }
}

int mxq_debug_report(mxq_debug_info* out, int reset)
{
    if (!out) return MXQ_ERR_NULL;
    *out = mxq_debug_info{};
#ifdef MXQ_DEBUG
    out->enabled = 1;
    if (cudaDeviceSynchronize() != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    out->checked_launches = debug_checked_launches().load();
    for (const DebugUnit& u : debug_units()) {
        unsigned int v = 0, bytes = 0;
        unsigned long long first = 0;
        if (u.read(&v, &first, &bytes) != 0) return MXQ_ERR_CUDA;
        if (v && !out->violations) {
            out->first_address = first;
            out->first_bytes = bytes;
        }
        out->violations += v;
        if (reset && u.reset() != 0) return MXQ_ERR_CUDA;
    }
    if (reset) debug_checked_launches().store(0);
#else
    (void)reset;
#endif
    return MXQ_OK;
}

int mxq_debug_trim_ranges(size_t bytes)
{
#ifdef MXQ_DEBUG
    debug_pending().trim = bytes;
    return 1;
#else
    (void)bytes;
    return 0;
#endif
}

int mxq_format_bits(int fmt) { return valid_format(fmt) ? fmt_info(fmt).bits : 0; }

size_t mxq_codes_bytes(size_t n, int fmt) { return valid_format(fmt) ? n * (size_t)fmt_info(fmt).bits / 8 : 0; }

size_t mxq_scales_bytes(size_t n, int block) { return block > 0 ? n / (size_t)block : 0; }

int mxq_block_supported(int block) { return valid_block(block) ? 1 : 0; }

int mxq_quantize(const void* src, int src_dtype, size_t n, int fmt, int block, void* codes, uint8_t* scales,
                 mxq_stream stream)
{
    if (!valid_format(fmt) || !valid_dtype(src_dtype)) return MXQ_ERR_FORMAT;
    if (int rc = check_sizes(n, block)) return rc;
    if (n == 0) return MXQ_OK;
    if (!src || !codes || !scales) return MXQ_ERR_NULL;
    if (!aligned(src, 32) || !aligned(codes, 32) || !aligned(scales, 16)) return MXQ_ERR_ALIGN;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(src, n * (src_dtype == MXQ_F32 ? 4u : 2u));
    MXQ_DEBUG_EXPECT(codes, n * (size_t)fmt_info(fmt).bits / 8);
    MXQ_DEBUG_EXPECT(scales, n / (size_t)block);
    return launch_quantize(src, src_dtype, n, fmt, block, codes, scales, static_cast<cudaStream_t>(stream));
}

int mxq_slice_scale(const void* codes, const uint8_t* scales, size_t n, int block, int src_fmt, int dst_fmt,
                    void* out_codes, uint8_t* out_scales, mxq_stream stream)
{
    if (!valid_format(src_fmt) || !valid_format(dst_fmt)) return MXQ_ERR_FORMAT;
    if (int rc = check_sizes(n, block)) return rc;
    if (n % 32) return MXQ_ERR_SIZE;
    if (!ss_pair_ok(src_fmt, dst_fmt)) return MXQ_ERR_PAIR;
    if (n == 0) return MXQ_OK;
    if (!codes || !scales || !out_codes || !out_scales) return MXQ_ERR_NULL;
    if (!aligned(codes, 32) || !aligned(out_codes, 32) || !aligned(scales, 16) || !aligned(out_scales, 16))
        return MXQ_ERR_ALIGN;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(codes, n * (size_t)fmt_info(src_fmt).bits / 8);
    MXQ_DEBUG_EXPECT(scales, n / (size_t)block);
    MXQ_DEBUG_EXPECT(out_codes, n * (size_t)fmt_info(dst_fmt).bits / 8);
    MXQ_DEBUG_EXPECT(out_scales, n / (size_t)block);
    return launch_slice_scale(codes, scales, n, block, src_fmt, dst_fmt, out_codes, out_scales,
                              static_cast<cudaStream_t>(stream));
}

int mxq_slice_scale_multi(const void* codes, const uint8_t* scales, size_t n, int block, int src_fmt, int ntargets,
                          const int* dst_fmts, void* const* out_codes, uint8_t* const* out_scales, mxq_stream stream)
{
    if (ntargets < 0 || ntargets > MXQ_MULTI_TARGETS_MAX) return MXQ_ERR_SIZE;
    if (ntargets == 0) return MXQ_OK;
    if (!dst_fmts || !out_codes || !out_scales) return MXQ_ERR_NULL;
    if (!valid_format(src_fmt)) return MXQ_ERR_FORMAT;
    for (int t = 0; t < ntargets; ++t)
        if (!valid_format(dst_fmts[t])) return MXQ_ERR_FORMAT;
    if (int rc = check_sizes(n, block)) return rc;
    if (n % 32) return MXQ_ERR_SIZE;
    for (int t = 0; t < ntargets; ++t)
        if (!ss_pair_ok(src_fmt, dst_fmts[t])) return MXQ_ERR_PAIR;
    if (n == 0) return MXQ_OK;
    if (!codes || !scales) return MXQ_ERR_NULL;
    if (!aligned(codes, 32) || !aligned(scales, 16)) return MXQ_ERR_ALIGN;
    for (int t = 0; t < ntargets; ++t) {
        if (!out_codes[t] || !out_scales[t]) return MXQ_ERR_NULL;
        if (!aligned(out_codes[t], 32) || !aligned(out_scales[t], 16)) return MXQ_ERR_ALIGN;
    }
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(codes, n * (size_t)fmt_info(src_fmt).bits / 8);
    MXQ_DEBUG_EXPECT(scales, n / (size_t)block);
    for (int k = 0; k < ntargets; ++k) {
        MXQ_DEBUG_EXPECT(out_codes[k], n * (size_t)fmt_info(dst_fmts[k]).bits / 8);
        MXQ_DEBUG_EXPECT(out_scales[k], n / (size_t)block);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int t = 0;
    while (t < ntargets) {
        if (t + 1 < ntargets) {
            const int rc = launch_slice_scale2(codes, scales, n, block, src_fmt, dst_fmts[t], dst_fmts[t + 1], out_codes[t],
                                               out_scales[t], out_codes[t + 1], out_scales[t + 1], s);
            if (rc == MXQ_OK) { t += 2; continue; }
            if (rc != MXQ_ERR_PAIR) return rc;          // no fused kernel for this pair: one at a time
        }
        if (int rc = launch_slice_scale(codes, scales, n, block, src_fmt, dst_fmts[t], out_codes[t], out_scales[t], s))
            return rc;
        ++t;
    }
    return MXQ_OK;
}

int mxq_dequantize(const void* codes, const uint8_t* scales, size_t n, int fmt, int block, void* dst, int dst_dtype,
                   mxq_stream stream)
{
    if (!valid_format(fmt) || !valid_dtype(dst_dtype)) return MXQ_ERR_FORMAT;
    if (int rc = check_sizes(n, block)) return rc;
    if (n % 32) return MXQ_ERR_SIZE;
    if (n == 0) return MXQ_OK;
    if (!codes || !scales || !dst) return MXQ_ERR_NULL;
    if (!aligned(codes, 32) || !aligned(dst, 32) || !aligned(scales, 16)) return MXQ_ERR_ALIGN;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(codes, n * (size_t)fmt_info(fmt).bits / 8);
    MXQ_DEBUG_EXPECT(scales, n / (size_t)block);
    MXQ_DEBUG_EXPECT(dst, n * (dst_dtype == MXQ_F32 ? 4u : 2u));
    return launch_dequantize(codes, scales, n, fmt, block, dst, dst_dtype, static_cast<cudaStream_t>(stream));
}

int mxq_fake_quant(const void* src, int dtype, size_t n, int fmt, int block, int mode, void* dst, mxq_stream stream)
{
    if (!valid_format(fmt) || !valid_dtype(dtype)) return MXQ_ERR_FORMAT;
    if (mode != MXQ_FQ_DIRECT && mode != MXQ_FQ_VIA_ANCHOR) return MXQ_ERR_FORMAT;
    if (int rc = check_sizes(n, block)) return rc;
    if (n == 0) return MXQ_OK;
    if (!src || !dst) return MXQ_ERR_NULL;
    if (!aligned(src, 32) || !aligned(dst, 32)) return MXQ_ERR_ALIGN;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(src, n * (dtype == MXQ_F32 ? 4u : 2u));
    MXQ_DEBUG_EXPECT(dst, n * (dtype == MXQ_F32 ? 4u : 2u));
    return launch_fake_quant(src, dtype, n, fmt, block, mode, dst, static_cast<cudaStream_t>(stream));
}

int mxq_fake_quant_batched(const mxq_fq_item* items, int count, int dtype, int fmt, int block, int mode,
                           mxq_stream stream)
{
    if (!valid_format(fmt) || !valid_dtype(dtype)) return MXQ_ERR_FORMAT;
    if (mode != MXQ_FQ_DIRECT && mode != MXQ_FQ_VIA_ANCHOR) return MXQ_ERR_FORMAT;
    if (!valid_block(block)) return MXQ_ERR_BLOCK;
    if (count < 0) return MXQ_ERR_SIZE;
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;
    const size_t epl = dtype == MXQ_F32 ? 8 : 16;           // elements per 32-byte lane unit
    for (int i = 0; i < count; ++i) {
        const mxq_fq_item& it = items[i];
        if (it.n % (size_t)block) return MXQ_ERR_SIZE;
        if (it.n == 0) continue;
        if (!it.src || !it.dst) return MXQ_ERR_NULL;
        if (!aligned(it.src, 32) || !aligned(it.dst, 32)) return MXQ_ERR_ALIGN;
    }
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        MXQ_DEBUG_EXPECT(items[i].src, items[i].n * (dtype == MXQ_F32 ? 4u : 2u));
        MXQ_DEBUG_EXPECT(items[i].dst, items[i].n * (dtype == MXQ_F32 ? 4u : 2u));
    }
    // launches of at most kFqBatchItemsMax tensors each: the item table rides in the kernel parameters
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<FqDeviceItem> chunk;
    chunk.reserve(kFqBatchItemsMax);
    size_t tiles = 0;
    auto flush = [&]() -> int {
        if (chunk.empty()) return MXQ_OK;
        const int rc = launch_fake_quant_batched(chunk.data(), (int)chunk.size(), tiles, dtype, fmt, block, mode, s);
        chunk.clear();
        tiles = 0;
        return rc;
    };
    for (int i = 0; i < count; ++i) {
        const mxq_fq_item& it = items[i];
        if (it.n == 0) continue;
        FqDeviceItem d;
        d.src = static_cast<const uint8_t*>(it.src);
        d.dst = static_cast<uint8_t*>(it.dst);
        d.nunits = it.n / epl;
        d.tile_begin = tiles;
        tiles += fq_batched_tiles(d.nunits);
        chunk.push_back(d);
        if ((int)chunk.size() == kFqBatchItemsMax)
            if (int rc = flush()) return rc;
    }
    return flush();
}

int mxq_quantize_batched(const mxq_q_item* items, int count, int src_dtype, int fmt, int block, mxq_stream stream)
{
    if (!valid_format(fmt) || !valid_dtype(src_dtype)) return MXQ_ERR_FORMAT;
    if (!valid_block(block)) return MXQ_ERR_BLOCK;
    if (count < 0) return MXQ_ERR_SIZE;
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;
    const size_t epl = src_dtype == MXQ_F32 ? 8 : 16;       // elements per 32-byte lane unit
    for (int i = 0; i < count; ++i) {
        const mxq_q_item& it = items[i];
        if (it.n % (size_t)block) return MXQ_ERR_SIZE;
        if (it.n == 0) continue;
        if (!it.src || !it.codes || !it.scales) return MXQ_ERR_NULL;
        if (!aligned(it.src, 32) || !aligned(it.codes, 32) || !aligned(it.scales, 16)) return MXQ_ERR_ALIGN;
    }
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        MXQ_DEBUG_EXPECT(items[i].src, items[i].n * (src_dtype == MXQ_F32 ? 4u : 2u));
        MXQ_DEBUG_EXPECT(items[i].codes, items[i].n * (size_t)fmt_info(fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].scales, items[i].n / (size_t)block);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<QDeviceItem> chunk;
    chunk.reserve(kQBatchItemsMax);
    size_t tiles = 0;
    auto flush = [&]() -> int {
        if (chunk.empty()) return MXQ_OK;
        const int rc = launch_quantize_batched(chunk.data(), (int)chunk.size(), tiles, src_dtype, fmt, block, s);
        chunk.clear();
        tiles = 0;
        return rc;
    };
    for (int i = 0; i < count; ++i) {
        const mxq_q_item& it = items[i];
        if (it.n == 0) continue;
        QDeviceItem d;
        d.src = static_cast<const uint8_t*>(it.src);
        d.codes = static_cast<uint8_t*>(it.codes);
        d.scales = it.scales;
        d.nunits = it.n / epl;
        d.tile_begin = tiles;
        tiles += q_batched_tiles(d.nunits);
        chunk.push_back(d);
        if ((int)chunk.size() == kQBatchItemsMax)
            if (int rc = flush()) return rc;
    }
    return flush();
}

int mxq_dequantize_batched(const mxq_dq_item* items, int count, int fmt, int block, int dst_dtype, mxq_stream stream)
{
    if (!valid_format(fmt) || !valid_dtype(dst_dtype)) return MXQ_ERR_FORMAT;
    if (!valid_block(block)) return MXQ_ERR_BLOCK;
    if (count < 0) return MXQ_ERR_SIZE;
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;
    for (int i = 0; i < count; ++i) {
        const mxq_dq_item& it = items[i];
        if (it.n % (size_t)block || it.n % 32) return MXQ_ERR_SIZE;
        if (it.n == 0) continue;
        if (!it.codes || !it.scales || !it.dst) return MXQ_ERR_NULL;
        if (!aligned(it.codes, 32) || !aligned(it.dst, 32) || !aligned(it.scales, 16)) return MXQ_ERR_ALIGN;
    }
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        MXQ_DEBUG_EXPECT(items[i].codes, items[i].n * (size_t)fmt_info(fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].scales, items[i].n / (size_t)block);
        MXQ_DEBUG_EXPECT(items[i].dst, items[i].n * (dst_dtype == MXQ_F32 ? 4u : 2u));
    }
    const size_t epu = dst_dtype == MXQ_F32 ? 8 : 32;        // elements per lane unit of the kernel that writes dst_dtype
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<DqDeviceItem> chunk;
    chunk.reserve(kDqBatchItemsMax);
    size_t tiles = 0;
    auto flush = [&]() -> int {
        if (chunk.empty()) return MXQ_OK;
        const int rc = launch_dequantize_batched(chunk.data(), (int)chunk.size(), tiles, fmt, block, dst_dtype, s);
        chunk.clear();
        tiles = 0;
        return rc;
    };
    for (int i = 0; i < count; ++i) {
        const mxq_dq_item& it = items[i];
        if (it.n == 0) continue;
        DqDeviceItem d;
        d.codes = static_cast<const uint8_t*>(it.codes);
        d.scales = it.scales;
        d.dst = static_cast<uint8_t*>(it.dst);
        d.nunits = it.n / epu;
        d.tile_begin = tiles;
        tiles += dq_batched_tiles(d.nunits);
        chunk.push_back(d);
        if ((int)chunk.size() == kDqBatchItemsMax)
            if (int rc = flush()) return rc;
    }
    return flush();
}

int mxq_fake_quant_bwd(const void* grad_out, int dtype, size_t n, void* grad_in, mxq_stream stream)
{
    if (!valid_dtype(dtype)) return MXQ_ERR_FORMAT;
    if (n == 0) return MXQ_OK;
    if (!grad_out || !grad_in) return MXQ_ERR_NULL;
    if (!aligned(grad_out, 32) || !aligned(grad_in, 32)) return MXQ_ERR_ALIGN;
    if (grad_out == grad_in) return MXQ_OK;
    MXQ_DEBUG_SCOPE();
    MXQ_DEBUG_EXPECT(grad_out, n * (dtype == MXQ_F32 ? 4u : 2u));
    MXQ_DEBUG_EXPECT(grad_in, n * (dtype == MXQ_F32 ? 4u : 2u));
    return launch_copy(grad_out, n * (dtype == MXQ_F32 ? 4u : 2u), grad_in, static_cast<cudaStream_t>(stream));
}

int mxq_slice_scale_batched(const mxq_ss_item* items, int count, int block, int src_fmt, int dst_fmt,
                            mxq_stream stream)
{
    if (!valid_format(src_fmt) || !valid_format(dst_fmt)) return MXQ_ERR_FORMAT;
    if (!valid_block(block)) return MXQ_ERR_BLOCK;
    if (block < 32) return MXQ_ERR_BLOCK;          // the batched sweep keeps one scale per code unit or fewer
    if (!ss_pair_ok(src_fmt, dst_fmt)) return MXQ_ERR_PAIR;
    if (count < 0) return MXQ_ERR_SIZE;
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;

    std::vector<SsDeviceItem> host;
    host.reserve((size_t)count);
    size_t tiles = 0;
    for (int i = 0; i < count; ++i) {
        const mxq_ss_item& it = items[i];
        if (it.n % (size_t)block || it.n % 32) return MXQ_ERR_SIZE;
        if (it.n == 0) continue;
        if (!it.codes || !it.scales || !it.out_codes || !it.out_scales) return MXQ_ERR_NULL;
        if (!aligned(it.codes, 32) || !aligned(it.out_codes, 32) || !aligned(it.scales, 16) ||
            !aligned(it.out_scales, 16))
            return MXQ_ERR_ALIGN;
        SsDeviceItem d;
        d.codes = static_cast<const uint8_t*>(it.codes);
        d.scales = it.scales;
        d.out_codes = static_cast<uint8_t*>(it.out_codes);
        d.out_scales = it.out_scales;
        d.nunits = it.n / 32;
        d.nscales = it.n / (size_t)block;
        d.tile_begin = tiles;
        tiles += ss_batched_tiles(d.nunits);
        host.push_back(d);
    }
    if (host.empty()) return MXQ_OK;
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        MXQ_DEBUG_EXPECT(items[i].codes, items[i].n * (size_t)fmt_info(src_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].scales, items[i].n / (size_t)block);
        MXQ_DEBUG_EXPECT(items[i].out_codes, items[i].n * (size_t)fmt_info(dst_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].out_scales, items[i].n / (size_t)block);
    }

    // the item table rides in the kernel's parameter space, kSsParamItemsMax tensors per launch: nothing
    // to allocate or copy, no state shared between calls; larger sets take several launches (each
    // launch's tiles are numbered from zero)
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (size_t first = 0; first < host.size(); first += kSsParamItemsMax) {
        const size_t cnt = host.size() - first < (size_t)kSsParamItemsMax ? host.size() - first : (size_t)kSsParamItemsMax;
        const size_t base = host[first].tile_begin;
        for (size_t i = first; i < first + cnt; ++i) host[i].tile_begin -= base;
        const size_t end = first + cnt < host.size() ? host[first + cnt].tile_begin : tiles;
        if (int rc = launch_slice_scale_batched_params(host.data() + first, (int)cnt, end - base, src_fmt, dst_fmt, s))
            return rc;
    }
    return MXQ_OK;
}

int mxq_slice_scale_pair_batched(const mxq_ss_pair_item* items, int count, int block, int src_fmt, int dst_fmt1,
                                 int dst_fmt2, mxq_stream stream)
{
    if (!valid_format(src_fmt) || !valid_format(dst_fmt1) || !valid_format(dst_fmt2)) return MXQ_ERR_FORMAT;
    if (!valid_block(block)) return MXQ_ERR_BLOCK;
    if (block < 32) return MXQ_ERR_BLOCK;
    if (!ss_pair_ok(src_fmt, dst_fmt1) || !ss_pair_ok(src_fmt, dst_fmt2)) return MXQ_ERR_PAIR;
    if (count < 0) return MXQ_ERR_SIZE;
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;
    for (int i = 0; i < count; ++i) {
        const mxq_ss_pair_item& it = items[i];
        if (it.n % (size_t)block || it.n % 32) return MXQ_ERR_SIZE;
        if (it.n == 0) continue;
        if (!it.codes || !it.scales || !it.out_codes1 || !it.out_scales1 || !it.out_codes2 || !it.out_scales2)
            return MXQ_ERR_NULL;
        if (!aligned(it.codes, 32) || !aligned(it.out_codes1, 32) || !aligned(it.out_codes2, 32) ||
            !aligned(it.scales, 16) || !aligned(it.out_scales1, 16) || !aligned(it.out_scales2, 16))
            return MXQ_ERR_ALIGN;
    }
    if (!slice_scale2_is_fused(src_fmt, dst_fmt1, dst_fmt2)) {
        // no fused kernel for this pair of targets: one single-target batched pass each
        std::vector<mxq_ss_item> one((size_t)count);
        for (int t = 0; t < 2; ++t) {
            for (int i = 0; i < count; ++i) {
                mxq_ss_item& o = one[(size_t)i];
                o.codes = items[i].codes;
                o.scales = items[i].scales;
                o.n = items[i].n;
                o.out_codes = t ? items[i].out_codes2 : items[i].out_codes1;
                o.out_scales = t ? items[i].out_scales2 : items[i].out_scales1;
            }
            if (int rc = mxq_slice_scale_batched(one.data(), count, block, src_fmt, t ? dst_fmt2 : dst_fmt1, stream)) return rc;
        }
        return MXQ_OK;
    }
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        MXQ_DEBUG_EXPECT(items[i].codes, items[i].n * (size_t)fmt_info(src_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].scales, items[i].n / (size_t)block);
        MXQ_DEBUG_EXPECT(items[i].out_codes1, items[i].n * (size_t)fmt_info(dst_fmt1).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].out_scales1, items[i].n / (size_t)block);
        MXQ_DEBUG_EXPECT(items[i].out_codes2, items[i].n * (size_t)fmt_info(dst_fmt2).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].out_scales2, items[i].n / (size_t)block);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<Ss2DeviceItem> chunk;
    chunk.reserve(kSs2BatchItemsMax);
    size_t tiles = 0;
    auto flush = [&]() -> int {
        if (chunk.empty()) return MXQ_OK;
        const int rc = launch_slice_scale2_batched(chunk.data(), (int)chunk.size(), tiles, src_fmt, dst_fmt1, dst_fmt2, s);
        chunk.clear();
        tiles = 0;
        return rc;
    };
    for (int i = 0; i < count; ++i) {
        const mxq_ss_pair_item& it = items[i];
        if (it.n == 0) continue;
        Ss2DeviceItem d;
        d.codes = static_cast<const uint8_t*>(it.codes);
        d.scales = it.scales;
        d.out_codes1 = static_cast<uint8_t*>(it.out_codes1);
        d.out_scales1 = it.out_scales1;
        d.out_codes2 = static_cast<uint8_t*>(it.out_codes2);
        d.out_scales2 = it.out_scales2;
        d.nunits = it.n / 32;
        d.nscales = it.n / (size_t)block;
        d.tile_begin = tiles;
        tiles += ss2_batched_tiles(d.nunits);
        chunk.push_back(d);
        if ((int)chunk.size() == kSs2BatchItemsMax)
            if (int rc = flush()) return rc;
    }
    return flush();
}

}  // extern "C"
#pragma GCC visibility pop
