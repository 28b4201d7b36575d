// mxq_slice_scale_batched_static: the whole-model Slice-and-Scale launch for callers that must not
// allocate device memory.  The item table that the batched kernel reads sits in a fixed array that
// is part of the library image instead of a cudaMalloc'd buffer.
//
// Who needs this: a serving process that has handed the whole HBM to its own pool (weights, KV
// cache) so that a stray cudaMalloc fails or eats into a budget somebody else planned; and a
// loop that must not take the device-wide synchronisation cudaMalloc / cudaFree imply.
// What the call still costs: a 57 KiB table on the caller's stack (a thread with a small stack
// needs about 64 KiB free), a stream-ordered copy of 0.6 - 57 KiB from that pageable table, for
// which the runtime may make the host wait on the stream, and on the first call per device the
// lookup of the array's address (which can load the library's device code).
#include <cstddef>
#include <mutex>

#include "mxq_kernels.cuh"
#include "mxq_launch.h"

namespace mxq {
namespace {

constexpr int kMaxDevices = 64;

// What one call hands to the kernel: the coarse index over the tile space, then the items.
struct StaticTable {
    TileIndex index;
    SsDeviceItem items[MXQ_STATIC_BATCH_MAX];
};

// The table itself: MXQ_STATIC_BATCH_MAX items of 56 bytes and the 520-byte index = 57 KiB on every GPU
// that loads the library, for the life of the process.  In host code this name is only a handle for
// cudaGetSymbolAddress; it is not a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_static_items[sizeof(StaticTable)];

std::mutex g_static_mutex;
StaticTable* g_static_table[kMaxDevices];       // device address of g_static_items, per device

// Device address of the table on the current device; looked up once per device, with that device
// current (the caller's), on the first call that reaches here.
int static_table(StaticTable** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MXQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_table[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_items) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return MXQ_ERR_CUDA;
        }
        g_static_table[dev] = static_cast<StaticTable*>(p);
    }
    *out = g_static_table[dev];
    return MXQ_OK;
}

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace
}  // namespace mxq

using namespace mxq;

#pragma GCC visibility push(default)
extern "C" int mxq_slice_scale_batched_static(const mxq_ss_item* items, int count, int block, int src_fmt,
                                              int dst_fmt, mxq_stream stream)
{
    if (fmt_info(src_fmt).kind < 0 || fmt_info(dst_fmt).kind < 0) return MXQ_ERR_FORMAT;
    if (block != 32 && block != 64 && block != 128) return MXQ_ERR_BLOCK;
    if (!ss_pair_ok(src_fmt, dst_fmt)) return MXQ_ERR_PAIR;
    if (count < 0 || count > MXQ_STATIC_BATCH_MAX) return MXQ_ERR_SIZE;     // beyond the fixed table
    if (count == 0) return MXQ_OK;
    if (!items) return MXQ_ERR_NULL;

    // host copy of the table on the stack: no heap, no pinned allocation
    StaticTable staged;
    SsDeviceItem* host = staged.items;
    int used = 0;
    size_t tiles = 0;
    for (int i = 0; i < count; ++i) {
        const mxq_ss_item& it = items[i];
        if (it.n % (size_t)block || it.n % 32) return MXQ_ERR_SIZE;
        if (it.n == 0) continue;
        if (!it.codes || !it.scales || !it.out_codes || !it.out_scales) return MXQ_ERR_NULL;
        if (!aligned(it.codes, 32) || !aligned(it.out_codes, 32) || !aligned(it.scales, 16) ||
            !aligned(it.out_scales, 16))
            return MXQ_ERR_ALIGN;
        SsDeviceItem& d = host[used++];
        d.codes = static_cast<const uint8_t*>(it.codes);
        d.scales = it.scales;
        d.out_codes = static_cast<uint8_t*>(it.out_codes);
        d.out_scales = it.out_scales;
        d.nunits = it.n / 32;
        d.nscales = it.n / (size_t)block;
        d.tile_begin = tiles;
        tiles += ss_batched_tiles(d.nunits);
    }
    if (used == 0) return MXQ_OK;
    MXQ_DEBUG_SCOPE();
    for (int i = 0; i < count; ++i) {
        MXQ_DEBUG_EXPECT(items[i].codes, items[i].n * (size_t)fmt_info(src_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].scales, items[i].n / (size_t)block);
        MXQ_DEBUG_EXPECT(items[i].out_codes, items[i].n * (size_t)fmt_info(dst_fmt).bits / 8);
        MXQ_DEBUG_EXPECT(items[i].out_scales, items[i].n / (size_t)block);
    }

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The table copy below reads `staged`, which is gone when this function returns.  A stream that is
    // being captured would record the copy instead of performing it, and every later replay would read
    // a dead stack frame and hand the kernel garbage pointers: refuse before anything is enqueued.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    if (capturing != cudaStreamCaptureStatusNone) return MXQ_ERR_CUDA;

    build_tile_index(staged.index, host, used, tiles);
    StaticTable* table = nullptr;
    if (int rc = static_table(&table)) return rc;
    // Entries [0, used) are rewritten by every call and the kernel reads no others, so nothing in
    // the table has to start from zero.  The source is pageable stack memory: the runtime has
    // staged the bytes by the time this returns (it may make the host wait for earlier work of the
    // stream to do so).
    const size_t nbytes = offsetof(StaticTable, items) + sizeof(SsDeviceItem) * (size_t)used;
    if (cudaMemcpyAsync(table, &staged, nbytes, cudaMemcpyHostToDevice, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    return launch_slice_scale_batched(table->items, &table->index, used, tiles, src_fmt, dst_fmt, s);
}
#pragma GCC visibility pop
