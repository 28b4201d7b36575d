// Bounds checking for debug builds of libmxq (-DMXQ_DEBUG; compute-sanitizer's job, done by the
// library itself so that it runs anywhere).  The C ABI layer registers the byte range of every
// buffer an entry point was given -- computed there from the element count, the format's width and
// the block size, not from the kernels' own index arithmetic.  Before each launch the launcher
// uploads the merged ranges to a table in device memory, and every global access the kernels make
// through the helpers of mxq_access.cuh is tested against it: an access that leaves every range is
// counted, its address recorded, and the access is SKIPPED (loads return zero) -- nothing traps and
// nothing faults, the host reads the outcome with mxq_debug_report().  Release builds compile all of
// this to nothing.
//
// One table per translation unit (a kernel's launcher lives in the kernel's unit); the units
// register a reader with a process-wide list, which mxq_debug_report() sums over.  The table belongs
// to the launch in flight: debug builds are for one stream at a time.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#ifdef MXQ_DEBUG
#include <algorithm>
#include <atomic>
#include <utility>
#include <vector>
#endif

namespace mxq {

#ifdef MXQ_DEBUG

constexpr int kDebugRanges = 4608;           // 1024 batched items x 4 buffers, and some

struct DebugRange {
    unsigned long long lo, hi;               // [lo, hi)
};

struct DebugState {
    unsigned int count;                      // ranges of the launch in flight; 0 = accesses are not checked
    unsigned int violations;                 // accesses outside every range (each one skipped)
    unsigned long long first_bad;            // address of the first one
    unsigned int first_bytes;                // and its size
    unsigned int pad;
    DebugRange ranges[kDebugRanges];         // sorted by lo, disjoint
};

namespace {
__device__ DebugState g_debug;
}

// True when [p, p + bytes) lies inside one registered range (or nothing is registered, or p is shared memory).
__device__ __forceinline__ bool debug_ok(const void* p, unsigned int bytes)
{
    const unsigned int n = g_debug.count;
    if (n == 0) return true;
    if (__isShared(p)) return true;          // the staging tiles are written with the same helpers
    const unsigned long long a = (unsigned long long)p;
    unsigned int lo = 0, hi = n;             // the last range that starts at or before a
    while (lo + 1 < hi) {
        const unsigned int mid = (lo + hi) >> 1;
        if (g_debug.ranges[mid].lo <= a) lo = mid;
        else hi = mid;
    }
    if (g_debug.ranges[lo].lo <= a && a + bytes <= g_debug.ranges[lo].hi) return true;
    if (atomicAdd(&g_debug.violations, 1u) == 0) {
        g_debug.first_bad = a;
        g_debug.first_bytes = bytes;
    }
    return false;
}

// ---- host side -----------------------------------------------------------------------------------

struct DebugPending {
    std::vector<DebugRange> ranges;          // what the entry point in progress registered (this thread)
    size_t trim = 0;                         // test hook: register every range this many bytes short
};

inline DebugPending& debug_pending()
{
    static thread_local DebugPending p;
    return p;
}

inline std::atomic<unsigned int>& debug_checked_launches()
{
    static std::atomic<unsigned int> n{0};
    return n;
}

inline void debug_expect(const void* p, size_t bytes)
{
    DebugPending& d = debug_pending();
    if (!p || bytes <= d.trim) return;
    d.ranges.push_back(DebugRange{(unsigned long long)(uintptr_t)p, (unsigned long long)(uintptr_t)p + bytes - d.trim});
}

// Clears what an entry point registered when it returns, whichever way it returns.
struct DebugScope {
    DebugScope() { debug_pending().ranges.clear(); }
    ~DebugScope() { debug_pending().ranges.clear(); }
};

struct DebugUnit {
    int (*read)(unsigned int* violations, unsigned long long* first_bad, unsigned int* first_bytes);
    int (*reset)();
};

inline std::vector<DebugUnit>& debug_units()
{
    static std::vector<DebugUnit> units;
    return units;
}

namespace {

// Uploads the pending ranges (sorted, overlapping and adjacent ones merged) to this unit's table,
// ordered on `stream` in front of the launch that follows.  The sources are pageable host memory:
// the runtime has staged them when the calls return.
inline int debug_upload(cudaStream_t stream)
{
    std::vector<DebugRange> r = debug_pending().ranges;
    std::sort(r.begin(), r.end(), [](const DebugRange& a, const DebugRange& b) { return a.lo < b.lo; });
    std::vector<DebugRange> merged;
    for (const DebugRange& x : r) {
        if (!merged.empty() && x.lo <= merged.back().hi) merged.back().hi = std::max(merged.back().hi, x.hi);
        else merged.push_back(x);
    }
    unsigned int count = merged.size() <= (size_t)kDebugRanges ? (unsigned int)merged.size() : 0u;
    if (count && cudaMemcpyToSymbolAsync(g_debug, merged.data(), sizeof(DebugRange) * count, offsetof(DebugState, ranges),
                                         cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return -1;
    if (cudaMemcpyToSymbolAsync(g_debug, &count, sizeof(count), offsetof(DebugState, count), cudaMemcpyHostToDevice,
                                stream) != cudaSuccess)
        return -1;
    if (count) debug_checked_launches().fetch_add(1);
    return 0;
}

inline int debug_read_unit(unsigned int* violations, unsigned long long* first_bad, unsigned int* first_bytes)
{
    struct {                                  // the fields in front of the ranges
        unsigned int count, violations;
        unsigned long long first_bad;
        unsigned int first_bytes, pad;
    } head;
    static_assert(sizeof(head) == offsetof(DebugState, ranges), "header layout");
    if (cudaMemcpyFromSymbol(&head, g_debug, sizeof(head)) != cudaSuccess) return -1;
    *violations = head.violations;
    *first_bad = head.first_bad;
    *first_bytes = head.first_bytes;
    return 0;
}

inline int debug_reset_unit()
{
    const unsigned int zero[6] = {0, 0, 0, 0, 0, 0};
    return cudaMemcpyToSymbol(g_debug, zero, offsetof(DebugState, ranges)) == cudaSuccess ? 0 : -1;
}

struct DebugRegistrar {
    DebugRegistrar() { debug_units().push_back(DebugUnit{&debug_read_unit, &debug_reset_unit}); }
};
DebugRegistrar g_debug_registrar;

}  // namespace

#define MXQ_DEBUG_SCOPE() ::mxq::DebugScope mxq_debug_scope_
#define MXQ_DEBUG_EXPECT(p, bytes) ::mxq::debug_expect((p), (bytes))

#else  // release

#define MXQ_DEBUG_SCOPE() ((void)0)
#define MXQ_DEBUG_EXPECT(p, bytes) ((void)0)

#endif

}  // namespace mxq
