// Global-memory access helpers: 256-bit and 128-bit vector loads/stores (sm_100a has 32-byte
// global accesses), lane-sized ragged pieces for the sub-byte code streams, and the bitstream
// pack/unpack of element codes in registers.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "mxq_debug.cuh"

namespace mxq {

// In debug builds (-DMXQ_DEBUG) every access below is first tested against the byte ranges the entry
// point registered (mxq_debug.cuh); one that falls outside is counted and skipped.
#ifdef MXQ_DEBUG
#define MXQ_CHECKED(p, bytes, on_fail) \
    if (!::mxq::debug_ok((p), (bytes))) { on_fail; }
#else
#define MXQ_CHECKED(p, bytes, on_fail)
#endif

// ---- programmatic dependent launch ----------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialization allowed: its
// CTAs may become resident while the previous kernel of the stream is still draining, so the
// ~2 us launch gap between short kernels disappears.  pdl_release() lets the next kernel start
// launching; pdl_acquire() blocks until the previous kernel has completed and its writes are
// visible.  Each kernel calls pdl_release() first and pdl_acquire() before its first global
// load or store (and before it returns, so that completion stays transitive along the stream),
// which keeps plain stream-order semantics for every buffer.

__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_acquire() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// What a kernel may do before pdl_acquire(): ask L2 for the lines its first loads will need.  A
// prefetch returns no data to the SM, so issuing it while the previous kernel may still be writing
// is harmless (L2 is where global memory is coherent; the loads after the wait read whatever the
// previous kernel left there).  The CTAs that become resident during the previous kernel's tail --
// up to a quarter of a grid here -- then find their input in L2 when the wait returns, and the
// tail's idle HBM cycles carry the next kernel's first reads: 4 - 9 % on the read-heavy kernels.
// Lane l of the warp that owns `tile` prefetches the line of each of its U units.
template <int U, int UNIT_BYTES>
__device__ __forceinline__ void prefetch_tile(const uint8_t* base, size_t tile, size_t nunits)
{
    const size_t u0 = tile * (32 * U) + (threadIdx.x & 31);
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) asm volatile("prefetch.global.L2 [%0];" :: "l"(base + unit * UNIT_BYTES));
    }
}

// ---- 32-byte accesses ---------------------------------------------------------------------

__device__ __forceinline__ void ld256(uint32_t (&w)[8], const void* p)
{
    MXQ_CHECKED(p, 32, { for (int j = 0; j < 8; ++j) w[j] = 0; return; })
    asm volatile("ld.global.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}

__device__ __forceinline__ void st256(void* p, const uint32_t (&w)[8])
{
    MXQ_CHECKED(p, 32, return)
    asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

// 32 bytes of one repeated word (the quiet-NaN fill of a poisoned block): a store of its own, under the
// block's predicate, instead of eight selects in front of the ordinary store.
__device__ __forceinline__ void st256_splat(void* p, uint32_t v)
{
    MXQ_CHECKED(p, 32, return)
    asm volatile("st.global.v8.u32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1};" :: "l"(p), "r"(v) : "memory");
}

// ---- single bytes (the scale streams) -------------------------------------------------------

__device__ __forceinline__ uint32_t ld_u8(const uint8_t* p)
{
    MXQ_CHECKED(p, 1, return 0)
    return *p;
}

__device__ __forceinline__ void st_u8(uint8_t* p, uint32_t v)
{
    MXQ_CHECKED(p, 1, return)
    *p = (uint8_t)v;
}

// ---- compile-time sized pieces --------------------------------------------------------------

// Largest power of two (<= 32) dividing `bytes`: the alignment every lane's piece keeps when
// lanes own consecutive pieces of `bytes` bytes starting from a 32-byte aligned base.
__host__ __device__ constexpr int piece_align(int bytes)
{
    int a = 1;
    while (a < 32 && bytes % (a * 2) == 0) a *= 2;
    return a;
}

// Load NW 32-bit words (NW*4 bytes) from `p`, which is aligned to piece_align(NW*4).
template <int NW>
__device__ __forceinline__ void load_words(uint32_t (&w)[NW], const void* p)
{
    constexpr int A = piece_align(NW * 4);
    const char* c = static_cast<const char*>(p);
    if constexpr (A != 32) {                                  // (32-byte pieces are checked by ld256)
        MXQ_CHECKED(p, NW * 4, { for (int i = 0; i < NW; ++i) w[i] = 0; return; })
    }
    if constexpr (A == 32) {
#pragma unroll
        for (int i = 0; i < NW; i += 8) {
            uint32_t t[8];
            ld256(t, c + i * 4);
#pragma unroll
            for (int j = 0; j < 8; ++j) w[i + j] = t[j];
        }
    } else if constexpr (A == 16) {
#pragma unroll
        for (int i = 0; i < NW; i += 4) {
            uint4 t = *reinterpret_cast<const uint4*>(c + i * 4);
            w[i] = t.x; w[i + 1] = t.y; w[i + 2] = t.z; w[i + 3] = t.w;
        }
    } else if constexpr (A == 8) {
#pragma unroll
        for (int i = 0; i < NW; i += 2) {
            uint2 t = *reinterpret_cast<const uint2*>(c + i * 4);
            w[i] = t.x; w[i + 1] = t.y;
        }
    } else {
        static_assert(A == 4, "pieces are whole words");
#pragma unroll
        for (int i = 0; i < NW; ++i) w[i] = *reinterpret_cast<const uint32_t*>(c + i * 4);
    }
}

// Load NB bytes (any count) from `p`, which is aligned to piece_align(NB), into the low bytes of
// the word array; bytes beyond NB are zero.
template <int NB, int NW>
__device__ __forceinline__ void load_bytes(uint32_t (&w)[NW], const void* p)
{
    static_assert(NW * 4 >= NB, "not enough words");
    if constexpr (NB % 4 == 0) {
        load_words<NB / 4>(w, p);
    } else {
        constexpr int A = piece_align(NB);                     // 1 or 2
        const char* c = static_cast<const char*>(p);
#pragma unroll
        for (int i = 0; i < NW; ++i) w[i] = 0;
        MXQ_CHECKED(p, NB, return)
        if constexpr (A == 2) {
#pragma unroll
            for (int i = 0; i < NB / 2; ++i)
                w[i / 2] |= (uint32_t)*reinterpret_cast<const uint16_t*>(c + i * 2) << ((i & 1) * 16);
        } else {
#pragma unroll
            for (int i = 0; i < NB; ++i) w[i / 4] |= (uint32_t)*reinterpret_cast<const uint8_t*>(c + i) << ((i & 3) * 8);
        }
    }
}

// Store the low NB bytes of the word array to `p`, which is aligned to piece_align(NB).
template <int NB, int NW>
__device__ __forceinline__ void store_bytes(void* p, const uint32_t (&w)[NW])
{
    static_assert(NW * 4 >= NB, "not enough words");
    constexpr int A = piece_align(NB);
    char* c = static_cast<char*>(p);
    if constexpr (A != 32) {                                  // (32-byte pieces are checked by st256)
        MXQ_CHECKED(p, NB, return)
    }
    if constexpr (A == 32) {
#pragma unroll
        for (int i = 0; i < NB / 4; i += 8) {
            uint32_t t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) t[j] = w[i + j];
            st256(c + i * 4, t);
        }
    } else if constexpr (A == 16) {
#pragma unroll
        for (int i = 0; i < NB / 4; i += 4)
            *reinterpret_cast<uint4*>(c + i * 4) = make_uint4(w[i], w[i + 1], w[i + 2], w[i + 3]);
    } else if constexpr (A == 8) {
#pragma unroll
        for (int i = 0; i < NB / 4; i += 2)
            *reinterpret_cast<uint2*>(c + i * 4) = make_uint2(w[i], w[i + 1]);
    } else if constexpr (A == 4) {
#pragma unroll
        for (int i = 0; i < NB / 4; ++i) *reinterpret_cast<uint32_t*>(c + i * 4) = w[i];
    } else if constexpr (A == 2) {
#pragma unroll
        for (int i = 0; i < NB / 2; ++i)
            *reinterpret_cast<uint16_t*>(c + i * 2) = (uint16_t)(w[i / 2] >> ((i & 1) * 16));
    } else {
#pragma unroll
        for (int i = 0; i < NB; ++i)
            *reinterpret_cast<uint8_t*>(c + i) = (uint8_t)(w[i / 4] >> ((i & 3) * 8));
    }
}

// ---- staged tile stores ------------------------------------------------------------------------
// A lane's piece of packed codes is OB bytes at lane * OB of its warp tile.  When OB is not one
// aligned vector a direct store takes several narrow instructions, each of which touches every
// 32-byte sector of the tile with a few bytes: a 6-bit tile (24 bytes per lane: a 16-byte and an
// 8-byte store at a 24-byte stride) issues 2.9 times its sectors at L1, a 7-bit tile seven 2- or
// 4-byte stores per lane.  Such tiles go through shared memory instead: lanes drop their pieces
// there, and a whole tile leaves as ONE bulk copy shared -> global issued by one lane (the copy
// engine writes full lines; no cluster, no tensor map, no multicast).  Only the ragged last tile of
// a tensor is copied out by the lanes as 16-byte pieces.
// Measured at 2^26 codes: MXINT8 -> MXINT6 and E4M3 -> E2M3 / E3M2 4 - 8 % faster than direct stores;
// the 20-, 12- and 10-byte pieces of the 5- and 3-bit streams are faster stored directly (2 - 8 %).

// store instructions a lane needs for a direct store of OB bytes
__host__ __device__ constexpr int direct_store_count(int bytes) { return bytes / piece_align(bytes); }

template <int OB>
struct StagedTile {
    static constexpr bool use = direct_store_count(OB) > 5 || OB == 24;
};

// Copy the first `nbytes` bytes of a warp's staging area to `gdst`; both are 16-byte aligned and
// TILE_BYTES (a multiple of 16) is the size of a whole tile.  Every lane of the warp calls it, after
// writing its own pieces to the area with ordinary stores.
template <int TILE_BYTES>
__device__ __forceinline__ void flush_stage(const uint8_t* stage, uint8_t* gdst, uint32_t nbytes)
{
    static_assert(TILE_BYTES % 16 == 0, "a bulk copy moves multiples of 16 bytes");
    const uint32_t lane = threadIdx.x & 31;
    if (nbytes == TILE_BYTES) {
        // the lanes' writes become visible to the copy engine, then one lane hands it the tile and
        // waits until the engine has read the area (it may be rewritten or released afterwards)
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        bool ok = true;
        MXQ_CHECKED(gdst, TILE_BYTES, ok = false)
        if (lane == 0 && ok) {
            const uint32_t saddr = (uint32_t)__cvta_generic_to_shared(stage);
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         :: "l"(gdst), "r"(saddr), "r"(TILE_BYTES) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        }
        __syncwarp();
        return;
    }
    __syncwarp();
    for (uint32_t i = lane * 16; i + 16 <= nbytes; i += 512) {
        MXQ_CHECKED(gdst + i, 16, continue)
        *reinterpret_cast<uint4*>(gdst + i) = *reinterpret_cast<const uint4*>(stage + i);
    }
    const uint32_t done = nbytes & ~15u;                        // a ragged tensor end: up to 15 bytes
    if (done + lane < nbytes) st_u8(gdst + done + lane, stage[done + lane]);
    __syncwarp();
}

// ---- bitstream of element codes in registers -------------------------------------------------

// Words needed for N codes of BITS bits.
__host__ __device__ constexpr int code_words(int n, int bits) { return (n * bits + 31) / 32; }

// Insert code number I (BITS wide, already masked) into the little-endian bitstream w[].
template <int BITS, int I, int NW>
__device__ __forceinline__ void put_code(uint32_t (&w)[NW], uint32_t code)
{
    constexpr int off = I * BITS, wi = off >> 5, sh = off & 31;
    if constexpr (sh == 0) w[wi] = code;
    else w[wi] |= code << sh;
    if constexpr (sh + BITS > 32) w[wi + 1] = code >> (32 - sh);
}

// Extract code number I.
template <int BITS, int I, int NW>
__device__ __forceinline__ uint32_t get_code(const uint32_t (&w)[NW])
{
    constexpr int off = I * BITS, wi = off >> 5, sh = off & 31;
    constexpr uint32_t mask = (1u << BITS) - 1u;
    if constexpr (sh + BITS <= 32) return (w[wi] >> sh) & mask;
    else return ((w[wi] >> sh) | (w[wi + 1] << (32 - sh))) & mask;
}

}  // namespace mxq
