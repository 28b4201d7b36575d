// The streaming kernels of libmxq.  Common shape: every lane owns a "unit" of 32 bytes of the
// widest stream it touches (one 256-bit global access), a warp sweeps tiles of 32*U consecutive
// units, and every tile gets a warp of its own: many small CTAs that the hardware schedules as
// earlier ones retire, which keeps the loads of new CTAs overlapped with the arithmetic and stores
// of older ones (a persistent wave with a stride loop measured 10-20 % slower on these streams).
//
//   quantize / fake_quant : unit = 32 B of FP32/BF16 input (8 / 16 elements); a block of 32
//                           elements spans 4 / 2 adjacent lanes, whose maxima meet by xor-shuffles.
//   slice_scale           : unit = 32 element codes = one block per lane, no cross-lane traffic.
//   dequantize            : to 16-bit outputs a unit is 32 element codes (64 B out); to FP32 it is 32 B
//                           of output (8 elements), see dequantize_wide_kernel.
//
// Every kernel lets its successor start launching at once, asks L2 for its own input lines, and only
// then waits for its predecessor (see pdl_release / prefetch_tile / pdl_acquire in mxq_access.cuh).
//
// All of them are bound by HBM traffic, with the integer/logic pipe (64 lanes per clock per SM) as
// the second bound; the arithmetic below is shaped to stay under it: packed 16-bit maxima, round-down
// FP32 adds instead of float->int conversions, four 8-bit codes per register (SWAR), per-byte signs
// by byte permutes and one multiply, the sm_100a narrowing conversion instructions for MXFP.
#pragma once
#include <cstdint>
#include <type_traits>
#include <utility>
#include <cuda_runtime.h>

#include "mxq_access.cuh"
#include "mxq_codec.cuh"

namespace mxq {


template <int N, class Fn>
__device__ __forceinline__ void static_for(Fn&& fn)
{
    [&]<int... I>(std::integer_sequence<int, I...>) { (fn(std::integral_constant<int, I>{}), ...); }
    (std::make_integer_sequence<int, N>{});
}

// ------------------------------------------------------------------------------------------
// Where a block's scale byte goes
// ------------------------------------------------------------------------------------------
// The kernels that produce scale bytes write them through put_scale(), overloaded on the type of
// the destination: a plain pointer (byte of block i at scales[i], the library's stored form), or a
// TiledScales record, which places them in the 128-row x 4-column tiles a block-scaled tensor-core
// matrix multiply reads (the step that consumes W_t, Sec. 3.5): tile (r / 128, c / 4) is 512
// consecutive bytes and holds the byte of row r, block-column c at
// (r mod 32) * 16 + (r div 32 mod 4) * 4 + c mod 4.

__device__ __forceinline__ void put_scale(uint8_t* scales, size_t blk, uint32_t byte)
{
    st_u8(scales + blk, byte);
}

// Division of a 32-bit block index by the row length in blocks, by multiply and shift (the
// round-up method for an invariant divisor: with s = ceil(log2 d) and m = floor(2^32 (2^s - d) / d) + 1,
// n / d = (t + ((n - t) >> min(s, 1))) >> max(s - 1, 0) where t is the high word of m * n).  The host
// fills in m and the two shifts (see make_tiled_scales in mxq_launch.h).
struct TiledScales {
    uint8_t* base;
    uint32_t kblocks;      // block-columns per row (the divisor)
    uint32_t magic, shift1, shift2;
    uint32_t col_tiles;    // ceil(kblocks / 4)
};

inline TiledScales make_tiled_scales(uint8_t* base, uint32_t kblocks)      // 1 <= kblocks <= 2^31
{
    uint32_t s = 0;
    while ((1ull << s) < kblocks) ++s;
    const uint64_t m = ((1ull << 32) * ((1ull << s) - kblocks)) / kblocks + 1;
    return TiledScales{base, kblocks, (uint32_t)m, s < 1 ? s : 1u, s > 1 ? s - 1 : 0u, (kblocks + 3) / 4};
}

// Byte offset of block `blk` (row-major index, below 2^32) inside the tiled buffer.
__host__ __device__ __forceinline__ size_t tiled_scale_offset(const TiledScales& t, size_t blk)
{
    const uint32_t n = (uint32_t)blk;
#ifdef __CUDA_ARCH__
    const uint32_t hi = __umulhi(t.magic, n);
#else
    const uint32_t hi = (uint32_t)(((uint64_t)t.magic * n) >> 32);
#endif
    const uint32_t r = (hi + ((n - hi) >> t.shift1)) >> t.shift2;
    const uint32_t c = n - r * t.kblocks;
    const size_t tile = (size_t)(r >> 7) * t.col_tiles + (c >> 2);
    return tile * 512 + (r & 31u) * 16u + ((r >> 5) & 3u) * 4u + (c & 3u);
}

__device__ __forceinline__ void put_scale(const TiledScales& t, size_t blk, uint32_t byte)
{
    st_u8(t.base + tiled_scale_offset(t, blk), byte);
}

// ------------------------------------------------------------------------------------------
// Source element types
// ------------------------------------------------------------------------------------------

struct F32 {
    static constexpr int id = MXQ_F32;
    static constexpr int size = 4;
    static constexpr int epl = 8;     // elements per 32-byte lane unit
};
struct BF16 {
    static constexpr int id = MXQ_BF16;
    static constexpr int size = 2;
    static constexpr int epl = 16;
};

// Element i of a lane unit as FP32 (exact widening for BF16).
template <class T, int I>
__device__ __forceinline__ float unit_elem(const uint32_t (&w)[8])
{
    if constexpr (T::size == 4) return __uint_as_float(w[I]);
    else return __uint_as_float((I & 1) ? (w[I >> 1] & 0xFFFF0000u) : (w[I >> 1] << 16));
}

__device__ __forceinline__ float max3_abs_nan(float a, float b, float c)
{
    float d;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(fabsf(a)), "f"(fabsf(b)), "f"(fabsf(c)));
    return d;
}

// FP32 bit pattern of max |element| over the lane unit; any NaN yields a NaN pattern, an
// infinity the infinity pattern (both >= 0x7F800000, both larger than every finite pattern).
template <class T>
__device__ __forceinline__ uint32_t unit_amax_bits(const uint32_t (&w)[8])
{
    if constexpr (T::size == 4) {
        float m0 = max3_abs_nan(__uint_as_float(w[0]), __uint_as_float(w[1]), __uint_as_float(w[2]));
        float m1 = max3_abs_nan(__uint_as_float(w[3]), __uint_as_float(w[4]), __uint_as_float(w[5]));
        float m2 = max3_abs_nan(__uint_as_float(w[6]), __uint_as_float(w[7]), m0);
        float m;
        asm("max.NaN.f32 %0, %1, %2;" : "=f"(m) : "f"(m1), "f"(m2));
        return __float_as_uint(m) & 0x7FFFFFFFu;
    } else {
        // BF16 magnitudes are ordered like their 15-bit patterns: packed 16-bit integer maxima.
        constexpr uint32_t kAbs = 0x7FFF7FFFu;
        uint32_t a = __vimax3_s16x2(w[0] & kAbs, w[1] & kAbs, w[2] & kAbs);
        uint32_t b = __vimax3_s16x2(w[3] & kAbs, w[4] & kAbs, w[5] & kAbs);
        uint32_t c = __vimax3_s16x2(w[6] & kAbs, w[7] & kAbs, a);
        uint32_t m = __vmaxu2(b, c);
        return max(m << 16, m & 0xFFFF0000u);
    }
}

template <int LPB>
__device__ __forceinline__ uint32_t group_max(uint32_t v)
{
#pragma unroll
    for (int o = 1; o < LPB; o <<= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// ------------------------------------------------------------------------------------------
// Q_f: quantize (Eq. 1-3)
// ------------------------------------------------------------------------------------------

// Four 6-bit codes, one per byte, -> the 24-bit stream c0 | c1 << 6 | c2 << 12 | c3 << 18 in bits
// 31..8 of the result (bits 7..0 clear).  Every field only ever moves LEFT relative to c3, so the
// moves are multiply-adds (the multiply pipe) instead of shifts and selects on the logic pipe:
// with the codes in bits 7..2 of their bytes, w + 3 (w & 0x00FF00FF) multiplies bytes 0 and 2 by 4,
// which joins each byte pair into a 12-bit field (bits 15..4 and 31..20); y + 15 (y & 0xFFFF) then
// multiplies the low field by 16, which joins the two.
__device__ __forceinline__ uint32_t squeeze6_top(uint32_t w)           // codes in bits 7..2, bits 1..0 clear
{
    const uint32_t y = (w & 0x00FF00FFu) * 3u + w;
    return (y & 0x0000FFFFu) * 15u + y;
}

__device__ __forceinline__ uint32_t squeeze6_low(uint32_t w)           // codes in bits 5..0, bits 7..6 clear
{
    const uint32_t y = (w & 0x00FF00FFu) * 12u + w * 4u;
    return (y & 0x0000FFFFu) * 15u + y;
}

// Four such streams (each in bits 31..8 of its word) -> three 32-bit words: whole bytes, so three
// byte permutes.
__device__ __forceinline__ void join24(uint32_t z0, uint32_t z1, uint32_t z2, uint32_t z3, uint32_t& o0, uint32_t& o1,
                                       uint32_t& o2)
{
    o0 = __byte_perm(z0, z1, 0x5321);
    o1 = __byte_perm(z1, z2, 0x6532);
    o2 = __byte_perm(z2, z3, 0x7653);
}

// Four B-bit codes, one per byte with the upper bits clear, -> one 4B-bit value (c0 | c1 << B | ...).
// Two shift-and-select steps: bytes to 2B-bit fields in the 16-bit halves, halves to one field.
// Whatever a shift drags along falls where the next select takes the other operand.
template <int B>
__device__ __forceinline__ uint32_t squeeze_bytes(uint32_t x)
{
    static_assert(B >= 1 && B <= 7, "codes narrower than a byte");
    constexpr uint32_t kEven = ((1u << B) - 1u) * 0x00010001u;           // the fields of bytes 0 and 2
    constexpr uint32_t kLow = (1u << (2 * B)) - 1u;
    const uint32_t y = (x & kEven) | ((x >> (8 - B)) & ~kEven);
    return (y & kLow) | ((y >> (16 - 2 * B)) & ~kLow);
}

// NZ words holding four clean B-bit codes each (one per byte) -> the little-endian bitstream.
template <int B, int NZ, int NW>
__device__ __forceinline__ void pack_code_bytes(const uint32_t (&z)[NZ], uint32_t (&out)[NW])
{
    constexpr int W = 4 * B;                                             // bits per squeezed word
    static_assert(NW * 32 >= NZ * W, "output too small");
    static_for<NZ>([&](auto j) {
        constexpr int J = decltype(j)::value;
        constexpr int off = J * W, wi = off >> 5, sh = off & 31;
        const uint32_t q = squeeze_bytes<B>(z[J]);
        if constexpr (sh == 0) out[wi] = q;
        else out[wi] |= q << sh;
        if constexpr (sh + W > 32) out[wi + 1] = q >> (32 - sh);
    });
}

// MXINT codes of four consecutive elements (Eq. 3), one per byte in the low F::bits bits.
//   v0..v3 : the raw elements, inv = 2^-shared_exp (|v| inv < 2^(bits-1), exact)
//   full   : 0xFF in the bytes whose element is negative, 0x00 elsewhere
// One round-down FFMA per element adds 2^15 + 0.5, where the FP32 spacing is 2^-8: byte 1 of the
// sum is floor(|r| + 0.5), the magnitude rounded to nearest with ties away from zero.  Three byte
// permutes gather the four magnitudes; clip and sign are then applied to all four at once.
template <class F>
__device__ __forceinline__ uint32_t quantize_int_quad(float v0, float v1, float v2, float v3, float inv, uint32_t full)
{
    constexpr float kMagic = 32768.5f;
    constexpr uint32_t k01 = 0x01010101u;
    constexpr uint32_t kInv255 = 0xFEFEFEFFu;                  // 255^-1 mod 2^32: mask -> 0/1 per byte
    constexpr uint32_t kMask = k01 * F::mask;
    const uint32_t y0 = __float_as_uint(__fmaf_rd(fabsf(v0), inv, kMagic));
    const uint32_t y1 = __float_as_uint(__fmaf_rd(fabsf(v1), inv, kMagic));
    const uint32_t y2 = __float_as_uint(__fmaf_rd(fabsf(v2), inv, kMagic));
    const uint32_t y3 = __float_as_uint(__fmaf_rd(fabsf(v3), inv, kMagic));
    uint32_t q = __byte_perm(__byte_perm(y0, y1, 0x0051), __byte_perm(y2, y3, 0x0051), 0x5410);
    q -= (q >> (F::bits - 1)) & k01;                           // 2^(b-1) -> 2^(b-1) - 1 (symmetric clip)
    if constexpr (F::bits == 8) {
        // negate in 7 bits, then set the sign bit: no carry leaves a byte even for a negative zero
        const uint32_t z = (q ^ (full & 0x7F7F7F7Fu)) + full * kInv255;
        return z ^ (full & 0x80808080u);
    } else {
        return ((q ^ (full & kMask)) + full * kInv255) & kMask;
    }
}

// 0xFF / 0x00 per byte: the signs of elements 4Q .. 4Q+3 of a lane unit, straight from the raw words.
template <class T, int Q>
__device__ __forceinline__ uint32_t unit_sign_bytes(const uint32_t (&w)[8])
{
    uint32_t full;
    if constexpr (T::size == 2) {
        // two BF16 per word: sign bits sit at the top of bytes 1 and 3 (selector bit 3 replicates it)
        asm("prmt.b32 %0, %1, %2, 0xFDB9;" : "=r"(full) : "r"(w[2 * Q]), "r"(w[2 * Q + 1]));
    } else {
        uint32_t a, b;
        asm("prmt.b32 %0, %1, %2, 0x00FB;" : "=r"(a) : "r"(w[4 * Q]), "r"(w[4 * Q + 1]));
        asm("prmt.b32 %0, %1, %2, 0x00FB;" : "=r"(b) : "r"(w[4 * Q + 2]), "r"(w[4 * Q + 3]));
        full = __byte_perm(a, b, 0x5410);
    }
    return full;
}

// Codes of one lane unit, packed as a little-endian bitstream.
template <class T, class F, int NW>
__device__ __forceinline__ void quantize_unit(const uint32_t (&w)[8], float inv, uint32_t (&out)[NW])
{
    if constexpr (F::kind == KIND_INT) {
        constexpr int NQ = T::epl / 4;
        uint32_t z[NQ];
        static_for<NQ>([&](auto qi) {
            constexpr int Q = decltype(qi)::value;
            z[Q] = quantize_int_quad<F>(unit_elem<T, 4 * Q>(w), unit_elem<T, 4 * Q + 1>(w), unit_elem<T, 4 * Q + 2>(w),
                                        unit_elem<T, 4 * Q + 3>(w), inv, unit_sign_bytes<T, Q>(w));
        });
        if constexpr (F::bits == 8) {
#pragma unroll
            for (int j = 0; j < NQ; ++j) out[j] = z[j];
        } else if constexpr (F::bits == 4) {
            // c0 | c1 << 4 lands in byte 0 and c2 | c3 << 4 in byte 2 of z | z >> 4
#pragma unroll
            for (int j = 0; j < NQ / 2; ++j)
                out[j] = __byte_perm(z[2 * j] | (z[2 * j] >> 4), z[2 * j + 1] | (z[2 * j + 1] >> 4), 0x6420);
        } else if constexpr (F::bits == 6 && NQ % 4 == 0) {
#pragma unroll
            for (int g = 0; g < NQ / 4; ++g) {
                const uint32_t s0 = squeeze6_low(z[4 * g]), s1 = squeeze6_low(z[4 * g + 1]), s2 = squeeze6_low(z[4 * g + 2]),
                               s3 = squeeze6_low(z[4 * g + 3]);
                join24(s0, s1, s2, s3, out[3 * g + 0], out[3 * g + 1], out[3 * g + 2]);
            }
        } else {
            pack_code_bytes<F::bits>(z, out);
        }
    } else if constexpr (!F::hw_cvt) {
        // E3M3 / E2M2: four elements at a time through the hardware neighbour format
        constexpr int NQ = T::epl / 4;
        uint32_t z[NQ];
        const float inv_k = inv * SoftFp<F>::pre_scale;          // exact: both are powers of two
        static_for<NQ>([&](auto qi) {
            constexpr int Q = decltype(qi)::value;
            z[Q] = quantize_fp_soft_quad<F>(unit_elem<T, 4 * Q>(w) * inv_k, unit_elem<T, 4 * Q + 1>(w) * inv_k,
                                            unit_elem<T, 4 * Q + 2>(w) * inv_k, unit_elem<T, 4 * Q + 3>(w) * inv_k);
        });
        pack_code_bytes<F::bits>(z, out);
    } else {
        static_for<T::epl / 2>([&](auto i) {
            constexpr int I = decltype(i)::value;
            uint2 c = quantize_pair<F>(unit_elem<T, 2 * I>(w), unit_elem<T, 2 * I + 1>(w), inv);
            if constexpr (F::bits == 8) {
                // two bytes at a time
                constexpr int wi = I / 2, sh = (I & 1) * 16;
                uint32_t pair = c.x | (c.y << 8);
                if constexpr (sh == 0) out[wi] = pair;
                else out[wi] |= pair << 16;
            } else {
                put_code<F::bits, 2 * I>(out, c.x);
                put_code<F::bits, 2 * I + 1>(out, c.y);
            }
        });
    }
}

// One warp tile (32 U lane units) of one tensor; shared by the single-tensor and the batched kernels.
// Every lane of the warp must call it (the block maxima meet by shuffles).
template <class T, class F, int BLOCK, int U, class SCALES>
__device__ __forceinline__ void quantize_tile(const uint8_t* __restrict__ src, size_t nunits, uint8_t* __restrict__ codes,
                                              const SCALES& scales, size_t tile, uint8_t* stage)
{
    constexpr int LPB = BLOCK / T::epl;                 // lanes per block
    static_assert(LPB >= 1 && LPB <= 32, "block must cover at least one lane unit");
    constexpr int OB = T::epl * F::bits / 8;            // code bytes per lane unit
    constexpr int NW = code_words(T::epl, F::bits);
    const int lane = threadIdx.x & 31;
    const size_t u0 = tile * (32 * U) + lane;
    uint32_t w[U][8];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) ld256(w[u], src + unit * 32);
        else {
#pragma unroll
            for (int j = 0; j < 8; ++j) w[u][j] = 0;
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        const uint32_t amax = group_max<LPB>(unit_amax_bits<T>(w[u]));
        const BlockScale s = block_scale<F>(amax);
        uint32_t out[NW];
        quantize_unit<T, F>(w[u], s.inv, out);
        if (s.byte == 0xFFu) {
#pragma unroll
            for (int j = 0; j < NW; ++j) out[j] = 0;
        }
        if constexpr (StagedTile<OB>::use) store_bytes<OB>(stage + (u * 32 + lane) * OB, out);
        if (unit < nunits) {
            if constexpr (!StagedTile<OB>::use) store_bytes<OB>(codes + unit * OB, out);
            if (lane % LPB == 0) put_scale(scales, unit / LPB, s.byte);
        }
    }
    if constexpr (StagedTile<OB>::use) {
        const size_t first = tile * (32 * U), left = nunits - first;
        flush_stage<32 * U * OB>(stage, codes + first * OB, (uint32_t)(left < 32 * U ? left : 32 * U) * OB);
    }
}

// The staging area of the calling warp for a quantize tile (null when a lane's code piece is stored
// directly).  Must be called by every thread of the CTA, outside divergent code.
template <class T, class F, int U, int THREADS>
__device__ __forceinline__ uint8_t* quantize_stage()
{
    constexpr int OB = T::epl * F::bits / 8;
    if constexpr (StagedTile<OB>::use) {
        __shared__ __align__(128) uint8_t stage_area[(THREADS / 32) * 32 * U * OB];
        return stage_area + (threadIdx.x >> 5) * (32 * U * OB);
    } else {
        return nullptr;
    }
}

// (Compiled for 16 resident CTAs of 128 threads, i.e. 32 registers: against the compiler's own choice the MXINT and
// 6-bit quantizers are 2 - 4 % faster at 2^26 elements, the others unchanged.)
template <class T, class F, int BLOCK, int U, int THREADS, class SCALES = uint8_t*>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS)
quantize_kernel(const uint8_t* __restrict__ src, size_t nunits, uint8_t* __restrict__ codes, SCALES scales)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t* stage = quantize_stage<T, F, U, THREADS>();
    prefetch_tile<U, 32>(src, tile, nunits);
    pdl_acquire();
    if (tile * (32 * U) < nunits) quantize_tile<T, F, BLOCK, U>(src, nunits, codes, scales, tile, stage);
}

// ------------------------------------------------------------------------------------------
// Fused fake-quant forward (Eq. 6 in reconstructed form)
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ float fma_keep_plus_zero(float a, float b)
{
    // a * b + (+0): turns a -0 product into +0 and changes nothing else
    float d;
    asm("fma.rn.f32 %0, %1, %2, 0f00000000;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// two FP32 values out of a packed narrow-float pair produced by quantize_fp_hw_pair
template <class F>
__device__ __forceinline__ float2 widen_hw_pair(uint32_t d)
{
    uint32_t h2;
    if constexpr (F::id == MXQ_FP8_E4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)d));
    else if constexpr (F::id == MXQ_FP6_E3M2) asm("cvt.rn.f16x2.e3m2x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)d));
    else if constexpr (F::id == MXQ_FP6_E2M3) asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)d));
    else asm("{ .reg .b8 t; cvt.u8.u32 t, %1; cvt.rn.f16x2.e2m1x2 %0, t; }" : "=r"(h2) : "r"(d));
    float2 f;
    asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, h; }"
        : "=f"(f.x), "=f"(f.y) : "r"(h2));
    return f;
}

// Element-format value (the real number P) of two inputs after quantization, as FP32.
//   DIRECT     : P = quantize_F(v inv)                       (inv = 2^-shared_exp of F)
//   VIA_ANCHOR : P = Q_{A->F}(quantize_A(v inv))             (inv = 2^-shared_exp of the anchor A)
template <class F, int MODE>
__device__ __forceinline__ float2 fake_quant_pair(float v0, float v1, float inv)
{
    using A = Fmt<F::kind == KIND_INT ? MXQ_INT8 : MXQ_FP8_E4M3>;
    constexpr bool via = MODE == MXQ_FQ_VIA_ANCHOR && F::id != A::id;
    constexpr int de = A::emax - F::emax;
    float2 p;
    if constexpr (F::kind == KIND_INT) {
        // floor(x + 0.5) for 0 <= x < 2^22 on the FP32 pipes alone: a round-down add of 2^22 + 0.5 lands
        // on the 0.5 grid of [2^22, 2^23), a round-down add of another 2^22 on the integer grid of
        // [2^23, 2^24).  The value stays biased by 2^23 until the clip.
        auto one = [&](float v) {
            float y = __fmaf_rd(fabsf(v), inv, 4194304.5f);                            // 2^22 + h, h = |r| + 0.5 on the 0.5 grid
            if constexpr (via) {
                // Eq. 4 on the anchor magnitude q8 = floor(h): floor(q8 / 2^de + 0.5) = floor(h / 2^de + 0.5),
                // since flooring before a division by an integer changes nothing.  So the anchor's integer
                // step is skipped: one more round-down multiply-add onto the 0.5 grid.
                // (Clipping q8 to 127 first would change nothing either: 127 and 128 both end in the clipped bin.)
                constexpr float kScale = 1.0f / (float)(1 << de);
                constexpr float kBias = 4194304.5f - 4194304.0f / (float)(1 << de);    // exact in FP32
                y = __fmaf_rd(y, kScale, kBias);
            }
            float z = __fadd_rd(y, 4194304.0f);                                        // 2^23 + floor(.)
            z = fminf(z, 8388608.0f + (float)F::max_mag);                              // symmetric clip
            const float qf = z - 8388608.0f;                                           // exact small integer
            return __uint_as_float(__float_as_uint(qf) | (__float_as_uint(v) & 0x80000000u));
        };
        p.x = one(v0);
        p.y = one(v1);
    } else {
        // E3M3 / E2M2 are quantized as 2^-k times the value in their hardware neighbour format (see SoftFp)
        constexpr int k = [] { if constexpr (F::hw_cvt) return 0; else return SoftFp<F>::k; }();
        float r0, r1;
        if constexpr (via) {
            // anchor codes -> exact FP16 values -> divide by 2^(de + k) (exact) -> FP32
            uint32_t a = quantize_fp_hw_pair<A>(v0 * inv, v1 * inv);
            uint32_t h2;
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)a));
            constexpr uint32_t kHalf = (uint32_t)(15 - de - k) << 10;          // 2^-(de + k) as FP16
            asm("mul.rn.f16x2 %0, %0, %1;" : "+r"(h2) : "r"(kHalf | (kHalf << 16)));
            asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, h; }"
                : "=f"(r0), "=f"(r1) : "r"(h2));
        } else {
            const float inv_k = inv * __uint_as_float((uint32_t)(127 - k) << 23);  // exact: powers of two
            r0 = v0 * inv_k;
            r1 = v1 * inv_k;
        }
        if constexpr (F::hw_cvt) {
            p = widen_hw_pair<F>(quantize_fp_hw_pair<F>(r0, r1));
        } else {
            p = widen_hw_pair<Fmt<SoftFp<F>::hw>>(quantize_fp_soft_pair<F>(r0, r1));
            p.x *= SoftFp<F>::post_scale;
            p.y *= SoftFp<F>::post_scale;
        }
    }
    return p;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// One warp tile (32 U lane units) of one tensor; shared by the single-tensor and the batched kernels.
// Every lane of the warp must call it (the block maxima meet by shuffles).
template <class T, class F, int BLOCK, int MODE, int U>
__device__ __forceinline__ void fake_quant_tile(const uint8_t* src, size_t nunits, uint8_t* dst, size_t tile)
{
    using A = Fmt<F::kind == KIND_INT ? MXQ_INT8 : MXQ_FP8_E4M3>;
    constexpr bool via = MODE == MXQ_FQ_VIA_ANCHOR && F::id != A::id;
    using S = std::conditional_t<via, A, F>;            // the format whose scale Eq. 1 computes
    constexpr int de = A::emax - F::emax;
    constexpr int LPB = BLOCK / T::epl;
    static_assert(LPB >= 1 && LPB <= 32, "block must cover at least one lane unit");
    const size_t u0 = tile * (32 * U) + (threadIdx.x & 31);
    uint32_t w[U][8];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) ld256(w[u], src + unit * 32);
        else {
#pragma unroll
            for (int j = 0; j < 8; ++j) w[u][j] = 0;
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        const uint32_t amax = group_max<LPB>(unit_amax_bits<T>(w[u]));
        const BlockScale s = block_scale<S>(amax);
        // X of the target format: the anchor's byte moved up by de, saturating (Eq. 4-5)
        const uint32_t byte = via ? min(s.byte + (uint32_t)de, 254u) : s.byte;
        const float X = scale_value(byte);
        uint32_t out[8];
        static_for<T::epl / 2>([&](auto i) {
            constexpr int I = decltype(i)::value;
            const float v0 = unit_elem<T, 2 * I>(w[u]), v1 = unit_elem<T, 2 * I + 1>(w[u]);
            float2 p = fake_quant_pair<F, MODE>(v0, v1, s.inv);
            float y0, y1;
            if constexpr (F::kind == KIND_INT) {          // MXINT zero reconstructs to +0
                y0 = fma_keep_plus_zero(p.x, X);
                y1 = fma_keep_plus_zero(p.y, X);
            } else {
                y0 = p.x * X;
                y1 = p.y * X;
            }
            if constexpr (T::size == 4) {
                out[2 * I] = __float_as_uint(y0);
                out[2 * I + 1] = __float_as_uint(y1);
            } else {
                out[I] = pack_bf16x2(y0, y1);
            }
        });
        if (unit < nunits) {
            if (s.byte == 0xFFu) st256_splat(dst + unit * 32, T::size == 4 ? 0x7FC00000u : 0x7FC07FC0u);   // poisoned block
            else st256(dst + unit * 32, out);
        }
    }
}

template <class T, class F, int BLOCK, int MODE, int U, int THREADS>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS)
fake_quant_kernel(const uint8_t* src, size_t nunits, uint8_t* dst)   // dst may equal src
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    prefetch_tile<U, 32>(src, tile, nunits);
    pdl_acquire();
    if (tile * (32 * U) < nunits) fake_quant_tile<T, F, BLOCK, MODE, U>(src, nunits, dst, tile);
}

// Which tensor of a batch owns a tile.  The batched kernels lay the tiles of all tensors end to end;
// the items (sorted by tile_begin) ride in the kernel parameters.  A plain binary search over a few
// hundred items costs eight dependent constant-memory reads and some fifty instructions per warp
// tile, 10 - 20 % of such a kernel.  The host therefore adds a coarse index: the tile space is cut
// into at most 256 segments of 2^shift tiles, coarse[k] is the item that owns the first tile of
// segment k (coarse[last + 1] the last item), and a tile's owner lies between the entries of its
// segment's two ends -- usually the same item or neighbours, so the search that remains takes zero
// to two steps.
struct TileIndex {
    uint32_t shift;
    uint16_t coarse[258];
};

template <class ITEM>
inline void build_tile_index(TileIndex& ix, const ITEM* items, int count, size_t total_tiles)
{
    ix.shift = 0;
    while ((total_tiles >> ix.shift) > 255) ++ix.shift;
    const size_t nseg = total_tiles ? ((total_tiles - 1) >> ix.shift) + 1 : 1;
    int it = 0;
    for (size_t k = 0; k < nseg; ++k) {
        const size_t first = k << ix.shift;
        while (it + 1 < count && items[it + 1].tile_begin <= first) ++it;
        ix.coarse[k] = (uint16_t)it;
    }
    for (size_t k = nseg; k < 258; ++k) ix.coarse[k] = (uint16_t)(count - 1);
}

// `items` is an array inside a __grid_constant__ kernel parameter; tile < total_tiles.
template <class ITEM>
__host__ __device__ __forceinline__ int find_item(const ITEM* items, const TileIndex& ix, size_t tile)
{
    const uint32_t k = (uint32_t)(tile >> ix.shift);
    int lo = ix.coarse[k], hi = ix.coarse[k + 1];
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (items[mid].tile_begin <= tile) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

// The fake-quant of a whole set of tensors (every quantized weight of a model in one QAT step, Eq. 6)
// in one launch: the tiles of all tensors laid end to end, the item table in the kernel's parameters.
struct FqDeviceItem {
    const uint8_t* src;
    uint8_t* dst;
    size_t nunits;
    size_t tile_begin;     // first global tile index of this tensor
};

template <int K>
struct FqItemBlock {
    FqDeviceItem items[K];
    TileIndex index;
};

template <class T, class F, int BLOCK, int MODE, int U, int R, int THREADS, int K>
__global__ void __launch_bounds__(THREADS, 14)
fake_quant_batched_kernel(const __grid_constant__ FqItemBlock<K> blk, int count, size_t total_tiles)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    // the item table is a kernel parameter, so the lookup may run before the dependency wait
    const FqDeviceItem& t = blk.items[tile < total_tiles ? find_item(blk.items, blk.index, tile) : 0];
    // A tile of the batch is R consecutive warp tiles of ONE tensor, converted one after the other: the
    // lookup above (some 25 instructions per thread) is paid once per R * 32 * U lane units.
    const size_t first = (tile - t.tile_begin) * R;
    if (tile < total_tiles) {
#pragma unroll
        for (int r = 0; r < R; ++r) prefetch_tile<U, 32>(t.src, first + r, t.nunits);
    }
    pdl_acquire();
    if (tile >= total_tiles) return;                      // whole warps leave together
#pragma unroll 1
    for (int r = 0; r < R; ++r)
        if ((first + r) * (32 * U) < t.nunits) fake_quant_tile<T, F, BLOCK, MODE, U>(t.src, t.nunits, t.dst, first + r);
}

// Q_f (Eq. 1-3) over a whole set of tensors in one launch (the anchor checkpoint of a model, Sec. 3.5:
// every linear weight quantized once and stored): tiles of all tensors end to end, items in the parameters.
struct QDeviceItem {
    const uint8_t* src;
    uint8_t* codes;
    uint8_t* scales;
    size_t nunits;
    size_t tile_begin;
};

template <int K>
struct QItemBlock {
    QDeviceItem items[K];
    TileIndex index;
};

template <class T, class F, int BLOCK, int U, int THREADS, int K>
__global__ void __launch_bounds__(THREADS, 14)     // 14 resident CTAs: the MXINT8 anchor of the 224-tensor set 3.01 ms against 3.30
quantize_batched_kernel(const __grid_constant__ QItemBlock<K> blk, int count, size_t total_tiles)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t* stage = quantize_stage<T, F, U, THREADS>();
    const QDeviceItem& t = blk.items[tile < total_tiles ? find_item(blk.items, blk.index, tile) : 0];
    if (tile < total_tiles) prefetch_tile<U, 32>(t.src, tile - t.tile_begin, t.nunits);
    pdl_acquire();
    if (tile >= total_tiles) return;                      // whole warps leave together
    quantize_tile<T, F, BLOCK, U>(t.src, t.nunits, t.codes, t.scales, tile - t.tile_begin, stage);
}

// ------------------------------------------------------------------------------------------
// Q_{h->l}: Slice-and-Scale (Eq. 4-5).  One lane = 32 codes.
// ------------------------------------------------------------------------------------------

// Eq. 4 on four MXINT8 codes at once (one per byte): returns the four low-format codes, one per
// byte, in the TOP BL bits of the byte (the bits below are clear).  Sign-magnitude SWAR; no carry
// crosses a byte until the last step, whose stray carry lands in a bit that is masked off.
//   full : 0xFF in the bytes that are negative (byte permute with sign replication)
//   a    : |p| - s per byte, s the 0/1 sign (one's complement of the negative bytes)
//   T    : |p| + 2^(de-1) <= 128 + 2^(de-1); the shifted value q = T >> de sits in T's top BL bits.
//          q reaches 2^(BL-1) exactly when T >= 128, and then those top bits read 100..0: flipping
//          them (xor with the replicated top bit of T) gives 011..1, the clipped magnitude.
//   two's complement of the negative bytes: flip the BL bits, add one at bit de.  The add can carry
//   out of a byte only for q = 0 (the bits are all ones), into bit 0 of the next byte, which is
//   cleared before (so that it cannot travel) and after.
// The integer/logic pipe is the scarce resource here, so the per-byte 0/1 sign comes from the
// 0xFF/0x00 mask by a multiply-add with 255^-1 (mod 2^32), which runs on the multiply pipe:
// mask = 255 * sum(s_i 256^i), hence mask * 255^-1 = sum(s_i 256^i) exactly.
// (Checked against the scalar definition for all 2^32 input words on the host.)
template <int BL>
__device__ __forceinline__ uint32_t ss_int8_word_top(uint32_t x)
{
    constexpr int de = 8 - BL;
    constexpr uint32_t k01 = 0x01010101u;
    constexpr uint32_t kInv255 = 0xFEFEFEFFu;
    constexpr uint32_t kH = k01 * (1u << (de - 1));            // rounding increment
    constexpr uint32_t kTop = k01 * ((0xFFu << de) & 0xFFu);   // the top BL bits of every byte
    uint32_t full, ov;
    asm("prmt.b32 %0, %1, %1, 0xBA98;" : "=r"(full) : "r"(x)); // selector bit 3: replicate the byte's sign
    const uint32_t a = x ^ full;
    const uint32_t t = a + (full * kInv255 + kH);
    asm("prmt.b32 %0, %1, %1, 0xBA98;" : "=r"(ov) : "r"(t));   // 0xFF where the magnitude clips
    const uint32_t m = (t ^ ov ^ full) & kTop;
    return (full * (kInv255 << de) + m) & kTop;
}

// The same four codes in the low BL bits of their bytes.
template <int BL>
__device__ __forceinline__ uint32_t ss_int8_word(uint32_t x)
{
    return ss_int8_word_top<BL>(x) >> (8 - BL);
}

__device__ __forceinline__ bool has_e4m3_nan(uint32_t x)
{
    return (((x & 0x7F7F7F7Fu) + 0x01010101u) & 0x80808080u) != 0;
}

// Eq. 5 on E4M3 codes through the conversion instructions: exact widening to FP16, exact division
// by 2^de, FP32, narrowing cvt (nearest even, saturating).  Register halves and bytes are split and
// joined with mov so that no shift or mask is spent on them.

// four E4M3 codes of one word as two FP16 pairs (exact).  Kept apart from the scaling so that two
// targets converted from the same word share it.
__device__ __forceinline__ void e4m3_word_to_f16(uint32_t w, uint32_t& a, uint32_t& b)
{
    asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; cvt.rn.f16x2.e4m3x2 %0, l; cvt.rn.f16x2.e4m3x2 %1, h; }"
        : "=r"(a), "=r"(b) : "r"(w));
}

// two FP16 pairs (four E4M3 codes of one word), already divided by 2^de, as four FP32 values
template <int DE>
__device__ __forceinline__ void e4m3_word_scaled(uint32_t w, float (&f)[4])
{
    constexpr uint32_t kHalf = (uint32_t)(15 - DE) << 10;      // 2^-de as FP16
    uint32_t a, b;
    e4m3_word_to_f16(w, a, b);
    asm("{ .reg .b16 l, h; .reg .b32 a, b;\n"
        "  mul.rn.f16x2 a, %4, %6;  mul.rn.f16x2 b, %5, %6;\n"
        "  mov.b32 {l, h}, a;  cvt.f32.f16 %0, l;  cvt.f32.f16 %1, h;\n"
        "  mov.b32 {l, h}, b;  cvt.f32.f16 %2, l;  cvt.f32.f16 %3, h; }"
        : "=f"(f[0]), "=f"(f[1]), "=f"(f[2]), "=f"(f[3]) : "r"(a), "r"(b), "r"(kHalf | (kHalf << 16)));
}

// four E4M3 codes (one word) -> four 6-bit codes, one per byte
template <class FL>
__device__ __forceinline__ uint32_t ss_e4m3_word_to6(uint32_t w)
{
    static_assert(FL::bits == 6 && FL::hw_cvt, "6-bit target with a narrowing cvt");
    float f[4];
    e4m3_word_scaled<8 - FL::emax>(w, f);
    uint32_t d;
    if constexpr (FL::id == MXQ_FP6_E2M3)
        asm("{ .reg .b16 l, h; cvt.rn.satfinite.e2m3x2.f32 l, %2, %1; cvt.rn.satfinite.e2m3x2.f32 h, %4, %3; mov.b32 %0, {l, h}; }"
            : "=r"(d) : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]));
    else
        asm("{ .reg .b16 l, h; cvt.rn.satfinite.e3m2x2.f32 l, %2, %1; cvt.rn.satfinite.e3m2x2.f32 h, %4, %3; mov.b32 %0, {l, h}; }"
            : "=r"(d) : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]));
    return d;
}

// eight E4M3 codes (two words) -> eight E2M1 codes in one word
__device__ __forceinline__ uint32_t ss_e4m3_words_to_e2m1(uint32_t w0, uint32_t w1)
{
    float f[4], g[4];
    e4m3_word_scaled<6>(w0, f);
    e4m3_word_scaled<6>(w1, g);
    uint32_t d;
    asm("{ .reg .b8 a, b, c, e;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 a, %2, %1;  cvt.rn.satfinite.e2m1x2.f32 b, %4, %3;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 c, %6, %5;  cvt.rn.satfinite.e2m1x2.f32 e, %8, %7;\n"
        "  mov.b32 %0, {a, b, c, e}; }"
        : "=r"(d) : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "f"(g[0]), "f"(g[1]), "f"(g[2]), "f"(g[3]));
    return d;
}

// Eq. 5 for the two MXFP targets without a narrowing instruction, E3M3 (7 bits, de = 4) and E2M2
// (5 bits, de = 6), on four E4M3 codes per register (no NaN codes among them): the anchor values
// divided by 2^(de + k) = 2^8 (exact in FP16), converted to the hardware neighbour format whose grid is
// 2^-k times the target's (see SoftFp), the one code above the target's largest clipped back.
template <class FL>
__device__ __forceinline__ uint32_t ss_e4m3_word_soft(uint32_t x)
{
    using S = SoftFp<FL>;
    constexpr uint32_t k01 = 0x01010101u;
    constexpr int de = 8 - FL::emax;
    uint32_t c;
    float f[4];
    e4m3_word_scaled<de + S::k>(x, f);
    if constexpr (S::e3m3)
        asm("{ .reg .b16 l, h; cvt.rn.satfinite.e4m3x2.f32 l, %2, %1; cvt.rn.satfinite.e4m3x2.f32 h, %4, %3; mov.b32 %0, {l, h}; }"
            : "=r"(c) : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]));
    else
        asm("{ .reg .b16 l, h; cvt.rn.satfinite.e3m2x2.f32 l, %2, %1; cvt.rn.satfinite.e3m2x2.f32 h, %4, %3; mov.b32 %0, {l, h}; }"
            : "=r"(c) : "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]));
    uint32_t mag = c & (k01 * S::hw_mag_mask);
    mag -= (mag >> (FL::bits - 1)) & k01;
    return mag | ((c >> 1) & (k01 << (FL::bits - 1)));
}

// Every legal pair, one element at a time (exact, slow): the reference path inside the kernels.
template <class FH, class FL, int NWI, int NWO>
__device__ __forceinline__ void ss_unit_by_element(const uint32_t (&in)[NWI], uint32_t (&out)[NWO])
{
#pragma unroll
    for (int j = 0; j < NWO; ++j) out[j] = 0;
    static_for<32>([&](auto i) {
        constexpr int I = decltype(i)::value;
        const uint32_t c = get_code<FH::bits, I>(in);
        uint32_t d;
        if constexpr (FH::kind == KIND_INT) d = ss_int_elem<FH, FL>(c);
        else d = ss_fp_elem<FH, FL>(c);
        put_code<FL::bits, I>(out, d);
    });
}

template <class FH, class FL>
__host__ __device__ constexpr bool ss_e4m3_has_fast_path()
{
    return FH::id == MXQ_FP8_E4M3 && FL::id != MXQ_FP8_E4M3 &&
           (FL::hw_cvt || FL::id == MXQ_FP7_E3M3 || FL::id == MXQ_FP5_E2M2);
}

__device__ __forceinline__ bool unit_has_e4m3_nan(const uint32_t (&in)[8])
{
    bool nan = false;
#pragma unroll
    for (int j = 0; j < 8; ++j) nan |= has_e4m3_nan(in[j]);
    return nan;
}

// The 32 E4M3 codes of one lane, none of them a NaN code, to any lower MXFP format.
template <class FL, int NWO>
__device__ __forceinline__ void ss_e4m3_unit_fast(const uint32_t (&in)[8], uint32_t (&out)[NWO])
{
    if constexpr (FL::hw_cvt && FL::bits == 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) out[j] = ss_e4m3_words_to_e2m1(in[2 * j], in[2 * j + 1]);
    } else if constexpr (FL::hw_cvt) {
        uint32_t z[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) z[j] = squeeze6_low(ss_e4m3_word_to6<FL>(in[j]));
#pragma unroll
        for (int g = 0; g < 2; ++g)
            join24(z[4 * g + 0], z[4 * g + 1], z[4 * g + 2], z[4 * g + 3], out[3 * g + 0], out[3 * g + 1], out[3 * g + 2]);
    } else {
        uint32_t z[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) z[j] = ss_e4m3_word_soft<FL>(in[j]);
        pack_code_bytes<FL::bits>(z, out);
    }
}

// Convert the 32 codes of one lane.  in: 8*FH::bits/8... words of the high format's bitstream.
template <class FH, class FL, int NWI, int NWO>
__device__ __forceinline__ void slice_scale_unit(const uint32_t (&in)[NWI], uint32_t (&out)[NWO])
{
    if constexpr (FH::id == FL::id) {
#pragma unroll
        for (int j = 0; j < NWO; ++j) out[j] = in[j];
    } else if constexpr (FH::id == MXQ_INT8 && FL::bits == 4) {
        // the codes come back in the high nibbles: w * 17 drops each one into the low nibble of the
        // byte above as well, so bytes 1 and 3 of it hold c0 | c1 << 4 and c2 | c3 << 4
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t a = ss_int8_word_top<4>(in[2 * j]), b = ss_int8_word_top<4>(in[2 * j + 1]);
            out[j] = __byte_perm(a * 16u + a, b * 16u + b, 0x7531);
        }
    } else if constexpr (FH::id == MXQ_INT8 && FL::bits == 6) {
        uint32_t z[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) z[j] = squeeze6_top(ss_int8_word_top<6>(in[j]));
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            join24(z[4 * g + 0], z[4 * g + 1], z[4 * g + 2], z[4 * g + 3], out[3 * g + 0], out[3 * g + 1], out[3 * g + 2]);
        }
    } else if constexpr (FH::id == MXQ_INT8 && FL::kind == KIND_INT) {
        // MXINT7 / 5 / 3 / 2: the same four-codes-per-register arithmetic, generic packing
        uint32_t z[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) z[j] = ss_int8_word<FL::bits>(in[j]);
        pack_code_bytes<FL::bits>(z, out);
    } else if constexpr (ss_e4m3_has_fast_path<FH, FL>()) {
        if (!unit_has_e4m3_nan(in)) ss_e4m3_unit_fast<FL>(in, out);
        else ss_unit_by_element<FH, FL>(in, out);     // an E4M3 NaN code (never produced by the quantizer)
    } else {
        ss_unit_by_element<FH, FL>(in, out);          // every other pair, including non-anchor sources
    }
}

// Scale bytes are an element-wise stream of their own: byte -> min(byte + de, 254), 0xFF kept.
__device__ __forceinline__ uint8_t ss_scale_byte(uint32_t b, int de)
{
    return (uint8_t)(b == 0xFFu ? 0xFFu : min(b + (uint32_t)de, 254u));
}

// One warp tile (32 U lane units) of one tensor; shared by the single-tensor and the batched
// kernels.  The scale bytes are an element-wise stream of their own: lane unit i also converts
// scale i, and scale nunits + i when the block is smaller than a lane unit (block 16).
template <class FH, class FL, int U, class SCALES>
__device__ __forceinline__ void slice_scale_tile(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                                 size_t nunits, size_t nscales, uint8_t* __restrict__ out_codes,
                                                 const SCALES& out_scales, size_t tile, uint8_t* stage)
{
    constexpr int IB = 4 * FH::bits, OB = 4 * FL::bits;      // bytes per lane unit
    constexpr int NWI = IB / 4, NWO = OB / 4;
    constexpr int de = FH::emax - FL::emax;
    const size_t u0 = tile * (32 * U) + (threadIdx.x & 31);
    uint32_t w[U][NWI];
    uint32_t sb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) load_words<NWI>(w[u], codes + unit * IB);
        else {
#pragma unroll
            for (int j = 0; j < NWI; ++j) w[u][j] = 0;
        }
        sb[u] = unit < nscales ? ld_u8(scales + unit) : 0;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nscales) put_scale(out_scales, unit, ss_scale_byte(sb[u], de));
        uint32_t out[NWO];
        slice_scale_unit<FH, FL>(w[u], out);
        if constexpr (StagedTile<OB>::use) store_bytes<OB>(stage + (u * 32 + (threadIdx.x & 31)) * OB, out);
        else if (unit < nunits) store_bytes<OB>(out_codes + unit * OB, out);
    }
    if constexpr (StagedTile<OB>::use) {
        const size_t first = tile * (32 * U), left = nunits - first;
        flush_stage<32 * U * OB>(stage, out_codes + first * OB, (uint32_t)(left < 32 * U ? left : 32 * U) * OB);
    }
    if (nscales > nunits) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = nunits + u0 + u * 32;
            if (i < nscales) put_scale(out_scales, i, ss_scale_byte(ld_u8(scales + i), de));
        }
    }
}

// The staging area of the calling warp for a Slice-and-Scale tile (null when the target's pieces are
// single vectors).  Must be called by every thread of the CTA, outside divergent code.
template <class FL, int U, int THREADS>
__device__ __forceinline__ uint8_t* slice_scale_stage()
{
    constexpr int OB = 4 * FL::bits;
    if constexpr (StagedTile<OB>::use) {
        __shared__ __align__(128) uint8_t stage_area[(THREADS / 32) * 32 * U * OB];
        return stage_area + (threadIdx.x >> 5) * (32 * U * OB);
    } else {
        return nullptr;
    }
}

// Resident CTAs (of 128 threads) per SM the single-tensor kernel is compiled for, i.e. its register
// budget.  Measured at 2^26 codes with 10 / 12 / 14 / 16 CTAs: the MXINT conversions are fastest with
// room for 40 - 48 registers (both lane units' arithmetic interleaves; MXINT8 -> MXINT4 8 % faster
// than at 32 registers), the MXFP ones with 14 - 16 CTAs (E4M3 -> E2M3 8 % faster than at 50
// registers); with tiled scale outputs 14 CTAs would spill, so those keep 12.
template <class FH, class SCALES>
__host__ __device__ constexpr int slice_scale_min_ctas()
{
    if constexpr (!std::is_same_v<SCALES, uint8_t*>) return 12;
    else return FH::kind == KIND_INT ? 10 : 14;
}

template <class FH, class FL, int U, int THREADS, class SCALES = uint8_t*>
__global__ void __launch_bounds__(THREADS, slice_scale_min_ctas<FH, SCALES>())
slice_scale_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales, size_t nunits,
                   size_t nscales, uint8_t* __restrict__ out_codes, SCALES out_scales)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t* stage = slice_scale_stage<FL, U, THREADS>();
    prefetch_tile<U, 4 * FH::bits>(codes, tile, nunits);
    pdl_acquire();
    if (tile * (32 * U) < nunits)
        slice_scale_tile<FH, FL, U>(codes, scales, nunits, nscales, out_codes, out_scales, tile, stage);
}

// Two targets from one read of the anchor (the elastic-serving case: one stored checkpoint, several
// lower precisions wanted at once).  Per element 1.03 bytes are read once instead of twice.
// (Left to itself the compiler gives this kernel 64 - 71 registers, 7 CTAs per SM; asked for 12 CTAs it
// finds 40 without spilling, and the launch is 2 % shorter.)
// One warp tile of the two-target conversion; shared by the single-tensor and the batched kernels.
template <class FH, class FL1, class FL2, int U>
__device__ __forceinline__ void slice_scale2_tile(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                                  size_t nunits, size_t nscales, uint8_t* __restrict__ out_codes1,
                                                  uint8_t* __restrict__ out_scales1, uint8_t* __restrict__ out_codes2,
                                                  uint8_t* __restrict__ out_scales2, size_t tile, uint8_t* stage1,
                                                  uint8_t* stage2)
{
    constexpr int IB = 4 * FH::bits, NWI = IB / 4;
    constexpr int OB1 = 4 * FL1::bits, OB2 = 4 * FL2::bits;
    constexpr int de1 = FH::emax - FL1::emax, de2 = FH::emax - FL2::emax;
    const size_t u0 = tile * (32 * U) + (threadIdx.x & 31);
    uint32_t w[U][NWI];
    uint32_t sb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) load_words<NWI>(w[u], codes + unit * IB);
        else {
#pragma unroll
            for (int j = 0; j < NWI; ++j) w[u][j] = 0;
        }
        sb[u] = unit < nscales ? ld_u8(scales + unit) : 0;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nscales) {
            st_u8(out_scales1 + unit, ss_scale_byte(sb[u], de1));
            st_u8(out_scales2 + unit, ss_scale_byte(sb[u], de2));
        }
        uint32_t o1[OB1 / 4], o2[OB2 / 4];
        if constexpr (ss_e4m3_has_fast_path<FH, FL1>() && ss_e4m3_has_fast_path<FH, FL2>()) {
            // one NaN-code check, both conversions in one straight line: what they share (the widening
            // of the anchor codes, the scaled values when de is the same) is computed once
            if (!unit_has_e4m3_nan(w[u])) {
                ss_e4m3_unit_fast<FL1>(w[u], o1);
                ss_e4m3_unit_fast<FL2>(w[u], o2);
            } else {
                ss_unit_by_element<FH, FL1>(w[u], o1);
                ss_unit_by_element<FH, FL2>(w[u], o2);
            }
        } else {
            slice_scale_unit<FH, FL1>(w[u], o1);
            slice_scale_unit<FH, FL2>(w[u], o2);
        }
        if constexpr (StagedTile<OB1>::use) store_bytes<OB1>(stage1 + (u * 32 + (threadIdx.x & 31)) * OB1, o1);
        else if (unit < nunits) store_bytes<OB1>(out_codes1 + unit * OB1, o1);
        if constexpr (StagedTile<OB2>::use) store_bytes<OB2>(stage2 + (u * 32 + (threadIdx.x & 31)) * OB2, o2);
        else if (unit < nunits) store_bytes<OB2>(out_codes2 + unit * OB2, o2);
    }
    {
        const size_t first = tile * (32 * U), left = nunits - first;
        const uint32_t valid = (uint32_t)(left < 32 * U ? left : 32 * U);
        if constexpr (StagedTile<OB1>::use) flush_stage<32 * U * OB1>(stage1, out_codes1 + first * OB1, valid * OB1);
        if constexpr (StagedTile<OB2>::use) flush_stage<32 * U * OB2>(stage2, out_codes2 + first * OB2, valid * OB2);
    }
    if (nscales > nunits) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = nunits + u0 + u * 32;
            if (i < nscales) {
                const uint32_t b = ld_u8(scales + i);
                st_u8(out_scales1 + i, ss_scale_byte(b, de1));
                st_u8(out_scales2 + i, ss_scale_byte(b, de2));
            }
        }
    }
}

// The two staging areas of the calling warp (null where the target's pieces are stored directly).
// Must be called by every thread of the CTA, outside divergent code.
template <class FL1, class FL2, int U, int THREADS>
__device__ __forceinline__ void slice_scale2_stages(uint8_t*& stage1, uint8_t*& stage2)
{
    constexpr int OB1 = 4 * FL1::bits, OB2 = 4 * FL2::bits;
    stage1 = nullptr;
    stage2 = nullptr;
    if constexpr (StagedTile<OB1>::use) {
        __shared__ __align__(128) uint8_t area1[(THREADS / 32) * 32 * U * OB1];
        stage1 = area1 + (threadIdx.x >> 5) * (32 * U * OB1);
    }
    if constexpr (StagedTile<OB2>::use) {
        __shared__ __align__(128) uint8_t area2[(THREADS / 32) * 32 * U * OB2];
        stage2 = area2 + (threadIdx.x >> 5) * (32 * U * OB2);
    }
}

template <class FH, class FL1, class FL2, int U, int THREADS>
__global__ void __launch_bounds__(THREADS, 1536 / THREADS)
slice_scale2_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales, size_t nunits, size_t nscales,
                    uint8_t* __restrict__ out_codes1, uint8_t* __restrict__ out_scales1,
                    uint8_t* __restrict__ out_codes2, uint8_t* __restrict__ out_scales2)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t *stage1, *stage2;
    slice_scale2_stages<FL1, FL2, U, THREADS>(stage1, stage2);
    prefetch_tile<U, 4 * FH::bits>(codes, tile, nunits);
    pdl_acquire();
    if (tile * (32 * U) >= nunits) return;                     // whole warps leave together
    slice_scale2_tile<FH, FL1, FL2, U>(codes, scales, nunits, nscales, out_codes1, out_scales1, out_codes2, out_scales2,
                                       tile, stage1, stage2);
}

// Device-side item of the batched conversion (one tensor), with its place in the flattened
// tile space of the whole batch.
struct SsDeviceItem {
    const uint8_t* codes;
    const uint8_t* scales;
    uint8_t* out_codes;
    uint8_t* out_scales;
    size_t nunits;
    size_t nscales;
    size_t tile_begin;     // first global tile index of this tensor
};

// All tensors in one launch: the tiles of every tensor are laid end to end and every warp finds the
// tensor its tile belongs to by a binary search of the item table, so small tensors do not leave
// SMs idle.
template <class FH, class FL, int U, int THREADS>
__global__ void __launch_bounds__(THREADS)
slice_scale_batched_kernel(const SsDeviceItem* __restrict__ items, const TileIndex* __restrict__ index, int count,
                           size_t total_tiles)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t* stage = slice_scale_stage<FL, U, THREADS>();
    pdl_acquire();
    if (tile >= total_tiles) return;
    // items are sorted by tile_begin: the last one that starts at or before this tile owns it
    // (table and index are device memory written by the copy in front of this launch: read after the wait)
    const SsDeviceItem t = items[find_item(items, *index, tile)];
    slice_scale_tile<FH, FL, U>(t.codes, t.scales, t.nunits, t.nscales, t.out_codes, t.out_scales, tile - t.tile_begin,
                                stage);
}

// The same launch with the item table carried in the kernel's parameter space (K items, 56 bytes
// each, plus the coarse index: K = 64 stays near the classic 4 KB of parameters, K = 512 uses the
// 32 KB that sm_70 and later allow).  No device buffer, no host-to-device copy in front of the kernel.
template <int K>
struct SsItemBlock {
    SsDeviceItem items[K];
    TileIndex index;
};

template <class FH, class FL, int U, int THREADS, int K>
__global__ void __launch_bounds__(THREADS)
slice_scale_batched_param_kernel(const __grid_constant__ SsItemBlock<K> blk, int count, size_t total_tiles)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t* stage = slice_scale_stage<FL, U, THREADS>();
    // parameters: readable before the wait
    const SsDeviceItem& t = blk.items[tile < total_tiles ? find_item(blk.items, blk.index, tile) : 0];
    if (tile < total_tiles) prefetch_tile<U, 4 * FH::bits>(t.codes, tile - t.tile_begin, t.nunits);
    pdl_acquire();
    if (tile >= total_tiles) return;
    slice_scale_tile<FH, FL, U>(t.codes, t.scales, t.nunits, t.nscales, t.out_codes, t.out_scales, tile - t.tile_begin,
                                stage);
}

// Two targets from one read of every anchor of a set of tensors (the whole-model conversion of Sec. 3.5
// for a deployment that serves two lower precisions at once): items of 72 bytes, 256 per launch.
struct Ss2DeviceItem {
    const uint8_t* codes;
    const uint8_t* scales;
    uint8_t* out_codes1;
    uint8_t* out_scales1;
    uint8_t* out_codes2;
    uint8_t* out_scales2;
    size_t nunits;
    size_t nscales;
    size_t tile_begin;
};

template <int K>
struct Ss2ItemBlock {
    Ss2DeviceItem items[K];
    TileIndex index;
};

// (The item's six pointers live in registers here.  Measured over the 224-tensor weight set with 6 / 8 / 10 / 12
// resident CTAs: 10 -- 48 registers, 12 - 20 bytes of spills in the MXFP variants -- is the fastest for the
// MXFP pair (2.42 ms against 2.60 at 8 and 3.13 at 12) and within 2 % of the best for the MXINT pair.)
template <class FH, class FL1, class FL2, int U, int THREADS, int K>
__global__ void __launch_bounds__(THREADS, 10)
slice_scale2_batched_kernel(const __grid_constant__ Ss2ItemBlock<K> blk, int count, size_t total_tiles)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t *stage1, *stage2;
    slice_scale2_stages<FL1, FL2, U, THREADS>(stage1, stage2);
    const Ss2DeviceItem& t = blk.items[tile < total_tiles ? find_item(blk.items, blk.index, tile) : 0];
    if (tile < total_tiles) prefetch_tile<U, 4 * FH::bits>(t.codes, tile - t.tile_begin, t.nunits);
    pdl_acquire();
    if (tile >= total_tiles) return;
    slice_scale2_tile<FH, FL1, FL2, U>(t.codes, t.scales, t.nunits, t.nscales, t.out_codes1, t.out_scales1, t.out_codes2,
                                       t.out_scales2, tile - t.tile_begin, stage1, stage2);
}

// The batched conversion with every tensor's scale bytes written in the tiled order (block 32): the
// item carries the matrix's TiledScales record in place of a plain pointer.  K = 256 items of 72 bytes
// ride in the kernel parameters.
struct SsTiledDeviceItem {
    const uint8_t* codes;
    const uint8_t* scales;
    uint8_t* out_codes;
    TiledScales out_scales;
    size_t nunits;
    size_t tile_begin;
};

template <int K>
struct SsTiledItemBlock {
    SsTiledDeviceItem items[K];
    TileIndex index;
};

template <class FH, class FL, int U, int THREADS, int K>
__global__ void __launch_bounds__(THREADS)
slice_scale_tiled_batched_kernel(const __grid_constant__ SsTiledItemBlock<K> blk, int count, size_t total_tiles)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    uint8_t* stage = slice_scale_stage<FL, U, THREADS>();
    // parameters: readable before the wait
    const SsTiledDeviceItem& t = blk.items[tile < total_tiles ? find_item(blk.items, blk.index, tile) : 0];
    if (tile < total_tiles) prefetch_tile<U, 4 * FH::bits>(t.codes, tile - t.tile_begin, t.nunits);
    pdl_acquire();
    if (tile >= total_tiles) return;
    slice_scale_tile<FH, FL, U>(t.codes, t.scales, t.nunits, t.nunits, t.out_codes, t.out_scales, tile - t.tile_begin,
                                stage);
}

// ------------------------------------------------------------------------------------------
// Reconstruction V^ = X P.  One lane = 32 codes.
// ------------------------------------------------------------------------------------------

// Two kernels.  For 16-bit outputs a lane takes 32 codes (one block: 16 - 32 bytes of codes in one
// vector load) and writes 64 bytes; for FP32 outputs that shape would spread every store instruction
// of a warp over 32 different 128-byte lines (measured 84 % of the copy rate), so there a lane unit
// is 32 bytes of OUTPUT instead and every store instruction covers 1 KB of consecutive addresses
// (98 %).  The second shape was 1 - 2 % slower than the first for BF16 outputs.

template <class F, class T, int U>
__device__ __forceinline__ void dequantize_tile(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                                size_t nunits, int units_per_scale_shift, int scales_per_unit,
                                                uint8_t* __restrict__ dst, size_t tile)
{
    constexpr int IB = 4 * F::bits, NWI = IB / 4;
    constexpr int OBYTES = 32 * T::size;                      // 64 or 128 bytes out per lane
    const int lane = threadIdx.x & 31;
    const size_t u0 = tile * (32 * U) + lane;
    uint32_t w[U][NWI];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) load_words<NWI>(w[u], codes + unit * IB);
        else {
#pragma unroll
            for (int j = 0; j < NWI; ++j) w[u][j] = 0;
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit >= nunits) continue;
        // scales_per_unit is 1 (block >= 32: one scale shared by 2^shift units) or 2 (block 16)
        uint32_t sbyte[2];
        if (scales_per_unit == 1) {
            sbyte[0] = sbyte[1] = ld_u8(scales + (unit >> units_per_scale_shift));
        } else {
            sbyte[0] = ld_u8(scales + unit * 2);
            sbyte[1] = ld_u8(scales + unit * 2 + 1);
        }
        uint8_t* o = dst + unit * OBYTES;
        // four 32-byte stores for FP32 (8 elements each), two for BF16 (16 elements each)
        constexpr int EPS = 32 / T::size;
        static_for<32 / EPS>([&](auto k) {
            constexpr int K = decltype(k)::value;
            const uint32_t sbk = sbyte[(K * EPS) / 16];
            uint32_t out[8];
            if (sbk == 0xFFu) {
#pragma unroll
                for (int j = 0; j < 8; ++j) out[j] = T::size == 4 ? 0x7FC00000u : 0x7FC07FC0u;
            } else if (F::id == MXQ_FP8_E4M3 && T::size == 2 &&
                       !(has_e4m3_nan(w[u][(4 * K) % NWI]) | has_e4m3_nan(w[u][(4 * K + 1) % NWI]) |
                         has_e4m3_nan(w[u][(4 * K + 2) % NWI]) | has_e4m3_nan(w[u][(4 * K + 3) % NWI]))) {
                // MXFP8 anchor codes (no NaN code among these 16): the widening conversion gives the
                // exact values, one FP32 multiply applies the scale as in the generic path below
                const float X = scale_value(sbk);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t a, b;
                    e4m3_word_to_f16(w[u][(4 * K + j) % NWI], a, b);
                    float f0, f1, f2, f3;
                    asm("{ .reg .b16 l, h; mov.b32 {l, h}, %4; cvt.f32.f16 %0, l; cvt.f32.f16 %1, h;\n"
                        "  mov.b32 {l, h}, %5; cvt.f32.f16 %2, l; cvt.f32.f16 %3, h; }"
                        : "=f"(f0), "=f"(f1), "=f"(f2), "=f"(f3) : "r"(a), "r"(b));
                    out[2 * j] = pack_bf16x2(f0 * X, f1 * X);
                    out[2 * j + 1] = pack_bf16x2(f2 * X, f3 * X);
                }
            } else {
                const float X = scale_value(sbk);
                static_for<EPS / 2>([&](auto i) {
                    constexpr int I = K * EPS + 2 * decltype(i)::value;
                    const uint32_t c0 = get_code<F::bits, I>(w[u]), c1 = get_code<F::bits, I + 1>(w[u]);
                    float y0 = decode<F>(c0) * X;
                    float y1 = decode<F>(c1) * X;
                    // an E4M3 NaN code reconstructs to the canonical quiet NaN
                    bool n0 = false, n1 = false;
                    if constexpr (F::has_nan) {
                        n0 = (c0 & 0x7Fu) == 0x7Fu;
                        n1 = (c1 & 0x7Fu) == 0x7Fu;
                    }
                    if constexpr (T::size == 4) {
                        out[I - K * EPS] = n0 ? 0x7FC00000u : __float_as_uint(y0);
                        out[I - K * EPS + 1] = n1 ? 0x7FC00000u : __float_as_uint(y1);
                    } else {
                        uint32_t p = pack_bf16x2(y0, y1);
                        if (n0) p = (p & 0xFFFF0000u) | 0x7FC0u;
                        if (n1) p = (p & 0x0000FFFFu) | 0x7FC00000u;
                        out[(I - K * EPS) / 2] = p;
                    }
                });
            }
            st256(o + K * 32, out);
        });
    }
}

template <class F, class T, int U, int THREADS>
__global__ void __launch_bounds__(THREADS)
dequantize_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales, size_t nunits,
                  int units_per_scale_shift, int scales_per_unit, uint8_t* __restrict__ dst)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    pdl_acquire();
    if (tile * (32 * U) < nunits)
        dequantize_tile<F, T, U>(codes, scales, nunits, units_per_scale_shift, scales_per_unit, dst, tile);
}


// A lane unit is 32 bytes of OUTPUT (16 BF16 or 8 FP32 elements), so that every store instruction
// of a warp covers 1 KB of consecutive addresses; the codes of a unit are 2 x bits or bits bytes,
// read with the widest access their alignment allows.  A unit never straddles a block (blocks are
// at least 16 elements), so it needs one scale: scales[unit >> scale_shift].
template <class F, class T, int U>
__device__ __forceinline__ void dequantize_wide_tile(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                                     size_t nunits, int scale_shift, uint8_t* __restrict__ dst, size_t tile)
{
    constexpr int EPL = T::epl;                               // elements per lane unit
    constexpr int IB = EPL * F::bits / 8;                     // code bytes per lane unit
    constexpr int NWI = (IB + 3) / 4;
    const size_t u0 = tile * (32 * U) + (threadIdx.x & 31);
    uint32_t w[U][NWI];
    uint32_t sb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        if (unit < nunits) {
            load_bytes<IB>(w[u], codes + unit * IB);
            sb[u] = ld_u8(scales + (unit >> scale_shift));
        } else {
#pragma unroll
            for (int j = 0; j < NWI; ++j) w[u][j] = 0;
            sb[u] = 0;
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t unit = u0 + u * 32;
        uint32_t out[8];
        const float X = scale_value(min(sb[u], 254u));
        static_for<EPL / 2>([&](auto i) {
            constexpr int I = 2 * decltype(i)::value;
            const uint32_t c0 = get_code<F::bits, I>(w[u]), c1 = get_code<F::bits, I + 1>(w[u]);
            float y0 = decode<F>(c0) * X;
            float y1 = decode<F>(c1) * X;
            // an E4M3 NaN code reconstructs to the canonical quiet NaN
            bool n0 = false, n1 = false;
            if constexpr (F::has_nan) {
                n0 = (c0 & 0x7Fu) == 0x7Fu;
                n1 = (c1 & 0x7Fu) == 0x7Fu;
            }
            if constexpr (T::size == 4) {
                out[I] = n0 ? 0x7FC00000u : __float_as_uint(y0);
                out[I + 1] = n1 ? 0x7FC00000u : __float_as_uint(y1);
            } else {
                uint32_t p = pack_bf16x2(y0, y1);
                if (n0) p = (p & 0xFFFF0000u) | 0x7FC0u;
                if (n1) p = (p & 0x0000FFFFu) | 0x7FC00000u;
                out[I / 2] = p;
            }
        });
        if (sb[u] == 0xFFu) {                                 // poisoned block
#pragma unroll
            for (int j = 0; j < 8; ++j) out[j] = T::size == 4 ? 0x7FC00000u : 0x7FC07FC0u;
        }
        if (unit < nunits) st256(dst + unit * 32, out);
    }
}

template <class F, class T, int U, int THREADS>
__global__ void __launch_bounds__(THREADS)
dequantize_wide_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales, size_t nunits, int scale_shift,
                       uint8_t* __restrict__ dst)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    pdl_acquire();
    if (tile * (32 * U) < nunits) dequantize_wide_tile<F, T, U>(codes, scales, nunits, scale_shift, dst, tile);
}

// Reconstruction of a whole set of tensors in one launch (tiles end to end, items in the parameters).
// `shift` and `scales_per_unit` are those of the single-tensor kernel of the same output type.
struct DqDeviceItem {
    const uint8_t* codes;
    const uint8_t* scales;
    uint8_t* dst;
    size_t nunits;
    size_t tile_begin;
};

template <int K>
struct DqItemBlock {
    DqDeviceItem items[K];
    TileIndex index;
};

template <class F, class T, int U, int THREADS, int K>
__global__ void __launch_bounds__(THREADS)
dequantize_batched_kernel(const __grid_constant__ DqItemBlock<K> blk, int count, size_t total_tiles, int shift,
                          int scales_per_unit)
{
    pdl_release();
    const size_t tile = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    const DqDeviceItem& t = blk.items[tile < total_tiles ? find_item(blk.items, blk.index, tile) : 0];
    pdl_acquire();
    if (tile >= total_tiles) return;
    if constexpr (T::size == 4) dequantize_wide_tile<F, T, U>(t.codes, t.scales, t.nunits, shift, t.dst, tile - t.tile_begin);
    else dequantize_tile<F, T, U>(t.codes, t.scales, t.nunits, shift, scales_per_unit, t.dst, tile - t.tile_begin);
}

// ------------------------------------------------------------------------------------------
// Straight-through backward: a plain copy
// ------------------------------------------------------------------------------------------

template <int U, int THREADS>
__global__ void __launch_bounds__(THREADS)
copy_kernel(const uint8_t* __restrict__ src, size_t nbytes, uint8_t* __restrict__ dst)
{
    pdl_release();
    const size_t nunits = nbytes / 32;
    const int lane = threadIdx.x & 31;
    const size_t warp = (size_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5);
    const size_t ntiles = (nunits + 32 * U - 1) / (32 * U);
    prefetch_tile<U, 32>(src, warp, nunits);
    pdl_acquire();
    if (const size_t tile = warp; tile < ntiles) {
        const size_t u0 = tile * (32 * U) + lane;
        uint32_t w[U][8];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (u0 + u * 32 < nunits) ld256(w[u], src + (u0 + u * 32) * 32);
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (u0 + u * 32 < nunits) st256(dst + (u0 + u * 32) * 32, w[u]);
    }
    // ragged tail (n * size need not be a multiple of 32 bytes)
    const size_t tid = (size_t)blockIdx.x * THREADS + threadIdx.x;
    for (size_t i = nunits * 32 + tid; i < nbytes; i += (size_t)gridDim.x * THREADS) st_u8(dst + i, ld_u8(src + i));
}

}  // namespace mxq
