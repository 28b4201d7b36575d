// Device-side element codec for the MX formats: format traits, the element quantizers
// (Eq. 2-3 of the MF-QAT paper), the Slice-and-Scale element maps (Eq. 4-5) and the decoders
// used by reconstruction.  Everything here works on registers; memory access lives in
// mxq_access.cuh and the kernels.
//
// Conventions (identical to the public header): e_max(MXINT b) = b - 2, symmetric clip,
// MXINT rounds to nearest with ties away from zero; MXFP rounds to nearest even onto the
// element grid with subnormals, saturates to the largest finite magnitude and keeps the sign
// of zero; FP8 E4M3 uses the OCP encoding.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/mxq.h"

namespace mxq {

enum { KIND_INT = 0, KIND_FP = 1 };

struct FmtInfo {
    int kind, bits, eta, mu;
};

__host__ __device__ constexpr FmtInfo fmt_info(int f)
{
    switch (f) {
    case MXQ_INT8: return {KIND_INT, 8, 0, 0};
    case MXQ_INT7: return {KIND_INT, 7, 0, 0};
    case MXQ_INT6: return {KIND_INT, 6, 0, 0};
    case MXQ_INT5: return {KIND_INT, 5, 0, 0};
    case MXQ_INT4: return {KIND_INT, 4, 0, 0};
    case MXQ_INT3: return {KIND_INT, 3, 0, 0};
    case MXQ_INT2: return {KIND_INT, 2, 0, 0};
    case MXQ_FP8_E4M3: return {KIND_FP, 8, 4, 3};
    case MXQ_FP7_E3M3: return {KIND_FP, 7, 3, 3};
    case MXQ_FP6_E3M2: return {KIND_FP, 6, 3, 2};
    case MXQ_FP6_E2M3: return {KIND_FP, 6, 2, 3};
    case MXQ_FP5_E2M2: return {KIND_FP, 5, 2, 2};
    case MXQ_FP4_E2M1: return {KIND_FP, 4, 2, 1};
    default: return {-1, 0, 0, 0};
    }
}

// Compile-time view of one element format.
template <int F>
struct Fmt {
    static constexpr FmtInfo I = fmt_info(F);
    static constexpr int id = F;
    static constexpr int kind = I.kind;
    static constexpr int bits = I.bits;
    static constexpr int eta = I.eta;
    static constexpr int mu = I.mu;
    static constexpr uint32_t mask = (1u << bits) - 1u;
    // exponent of the largest normal number (Sec. 3.3, Notation)
    static constexpr int emax = kind == KIND_INT ? bits - 2 : (1 << (eta > 0 ? eta - 1 : 0));
    static constexpr int bias = kind == KIND_FP ? (1 << (eta - 1)) - 1 : 0;
    static constexpr int emin = 1 - bias;                       // exponent of the smallest normal
    static constexpr bool has_nan = kind == KIND_FP && eta == 4 && mu == 3;
    // largest finite magnitude code (sign bit excluded)
    static constexpr uint32_t max_mag = kind == KIND_INT ? (1u << (bits - 1)) - 1u
                                                         : ((1u << (bits - 1)) - 1u) - (has_nan ? 1u : 0u);
    // formats the sm_100a cvt instruction narrows to directly
    static constexpr bool hw_cvt = F == MXQ_FP8_E4M3 || F == MXQ_FP6_E3M2 || F == MXQ_FP6_E2M3 || F == MXQ_FP4_E2M1;
};

__host__ __device__ constexpr int fmt_emax(int f)
{
    return fmt_info(f).kind == KIND_INT ? fmt_info(f).bits - 2 : (1 << (fmt_info(f).eta - 1));
}

// A Slice-and-Scale pair is legal when both formats belong to one family, the scale moves up or
// stays (de = e_max(h) - e_max(l) >= 0) and the codes do not get wider.
__host__ __device__ constexpr bool ss_pair_ok(int h, int l)
{
    return fmt_info(h).kind >= 0 && fmt_info(h).kind == fmt_info(l).kind && fmt_emax(h) >= fmt_emax(l) &&
           fmt_info(l).bits <= fmt_info(h).bits;
}

// ------------------------------------------------------------------------------------------
// Block scale (Eq. 1)
// ------------------------------------------------------------------------------------------

struct BlockScale {
    uint32_t byte;   // E8M0 byte, 0xFF for a poisoned block
    float inv;       // 2^-shared_exp (exact power of two)
};

// `amax_bits` = FP32 bit pattern of max_i |V_i| (sign cleared).  Inf/NaN patterns poison the block.
template <class F>
__device__ __forceinline__ BlockScale block_scale(uint32_t amax_bits)
{
    const uint32_t ex = amax_bits >> 23;
    // floor(log2 amax): exponent field for normals, position of the leading one for subnormals;
    // zero gives -150, which the clamp below turns into byte 0.
    int e = ex ? (int)ex - 127 : (31 - __clz(amax_bits)) - 149;
    int se = max(e - F::emax, -127);                 // e <= 127 and e_max >= 0: no upper clamp needed
    BlockScale s;
    s.byte = amax_bits >= 0x7F800000u ? 0xFFu : (uint32_t)(se + 127);
    uint32_t field = (uint32_t)(127 - se);           // exponent field of 2^-se, in [0, 254]
    uint32_t ib = field << 23;
    if constexpr (F::emax == 0) ib = field ? ib : 0x00400000u;   // 2^-127 is an FP32 subnormal
    s.inv = __uint_as_float(ib);
    return s;
}

// 2^(byte-127) as FP32 (byte 0 is the subnormal 2^-127).  byte must be <= 254.
__device__ __forceinline__ float scale_value(uint32_t byte)
{
    return __uint_as_float(byte ? byte << 23 : 0x00400000u);
}

// ------------------------------------------------------------------------------------------
// MXFP element quantizers (Eq. 2).  `v` is the raw element, `inv` = 2^-shared_exp; v * inv is exact.
// ------------------------------------------------------------------------------------------

// MXFP by plain ALU arithmetic, any (eta, mu): add 2^(ea + 23 - mu) so that the FP32 adder
// rounds |r| (nearest even) to the element grid of its binade (ea = max(exponent, emin)); the
// mantissa field of the sum is then the element's integer significand.
template <class F>
__device__ __forceinline__ uint32_t fp_magnitude_alu(float r)
{
    uint32_t rb = __float_as_uint(r);
    uint32_t eb = max(rb & 0x7F800000u, (uint32_t)(127 + F::emin) << 23);
    float c = __uint_as_float(eb + ((uint32_t)(23 - F::mu) << 23));
    float s = fabsf(r) + c;
    uint32_t m = __float_as_uint(s) & 0x007FFFFFu;
    uint32_t code = (eb >> (23 - F::mu)) - ((uint32_t)(127 + F::emin) << F::mu) + m;
    return min(code, F::max_mag);
}

template <class F>
__device__ __forceinline__ uint32_t quantize_fp_alu(float r)
{
    return fp_magnitude_alu<F>(r) | ((__float_as_uint(r) >> 31) << (F::bits - 1));
}

// MXFP through the sm_100a narrowing conversions (round-to-nearest-even, saturating).
// Returns code(r0) | code(r1) << 8 for 8- and 6-bit formats (6-bit codes sit in the low bits of
// their byte) and code(r0) | code(r1) << 4 for E2M1.
template <class F>
__device__ __forceinline__ uint32_t quantize_fp_hw_pair(float r0, float r1)
{
    static_assert(F::hw_cvt, "no narrowing cvt for this format");
    uint32_t d;
    if constexpr (F::id == MXQ_FP8_E4M3) {
        uint16_t h;
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(h) : "f"(r1), "f"(r0));
        d = h;
    } else if constexpr (F::id == MXQ_FP6_E3M2) {
        uint16_t h;
        asm("cvt.rn.satfinite.e3m2x2.f32 %0, %1, %2;" : "=h"(h) : "f"(r1), "f"(r0));
        d = h;
    } else if constexpr (F::id == MXQ_FP6_E2M3) {
        uint16_t h;
        asm("cvt.rn.satfinite.e2m3x2.f32 %0, %1, %2;" : "=h"(h) : "f"(r1), "f"(r0));
        d = h;
    } else {
        asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; cvt.u32.u8 %0, t; }"
            : "=r"(d) : "f"(r1), "f"(r0));
    }
    return d;
}

// The two MXFP formats without a narrowing instruction, E3M3 and E2M2, are the hardware formats E4M3
// and E3M2 with fewer binades: the mantissa width is the same, so 2^-k times the grid of E3M3 (E2M2),
// k = the difference of the exponent biases (4 / 2), IS the grid of E4M3 (E3M2) up to the image of the
// largest magnitude -- normal binades map to normal binades, and the uniform (subnormal) range of the
// one lands exactly on the subnormal range of the other.  Hence code_F(r) = code_hw(r / 2^k), the
// magnitude bits unchanged, except that the hardware format goes on above F's largest value: since
// |r| < 2^(e_max + 1), the only code it can give beyond F's largest is the next one (a single bit,
// 2^(bits - 1)), which is clipped back by subtracting that bit shifted down to 1.
template <class F>
struct SoftFp {
    static_assert(F::id == MXQ_FP7_E3M3 || F::id == MXQ_FP5_E2M2, "E3M3 or E2M2");
    static constexpr bool e3m3 = F::id == MXQ_FP7_E3M3;
    static constexpr int hw = e3m3 ? MXQ_FP8_E4M3 : MXQ_FP6_E3M2;        // the hardware neighbour
    static constexpr int k = e3m3 ? 4 : 2;                                // bias_hw - bias_F
    static constexpr float pre_scale = e3m3 ? 0.0625f : 0.25f;            // 2^-k
    static constexpr float post_scale = e3m3 ? 16.0f : 4.0f;              // 2^k
    static constexpr uint32_t hw_mag_mask = e3m3 ? 0x7Fu : 0x1Fu;
};

// Codes of four elements given as r / 2^k (r = v / X exact, |r| < 2^(e_max + 1)), one per byte.
template <class F>
__device__ __forceinline__ uint32_t quantize_fp_soft_quad(float r0, float r1, float r2, float r3)
{
    using S = SoftFp<F>;
    constexpr uint32_t k01 = 0x01010101u;
    uint32_t c;                                                           // four neighbour codes, one per byte
    if constexpr (S::e3m3)
        asm("{ .reg .b16 l, h; cvt.rn.satfinite.e4m3x2.f32 l, %2, %1; cvt.rn.satfinite.e4m3x2.f32 h, %4, %3; mov.b32 %0, {l, h}; }"
            : "=r"(c) : "f"(r0), "f"(r1), "f"(r2), "f"(r3));
    else
        asm("{ .reg .b16 l, h; cvt.rn.satfinite.e3m2x2.f32 l, %2, %1; cvt.rn.satfinite.e3m2x2.f32 h, %4, %3; mov.b32 %0, {l, h}; }"
            : "=r"(c) : "f"(r0), "f"(r1), "f"(r2), "f"(r3));
    uint32_t mag = c & (k01 * S::hw_mag_mask);
    mag -= (mag >> (F::bits - 1)) & k01;                                  // the one code above F's largest
    // sign: top bit of the neighbour's code -> top bit of F's code (one position down in both cases)
    return mag | ((c >> 1) & (k01 << (F::bits - 1)));
}

// Two elements given as r / 2^k -> their two neighbour-format codes (code(r0) | code(r1) << 8), the
// one code above F's largest clipped back: decoded as neighbour values they are P / 2^k.
template <class F>
__device__ __forceinline__ uint32_t quantize_fp_soft_pair(float r0, float r1)
{
    const uint32_t d = quantize_fp_hw_pair<Fmt<SoftFp<F>::hw>>(r0, r1);
    return d - ((d >> (F::bits - 1)) & 0x0101u);
}

// Quantize two scaled-on-the-fly elements to an MXFP format; returns the two codes in the low `bits`
// bits of .x and .y.  (MXINT elements are quantized four at a time, see quantize_int_quad.)
template <class F>
__device__ __forceinline__ uint2 quantize_pair(float v0, float v1, float inv)
{
    static_assert(F::kind == KIND_FP, "MXFP formats only");
    uint2 c;
    if constexpr (F::hw_cvt) {
        uint32_t d = quantize_fp_hw_pair<F>(v0 * inv, v1 * inv);
        if constexpr (F::bits == 4) {
            c.x = d & 0xFu;
            c.y = (d >> 4) & 0xFu;
        } else {
            c.x = d & 0xFFu;
            c.y = (d >> 8) & 0xFFu;
        }
    } else {
        c.x = quantize_fp_alu<F>(v0 * inv);
        c.y = quantize_fp_alu<F>(v1 * inv);
    }
    return c;
}

// ------------------------------------------------------------------------------------------
// Decoders: code -> FP32 value P (exact)
// ------------------------------------------------------------------------------------------

template <class F>
__device__ __forceinline__ float decode(uint32_t code)
{
    if constexpr (F::kind == KIND_INT) {
        int32_t q = (int32_t)(code << (32 - F::bits)) >> (32 - F::bits);   // sign extend
        // small integers to float without the conversion pipe: 1.5 * 2^23 + q, then subtract
        return __uint_as_float(0x4B400000u + (uint32_t)q) - 12582912.0f;
    } else {
        // Place the magnitude so that its exponent field lines up with FP32's: the result is
        // 2^(bias-127) times the element value, subnormal elements becoming FP32 subnormals;
        // one exact multiply by 2^(127-bias) rescales it.
        uint32_t mag = code & ((1u << (F::bits - 1)) - 1u);
        uint32_t b = (mag << (23 - F::mu)) | ((code >> (F::bits - 1)) << 31);
        return __uint_as_float(b) * __uint_as_float((uint32_t)(254 - F::bias) << 23);
    }
}

// ------------------------------------------------------------------------------------------
// Slice-and-Scale element maps (Eq. 4-5), scalar forms
// ------------------------------------------------------------------------------------------

// Eq. 4 on one sign-extended anchor element: shift the magnitude right by de, round on the most
// significant dropped bit, clip, restore the sign.
template <class FH, class FL>
__device__ __forceinline__ uint32_t ss_int_elem(uint32_t code)
{
    constexpr int de = FH::emax - FL::emax;
    int32_t p = (int32_t)(code << (32 - FH::bits)) >> (32 - FH::bits);
    uint32_t mag = (uint32_t)(p < 0 ? -p : p);
    uint32_t q = de > 0 ? (mag + (1u << (de > 0 ? de - 1 : 0))) >> de : mag;
    q = min(q, FL::max_mag);
    return (p < 0 ? 0u - q : q) & FL::mask;
}

// Eq. 5 on one anchor element: decode, divide by 2^de (exact), quantize to the low format.
// An E4M3 NaN code maps to the sign-preserved largest magnitude.
template <class FH, class FL>
__device__ __forceinline__ uint32_t ss_fp_elem(uint32_t code)
{
    constexpr int de = FH::emax - FL::emax;
    uint32_t mag = code & ((1u << (FH::bits - 1)) - 1u);
    uint32_t sign = code >> (FH::bits - 1);
    if (FH::has_nan && mag > FH::max_mag) return FL::max_mag | (sign << (FL::bits - 1));
    float x = decode<FH>(code) * __uint_as_float((uint32_t)(127 - de) << 23);
    return quantize_fp_alu<FL>(x);
}

}  // namespace mxq
