/*
 * mxq_oracle.c -- CPU oracle for block-wise microscaling (MX) quantization and the
 * Slice-and-Scale conversions of MF-QAT.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, scalar restatement of the
 * paper's equations, used only to check the CUDA library and to serve as the timed
 * CPU baseline of the bench.  It shares no code, header, table or constant with the
 * CUDA path and must never be called from a product code path.
 *
 * Arithmetic: every real number is held in a C `double`.  All inputs are FP32 or BF16
 * (at most 24 significant bits) and every scaling is by a power of two through
 * ldexp(), so each intermediate value below is exact; the only roundings are the ones
 * the method itself defines (Round / quantize) and the final store of a dequantized
 * value into FP32 or BF16.
 *
 * Paper passages followed (section / equation numbering in order of appearance):
 *   Eq. 1  (Sec. 3.3)  shared_exp = floor(log2 max|V_i|) - e_max(f),  X = 2^shared_exp
 *   Eq. 2  (Sec. 3.3)  P_i = quantize_f(V_i / X)
 *   Eq. 3  (Sec. 3.3)  MXINT: P_i = clip_b(Round(V_i / X))
 *   Eq. 4  (Sec. 3.3)  SSMXINT: P_l = clip_bl(Round(P_h / 2^de)), X_l = X_h 2^de, de = b_h - b_l
 *   Eq. 5  (Sec. 3.4)  SSMXFP : P_l = quantize_{eta_l,mu_l}(P_h / 2^de), X_l = X_h 2^de,
 *                      de = e_max(eta_h) - e_max(eta_l)
 *   Eq. 6  (Sec. 3.5)  W_A = Q_A(W_fp), W_t = Q_{A->t}(W_A)
 *   Sec. 3.3 Notation  reconstruction V^_i = X * P_i
 *
 * Readings taken where the paper is silent (each is listed with its reason in the
 * repository's design notes):
 *   - e_max(MXINT b) = b - 2 (P is a plain integer; 2^(b-2) <= |P|max < 2^(b-1)).
 *   - clip_b is symmetric: [-(2^(b-1)-1), +(2^(b-1)-1)].
 *   - Round for MXINT = nearest, ties away from zero (the Sec. 3.3 bit procedure
 *     "round using the most-significant dropped bit", applied to the magnitude).
 *   - quantize_{eta,mu} = round-to-nearest-even onto the element grid (subnormals
 *     kept), then saturation to the largest finite magnitude; the sign of a value
 *     that rounds to zero is kept.
 *   - the scale is stored as an E8M0 byte = shared_exp + 127, shared_exp clamped to
 *     [-127, 127]; an all-zero block gets byte 0; a block holding NaN or Inf gets
 *     byte 0xFF and all-zero codes, and dequantizes to NaN.
 *   - FP8 E4M3 follows the OCP encoding (S.1111.111 is NaN, no infinities); every
 *     other MXFP element format has no special codes.
 *
 * Parity pins (tests/test_oracle_*.py): exhaustive code tables against ml_dtypes /
 * torch casts and published value sets, the element quantizer against an
 * exact-rational brute-force nearest-neighbour search, hand-worked blocks in
 * tests/golden/, and the invariants that follow from Eq. 1-5.  Readings the paper
 * does not fix (listed above) are "parity unpinned" with respect to the authors'
 * unpublished code; they are pinned only to the definitions written here.
 *
 * Codes are exchanged ONE CODE PER BYTE (low `bits` bits used); mxo_pack / mxo_unpack
 * convert to and from the packed little-endian bitstream layout.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Element format descriptor                                                  */
/* ------------------------------------------------------------------------- */

/* kind 0: MXINT(b): a = b (2..8), m unused.   kind 1: MXFP: a = eta, m = mu. */
typedef struct {
    int kind;
    int a;
    int m;
} mxo_fmt;

enum { MXO_INT = 0, MXO_FP = 1 };
enum { MXO_F32 = 0, MXO_BF16 = 1 };
enum { MXO_FQ_DIRECT = 0, MXO_FQ_VIA_ANCHOR = 1 };

static int fmt_bits(mxo_fmt f) { return f.kind == MXO_INT ? f.a : 1 + f.a + f.m; }
static int fp_bias(mxo_fmt f) { return (1 << (f.a - 1)) - 1; }
/* OCP FP8 E4M3 is the only element format here with a NaN encoding. */
static int fp_has_nan(mxo_fmt f) { return f.kind == MXO_FP && f.a == 4 && f.m == 3; }

/* e_max(f): exponent of the largest normal number of the element format (Sec. 3.3
 * Notation).  MXINT(b): largest magnitude 2^(b-1)-1 has exponent b-2.  MXFP: the top
 * exponent code holds normal numbers in every format used here, so
 * e_max = (2^eta - 1) - bias = 2^(eta-1). */
int mxo_emax(int kind, int a, int m)
{
    (void)m;
    return kind == MXO_INT ? a - 2 : (1 << (a - 1));
}

/* Largest finite magnitude of the element format. */
double mxo_max_value(int kind, int a, int m)
{
    mxo_fmt f = { kind, a, m };
    if (kind == MXO_INT) return (double)((1 << (a - 1)) - 1);
    int emax = mxo_emax(kind, a, m);
    if (fp_has_nan(f)) /* top mantissa code of the top binade is NaN */
        return ldexp(2.0 - 2.0 * ldexp(1.0, -m), emax);
    return ldexp(2.0 - ldexp(1.0, -m), emax);
}

/* ------------------------------------------------------------------------- */
/* Element decode: code -> real value P                                       */
/* ------------------------------------------------------------------------- */

/* MXINT: two's-complement b-bit integer.  MXFP: sign | exponent(eta) | mantissa(mu),
 * E > 0: (-1)^s 2^(E-bias) (1 + M/2^mu);  E = 0: (-1)^s 2^(1-bias) M/2^mu. */
double mxo_decode(int kind, int a, int m, unsigned code)
{
    mxo_fmt f = { kind, a, m };
    int bits = fmt_bits(f);
    code &= (1u << bits) - 1u;
    if (kind == MXO_INT) {
        int q = (int)code;
        if (q >= (1 << (bits - 1))) q -= (1 << bits);
        return (double)q;
    }
    int s = (int)(code >> (bits - 1)) & 1;
    int E = (int)(code >> m) & ((1 << a) - 1);
    int M = (int)code & ((1 << m) - 1);
    if (fp_has_nan(f) && E == (1 << a) - 1 && M == (1 << m) - 1) return NAN;
    int bias = fp_bias(f);
    double mag;
    if (E > 0)
        mag = ldexp(1.0 + ldexp((double)M, -m), E - bias);
    else
        mag = ldexp(ldexp((double)M, -m), 1 - bias);
    return s ? -mag : mag;
}

/* ------------------------------------------------------------------------- */
/* Element quantizers: real r = V/X -> code (Eq. 2, Eq. 3)                    */
/* ------------------------------------------------------------------------- */

/* floor(log2 a) for finite a > 0, exact: frexp gives a = m 2^E with m in [0.5,1). */
static int floor_log2(double a)
{
    int E;
    (void)frexp(a, &E);
    return E - 1;
}

/* Eq. 3: P = clip_b(Round(r)); Round = nearest, ties away from zero; symmetric clip. */
static unsigned quantize_int(mxo_fmt f, double r)
{
    int b = f.a;
    double a = fabs(r);
    double q = floor(a);
    if (a - q >= 0.5) q += 1.0; /* a - floor(a) is exact */
    double lim = (double)((1 << (b - 1)) - 1);
    if (q > lim) q = lim;
    int qi = (int)q;
    if (r < 0) qi = -qi;
    return (unsigned)qi & ((1u << b) - 1u);
}

/* quantize_{eta,mu}(r): round-to-nearest-even onto the element grid, saturate. */
static unsigned quantize_fp(mxo_fmt f, double r)
{
    int eta = f.a, mu = f.m, bits = fmt_bits(f), bias = fp_bias(f);
    unsigned s = signbit(r) ? 1u : 0u;
    double a = fabs(r);
    if (a == 0.0) return s << (bits - 1);
    int ea = floor_log2(a);
    if (ea < 1 - bias) ea = 1 - bias;           /* subnormal range shares one ulp */
    double m = nearbyint(ldexp(a, mu - ea));    /* a / ulp, ulp = 2^(ea-mu); ties to even */
    double v = ldexp(m, ea - mu);
    double vmax = mxo_max_value(f.kind, eta, mu);
    if (v > vmax) v = vmax;                     /* clamping */
    unsigned E, M;
    if (v == 0.0) {
        E = 0; M = 0;
    } else {
        int ev = floor_log2(v);                 /* re-derive after a possible carry */
        if (ev < 1 - bias) {
            E = 0;
            M = (unsigned)ldexp(v, mu - (1 - bias));
        } else {
            E = (unsigned)(ev + bias);
            M = (unsigned)ldexp(ldexp(v, -ev) - 1.0, mu);
        }
    }
    return (s << (bits - 1)) | (E << mu) | M;
}

/* quantize_f for one already-scaled real number (exported for the element pins). */
unsigned mxo_quantize_elem(int kind, int a, int m, double r)
{
    mxo_fmt f = { kind, a, m };
    return kind == MXO_INT ? quantize_int(f, r) : quantize_fp(f, r);
}

/* ------------------------------------------------------------------------- */
/* Input / output element types                                               */
/* ------------------------------------------------------------------------- */

static double load_elem(const void *src, int dtype, size_t i)
{
    if (dtype == MXO_F32) return (double)((const float *)src)[i];
    uint32_t w = (uint32_t)((const uint16_t *)src)[i] << 16; /* BF16 = top half of FP32 */
    float x;
    memcpy(&x, &w, 4);
    return (double)x;
}

/* One round-to-nearest-even rounding of a double to BF16 (8 significant bits,
 * exponent range of FP32, subnormals kept, overflow to infinity). */
static uint16_t double_to_bf16(double v)
{
    uint16_t s = signbit(v) ? 0x8000u : 0u;
    if (isnan(v)) return 0x7FC0u;
    double a = fabs(v);
    if (isinf(a)) return s | 0x7F80u;
    if (a == 0.0) return s;
    int e = floor_log2(a);
    if (e < -126) e = -126;
    double m = nearbyint(ldexp(a, 7 - e));      /* in units of 2^(e-7) */
    double r = ldexp(m, e - 7);
    if (r >= ldexp(1.0, 128)) return s | 0x7F80u;
    if (r == 0.0) return s;
    int er = floor_log2(r);
    if (er < -126) return s | (uint16_t)ldexp(r, 133);                 /* subnormal */
    unsigned frac = (unsigned)ldexp(ldexp(r, -er) - 1.0, 7);
    return s | (uint16_t)(((unsigned)(er + 127) << 7) | frac);
}

static void store_elem(void *dst, int dtype, size_t i, double v)
{
    if (dtype == MXO_F32) {
        float x = (float)v;                     /* C cast: one RNE rounding */
        if (isnan(v)) { uint32_t q = 0x7FC00000u; memcpy(&x, &q, 4); }
        ((float *)dst)[i] = x;
    } else {
        ((uint16_t *)dst)[i] = double_to_bf16(v);
    }
}

/* ------------------------------------------------------------------------- */
/* Block quantizer Q_f (Eq. 1-3)                                              */
/* ------------------------------------------------------------------------- */

/* V[0..k) -> codes[0..k) (one per byte) and one E8M0 scale byte. */
static void quantize_block(const double *V, int k, mxo_fmt f, uint8_t *codes, uint8_t *scale)
{
    double amax = 0.0;
    for (int i = 0; i < k; ++i) {
        if (isnan(V[i]) || isinf(V[i])) {       /* poisoned block */
            *scale = 0xFF;
            memset(codes, 0, (size_t)k);
            return;
        }
        if (fabs(V[i]) > amax) amax = fabs(V[i]);
    }
    int shared_exp;
    if (amax == 0.0) {
        shared_exp = -127;
    } else {
        shared_exp = floor_log2(amax) - mxo_emax(f.kind, f.a, f.m);      /* Eq. 1 */
        if (shared_exp < -127) shared_exp = -127;
        if (shared_exp > 127) shared_exp = 127;
    }
    *scale = (uint8_t)(shared_exp + 127);
    for (int i = 0; i < k; ++i) {
        double r = ldexp(V[i], -shared_exp);                              /* V_i / X */
        codes[i] = (uint8_t)mxo_quantize_elem(f.kind, f.a, f.m, r);       /* Eq. 2-3 */
    }
}

int mxo_quantize(const void *src, int dtype, size_t n, int kind, int a, int m, int block,
                 uint8_t *codes, uint8_t *scales)
{
    if (block <= 0 || block > 1024 || n % (size_t)block) return -1;
    mxo_fmt f = { kind, a, m };
    double V[1024];
    for (size_t b = 0; b < n / (size_t)block; ++b) {
        for (int i = 0; i < block; ++i) V[i] = load_elem(src, dtype, b * block + i);
        quantize_block(V, block, f, codes + b * block, scales + b);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Slice-and-Scale Q_{h->l} (Eq. 4, Eq. 5)                                    */
/* ------------------------------------------------------------------------- */

/* One element.  MXINT: drop de low bits of the magnitude, round on the most
 * significant dropped bit, clip (Eq. 4 and the bit procedure under it).
 * MXFP: decode, divide by 2^de (exact), quantize to the low format (Eq. 5).
 * An E4M3 NaN code (never produced by the quantizer) maps to the sign-preserved
 * largest magnitude of the low format. */
unsigned mxo_slice_scale_elem(int kind, int ah, int mh, int al, int ml, unsigned code)
{
    mxo_fmt fh = { kind, ah, mh }, fl = { kind, al, ml };
    int de = mxo_emax(kind, ah, mh) - mxo_emax(kind, al, ml);
    if (de == 0 && ah == al && mh == ml) return code & ((1u << fmt_bits(fh)) - 1u);
    if (kind == MXO_INT) {
        int p = (int)mxo_decode(kind, ah, mh, code);
        int mag = p < 0 ? -p : p;
        int q = de > 0 ? (mag + (1 << (de - 1))) >> de : mag;
        int lim = (1 << (al - 1)) - 1;
        if (q > lim) q = lim;
        if (p < 0) q = -q;
        return (unsigned)q & ((1u << al) - 1u);
    }
    double x = mxo_decode(kind, ah, mh, code);
    if (isnan(x)) {
        unsigned s = (code >> (fmt_bits(fh) - 1)) & 1u;
        double big = mxo_max_value(kind, al, ml);
        return quantize_fp(fl, s ? -big : big);
    }
    return quantize_fp(fl, ldexp(x, -de));
}

int mxo_slice_scale(const uint8_t *codes_h, const uint8_t *scales_h, size_t n, int block,
                    int kind, int ah, int mh, int al, int ml,
                    uint8_t *codes_l, uint8_t *scales_l)
{
    if (block <= 0 || n % (size_t)block) return -1;
    int de = mxo_emax(kind, ah, mh) - mxo_emax(kind, al, ml);
    if (de < 0) return -2;
    for (size_t b = 0; b < n / (size_t)block; ++b) {
        unsigned sh = scales_h[b];
        unsigned sl = sh == 0xFF ? 0xFF : (sh + (unsigned)de > 254 ? 254 : sh + (unsigned)de);
        scales_l[b] = (uint8_t)sl;                                        /* X_l = X_h 2^de */
        for (int i = 0; i < block; ++i)
            codes_l[b * block + i] =
                (uint8_t)mxo_slice_scale_elem(kind, ah, mh, al, ml, codes_h[b * block + i]);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Reconstruction V^_i = X P_i (Sec. 3.3 Notation)                            */
/* ------------------------------------------------------------------------- */

int mxo_dequantize(const uint8_t *codes, const uint8_t *scales, size_t n, int kind, int a, int m,
                   int block, void *dst, int dtype)
{
    if (block <= 0 || n % (size_t)block) return -1;
    for (size_t b = 0; b < n / (size_t)block; ++b) {
        for (int i = 0; i < block; ++i) {
            size_t j = b * block + i;
            double v;
            if (scales[b] == 0xFF)
                v = NAN;
            else
                v = ldexp(mxo_decode(kind, a, m, codes[j]), (int)scales[b] - 127);
            store_elem(dst, dtype, j, v);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Fake-quant forward (Eq. 6) and straight-through backward                   */
/* ------------------------------------------------------------------------- */

/* DIRECT: dequantize(Q_f(V)).  VIA_ANCHOR: dequantize(Q_{A->f}(Q_A(V))) with A the
 * 8-bit anchor of f's family (MXINT8 or MXFP8 E4M3).  Output type = input type. */
int mxo_fake_quant(const void *src, int dtype, size_t n, int kind, int a, int m, int block,
                   int mode, void *dst)
{
    if (block <= 0 || block > 1024 || n % (size_t)block) return -1;
    mxo_fmt f = { kind, a, m };
    mxo_fmt A = kind == MXO_INT ? (mxo_fmt){ MXO_INT, 8, 0 } : (mxo_fmt){ MXO_FP, 4, 3 };
    double V[1024];
    uint8_t ch[1024], cl[1024], sh, sl;
    for (size_t b = 0; b < n / (size_t)block; ++b) {
        for (int i = 0; i < block; ++i) V[i] = load_elem(src, dtype, b * block + i);
        if (mode == MXO_FQ_VIA_ANCHOR) {
            quantize_block(V, block, A, ch, &sh);                         /* W_A = Q_A(W_fp) */
            mxo_slice_scale(ch, &sh, (size_t)block, block, kind, A.a, A.m, a, m, cl, &sl);
        } else {
            quantize_block(V, block, f, cl, &sl);
        }
        /* dequantize into the caller's buffer at this block's offset */
        size_t esz = dtype == MXO_F32 ? 4 : 2;
        mxo_dequantize(cl, &sl, (size_t)block, kind, a, m, block,
                       (char *)dst + b * block * esz, dtype);
    }
    return 0;
}

/* Straight-through estimator: the gradient passes unchanged (Sec. 3.5). */
int mxo_fake_quant_bwd(const void *grad_out, int dtype, size_t n, void *grad_in)
{
    memmove(grad_in, grad_out, n * (dtype == MXO_F32 ? 4u : 2u));
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Scale bytes in the tiled order of a block-scaled matrix multiply           */
/* ------------------------------------------------------------------------- */

/* [rows, kblocks] row-major -> tiles of 128 rows x 4 columns, 512 bytes each, tiles ordered
 * row-tile by row-tile; inside a tile the byte of (r, c) sits at (r mod 32)*16 + (r div 32)*4 + c.
 * Bytes that no (r, c) of the matrix maps to are 0.  `out` holds
 * ceil(rows/128) * ceil(kblocks/4) * 512 bytes. */
int mxo_tile_scales(const uint8_t *scales, size_t rows, size_t kblocks, uint8_t *out)
{
    size_t col_tiles = (kblocks + 3) / 4, row_tiles = (rows + 127) / 128;
    memset(out, 0, row_tiles * col_tiles * 512);
    for (size_t r = 0; r < rows; ++r)
        for (size_t c = 0; c < kblocks; ++c) {
            size_t tile = (r / 128) * col_tiles + c / 4;
            size_t rr = r % 128, cc = c % 4;
            out[tile * 512 + (rr % 32) * 16 + (rr / 32) * 4 + cc] = scales[r * kblocks + c];
        }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Packed storage: little-endian bitstream, element i at bits [i*bits,(i+1)*bits) */
/* ------------------------------------------------------------------------- */

int mxo_pack(const uint8_t *codes, size_t n, int bits, uint8_t *out)
{
    if ((n * (size_t)bits) % 8) return -1;
    memset(out, 0, n * (size_t)bits / 8);
    for (size_t i = 0; i < n; ++i)
        for (int j = 0; j < bits; ++j)
            if ((codes[i] >> j) & 1u) {
                size_t bit = i * (size_t)bits + (size_t)j;
                out[bit >> 3] |= (uint8_t)(1u << (bit & 7));
            }
    return 0;
}

int mxo_unpack(const uint8_t *packed, size_t n, int bits, uint8_t *codes)
{
    for (size_t i = 0; i < n; ++i) {
        unsigned c = 0;
        for (int j = 0; j < bits; ++j) {
            size_t bit = i * (size_t)bits + (size_t)j;
            c |= (unsigned)((packed[bit >> 3] >> (bit & 7)) & 1u) << j;
        }
        codes[i] = (uint8_t)c;
    }
    return 0;
}
