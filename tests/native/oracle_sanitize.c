/* Runs every entry point of the CPU oracle (oracle/mxq_oracle.c, compiled into this program with
 * -fsanitize=address,undefined) on exactly sized heap buffers: adversarial FP32 blocks (zeros,
 * subnormals, FLT_MAX, NaN, Inf), every element format, every legal Slice-and-Scale pair, all byte
 * values as codes and as scale bytes, blocks of 16 / 32 / 64 / 128.  Any out-of-bounds access, signed
 * overflow, bad shift or misaligned access aborts the program; it prints "ok" at the end. */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

int mxo_emax(int kind, int a, int m);
int mxo_quantize(const void *src, int dtype, size_t n, int kind, int a, int m, int block, uint8_t *codes, uint8_t *scales);
int mxo_slice_scale(const uint8_t *codes_h, const uint8_t *scales_h, size_t n, int block, int kind, int ah, int mh,
                    int al, int ml, uint8_t *codes_l, uint8_t *scales_l);
int mxo_dequantize(const uint8_t *codes, const uint8_t *scales, size_t n, int kind, int a, int m, int block, void *dst,
                   int dtype);
int mxo_fake_quant(const void *src, int dtype, size_t n, int kind, int a, int m, int block, int mode, void *dst);
int mxo_fake_quant_bwd(const void *grad_out, int dtype, size_t n, void *grad_in);
int mxo_tile_scales(const uint8_t *scales, size_t rows, size_t kblocks, uint8_t *out);
int mxo_pack(const uint8_t *codes, size_t n, int bits, uint8_t *out);
int mxo_unpack(const uint8_t *packed, size_t n, int bits, uint8_t *codes);

static const int FORMATS[13][3] = {{0, 8, 0}, {0, 7, 0}, {0, 6, 0}, {0, 5, 0}, {0, 4, 0}, {0, 3, 0}, {0, 2, 0},
                                   {1, 4, 3}, {1, 3, 3}, {1, 3, 2}, {1, 2, 3}, {1, 2, 2}, {1, 2, 1}};

static int bits_of(const int *f) { return f[0] == 0 ? f[1] : 1 + f[1] + f[2]; }

int main(void)
{
    const size_t n = 128 * 24;
    float *x = malloc(n * sizeof(float));
    uint16_t *xb = malloc(n * sizeof(uint16_t));
    const float special[] = {0.0f, -0.0f, 1.0f, -1.0f, 3.4028235e38f, -3.4028235e38f, 1e-45f, -1e-45f, 1.1754944e-38f,
                             5.8774718e-39f, 0.5f, 1.5f, 2.5f, 127.5f, 448.0f, 464.0f, 480.0f, 6.0f, 7.5f, 28.0f, 1e-30f};
    uint32_t r = 7;
    for (size_t i = 0; i < n; ++i) {
        r = r * 1664525u + 1013904223u;
        if (i < 128 * 4) x[i] = special[r % (sizeof special / sizeof special[0])];
        else x[i] = ldexpf((float)((int)(r >> 8) % 2001 - 1000) / 1000.0f, (int)(r % 61) - 30);
    }
    x[128 * 5 + 3] = NAN;
    x[128 * 6 + 9] = INFINITY;
    x[128 * 7 + 0] = -INFINITY;
    for (size_t i = 0; i < n; ++i) {
        uint32_t u;
        memcpy(&u, &x[i], 4);
        xb[i] = (uint16_t)(u >> 16);
    }
    const int blocks[] = {16, 32, 64, 128};
    for (int bi = 0; bi < 4; ++bi) {
        const int block = blocks[bi];
        for (int fi = 0; fi < 13; ++fi) {
            const int *f = FORMATS[fi];
            const int b = bits_of(f);
            uint8_t *codes = malloc(n), *scales = malloc(n / block), *packed = malloc(n * b / 8), *again = malloc(n);
            float *y = malloc(n * 4);
            uint16_t *yb = malloc(n * 2);
            for (int dtype = 0; dtype < 2; ++dtype) {
                const void *src = dtype == 0 ? (const void *)x : (const void *)xb;
                if (mxo_quantize(src, dtype, n, f[0], f[1], f[2], block, codes, scales)) return 2;
                if (mxo_pack(codes, n, b, packed) || mxo_unpack(packed, n, b, again) || memcmp(codes, again, n)) return 3;
                if (mxo_dequantize(codes, scales, n, f[0], f[1], f[2], block, y, 0)) return 4;
                if (mxo_dequantize(codes, scales, n, f[0], f[1], f[2], block, yb, 1)) return 4;
                for (int mode = 0; mode < 2; ++mode)
                    if (mxo_fake_quant(src, dtype, n, f[0], f[1], f[2], block, mode, dtype == 0 ? (void *)y : (void *)yb)) return 5;
                if (mxo_fake_quant_bwd(dtype == 0 ? (void *)y : (void *)yb, dtype, n, dtype == 0 ? (void *)y : (void *)yb)) return 6;
            }
            /* every byte value as a code of this format (masked to its width) and as a scale byte */
            for (size_t i = 0; i < n; ++i) codes[i] = (uint8_t)(i & ((1u << b) - 1u));
            for (size_t i = 0; i < n / block; ++i) scales[i] = (uint8_t)(i * 37u + 250u);
            if (mxo_dequantize(codes, scales, n, f[0], f[1], f[2], block, y, 0)) return 7;
            if (mxo_dequantize(codes, scales, n, f[0], f[1], f[2], block, yb, 1)) return 7;
            for (int li = 0; li < 13; ++li) {
                const int *l = FORMATS[li];
                if (l[0] != f[0] || bits_of(l) > b || mxo_emax(l[0], l[1], l[2]) > mxo_emax(f[0], f[1], f[2])) continue;
                uint8_t *lc = malloc(n), *ls = malloc(n / block);
                if (mxo_slice_scale(codes, scales, n, block, f[0], f[1], f[2], l[1], l[2], lc, ls)) return 8;
                free(lc);
                free(ls);
            }
            free(codes); free(scales); free(packed); free(again); free(y); free(yb);
        }
    }
    /* the tiled scale order: matrices that do and do not cover whole 128 x 4 tiles */
    const size_t shapes[][2] = {{128, 4}, {1, 1}, {129, 5}, {300, 7}, {256, 8}};
    for (int s = 0; s < 5; ++s) {
        const size_t rows = shapes[s][0], kb = shapes[s][1];
        uint8_t *in = malloc(rows * kb), *out = malloc(((rows + 127) / 128) * ((kb + 3) / 4) * 512);
        for (size_t i = 0; i < rows * kb; ++i) in[i] = (uint8_t)i;
        if (mxo_tile_scales(in, rows, kb, out)) return 9;
        free(in);
        free(out);
    }
    free(x);
    free(xb);
    puts("ok");
    return 0;
}
