/* The host-side argument checks of libmxq under AddressSanitizer / UBSan: this program links a build
 * of the library whose C ABI layer (argument validation, item-table construction) is compiled with
 * -fsanitize=address,undefined and walks the error paths that return before any CUDA call -- bad
 * enums, null and misaligned pointers, sizes that are not whole blocks, illegal format pairs, item
 * arrays (on the heap, exactly sized) with a bad entry at the end.  No GPU is needed.  Prints "ok". */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "../../include/mxq.h"

#define EXPECT(call, want)                                                     \
    do {                                                                       \
        int got_ = (call);                                                     \
        if (got_ != (want)) {                                                  \
            printf("line %d: %s returned %d, expected %d\n", __LINE__, #call, got_, (int)(want)); \
            return 1;                                                          \
        }                                                                      \
    } while (0)

int main(void)
{
    void *A = (void *)(uintptr_t)0x10000;          /* an aligned, never dereferenced "device" address */
    void *M = (void *)(uintptr_t)0x10008;          /* misaligned for every buffer kind */
    EXPECT(mxq_quantize(A, MXQ_BF16, 64, 99, 32, A, A, NULL), MXQ_ERR_FORMAT);
    EXPECT(mxq_quantize(A, 7, 64, MXQ_INT8, 32, A, A, NULL), MXQ_ERR_FORMAT);
    EXPECT(mxq_quantize(A, MXQ_BF16, 64, MXQ_INT8, 48, A, A, NULL), MXQ_ERR_BLOCK);
    EXPECT(mxq_quantize(A, MXQ_BF16, 65, MXQ_INT8, 32, A, A, NULL), MXQ_ERR_SIZE);
    EXPECT(mxq_quantize(NULL, MXQ_BF16, 64, MXQ_INT8, 32, A, A, NULL), MXQ_ERR_NULL);
    EXPECT(mxq_quantize(M, MXQ_BF16, 64, MXQ_INT8, 32, A, A, NULL), MXQ_ERR_ALIGN);
    EXPECT(mxq_quantize(NULL, MXQ_BF16, 0, MXQ_INT8, 32, NULL, NULL, NULL), MXQ_OK);
    EXPECT(mxq_slice_scale(A, A, 64, 32, MXQ_INT8, MXQ_FP4_E2M1, A, A, NULL), MXQ_ERR_PAIR);
    EXPECT(mxq_slice_scale(A, A, 64, 32, MXQ_INT4, MXQ_INT8, A, A, NULL), MXQ_ERR_PAIR);
    EXPECT(mxq_slice_scale(A, A, 48, 16, MXQ_INT8, MXQ_INT4, A, A, NULL), MXQ_ERR_SIZE);
    EXPECT(mxq_slice_scale(A, NULL, 64, 32, MXQ_INT8, MXQ_INT4, A, A, NULL), MXQ_ERR_NULL);
    EXPECT(mxq_slice_scale(A, A, 64, 32, MXQ_INT8, MXQ_INT4, M, A, NULL), MXQ_ERR_ALIGN);
    EXPECT(mxq_dequantize(A, A, 64, MXQ_INT4, 32, A, 9, NULL), MXQ_ERR_FORMAT);
    EXPECT(mxq_dequantize(A, A, 64, MXQ_INT4, 32, NULL, MXQ_F32, NULL), MXQ_ERR_NULL);
    EXPECT(mxq_fake_quant(A, MXQ_BF16, 64, MXQ_FP4_E2M1, 32, 2, A, NULL), MXQ_ERR_FORMAT);
    EXPECT(mxq_fake_quant(A, MXQ_BF16, 64, MXQ_FP4_E2M1, 32, MXQ_FQ_DIRECT, M, NULL), MXQ_ERR_ALIGN);
    EXPECT(mxq_fake_quant_bwd(A, MXQ_BF16, 64, A, NULL), MXQ_OK);          /* in place: nothing to do */
    EXPECT(mxq_fake_quant_bwd(A, MXQ_BF16, 64, NULL, NULL), MXQ_ERR_NULL);
    {
        int fmts[2] = {MXQ_INT6, MXQ_FP4_E2M1};
        void *oc[2] = {A, A};
        uint8_t *os[2] = {A, A};
        EXPECT(mxq_slice_scale_multi(A, A, 64, 32, MXQ_INT8, 2, fmts, oc, os, NULL), MXQ_ERR_PAIR);
        EXPECT(mxq_slice_scale_multi(A, A, 64, 32, MXQ_INT8, 9, fmts, oc, os, NULL), MXQ_ERR_SIZE);
        fmts[1] = MXQ_INT4;
        oc[1] = NULL;
        EXPECT(mxq_slice_scale_multi(A, A, 64, 32, MXQ_INT8, 2, fmts, oc, os, NULL), MXQ_ERR_NULL);
    }
    /* item arrays: many good entries, the bad one last, so the whole array is walked */
    const int count = 700;
    {
        mxq_ss_item *it = malloc(sizeof(mxq_ss_item) * count);
        for (int i = 0; i < count; ++i) it[i] = (mxq_ss_item){A, A, 64, A, A};
        it[count - 1].n = 65;
        EXPECT(mxq_slice_scale_batched(it, count, 32, MXQ_INT8, MXQ_INT4, NULL), MXQ_ERR_SIZE);
        EXPECT(mxq_slice_scale_batched_static(it, count, 32, MXQ_INT8, MXQ_INT4, NULL), MXQ_ERR_SIZE);
        it[count - 1] = (mxq_ss_item){A, A, 64, M, A};
        EXPECT(mxq_slice_scale_batched(it, count, 32, MXQ_INT8, MXQ_INT4, NULL), MXQ_ERR_ALIGN);
        EXPECT(mxq_slice_scale_batched_static(it, count, 32, MXQ_INT8, MXQ_INT4, NULL), MXQ_ERR_ALIGN);
        EXPECT(mxq_slice_scale_batched_static(it, MXQ_STATIC_BATCH_MAX + 1, 32, MXQ_INT8, MXQ_INT4, NULL), MXQ_ERR_SIZE);
        free(it);
    }
    {
        mxq_fq_item *it = malloc(sizeof(mxq_fq_item) * count);
        for (int i = 0; i < count; ++i) it[i] = (mxq_fq_item){A, A, 64};
        it[count - 1].dst = NULL;
        EXPECT(mxq_fake_quant_batched(it, count, MXQ_BF16, MXQ_INT4, 32, MXQ_FQ_VIA_ANCHOR, NULL), MXQ_ERR_NULL);
        free(it);
    }
    {
        mxq_q_item *it = malloc(sizeof(mxq_q_item) * count);
        for (int i = 0; i < count; ++i) it[i] = (mxq_q_item){A, 64, A, A};
        it[count - 1].scales = M;
        EXPECT(mxq_quantize_batched(it, count, MXQ_F32, MXQ_FP8_E4M3, 32, NULL), MXQ_ERR_ALIGN);
        free(it);
    }
    {
        mxq_dq_item *it = malloc(sizeof(mxq_dq_item) * count);
        for (int i = 0; i < count; ++i) it[i] = (mxq_dq_item){A, A, 64, A};
        it[count - 1].n = 16;
        EXPECT(mxq_dequantize_batched(it, count, MXQ_INT4, 16, MXQ_BF16, NULL), MXQ_ERR_SIZE);
        free(it);
    }
    {
        mxq_ss_tiled_item *it = malloc(sizeof(mxq_ss_tiled_item) * 300);
        for (int i = 0; i < 300; ++i) it[i] = (mxq_ss_tiled_item){A, A, 2, 64, A, A};
        it[299].cols = 48;
        EXPECT(mxq_slice_scale_tiled_batched(it, 300, 32, MXQ_FP8_E4M3, MXQ_FP4_E2M1, NULL), MXQ_ERR_SIZE);
        free(it);
    }
    EXPECT(mxq_tile_scales(A, 0, 4, A, NULL), MXQ_OK);
    EXPECT(mxq_tile_scales(NULL, 4, 4, A, NULL), MXQ_ERR_NULL);
    if (mxq_tiled_scales_bytes(129, 5) != 2 * 2 * 512 || mxq_codes_bytes(64, MXQ_INT6) != 48 || mxq_scales_bytes(64, 32) != 2) return 1;
    if (!mxq_status_string(MXQ_ERR_PAIR) || !mxq_status_string(12345)) return 1;
    puts("ok");
    return 0;
}
