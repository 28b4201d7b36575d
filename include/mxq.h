/*
 * mxq.h -- C ABI of libmxq: block-wise microscaling (MX) quantization, Slice-and-Scale
 * conversion, reconstruction and fused fake-quant for MF-QAT, as CUDA kernels for sm_100a.
 *
 * Method (section / equation numbers of the MF-QAT paper, equations counted in order of
 * appearance):
 *   Eq. 1  (Sec. 3.3)  shared_exp = floor(log2 max_i |V_i|) - e_max(f),  X = 2^shared_exp
 *   Eq. 2-3 (Sec. 3.3) P_i = quantize_f(V_i / X);  MXINT: P_i = clip_b(Round(V_i / X))
 *   Eq. 4  (Sec. 3.3)  SSMXINT: P_l = clip(Round(P_h / 2^de)),  X_l = X_h 2^de,  de = b_h - b_l
 *   Eq. 5  (Sec. 3.4)  SSMXFP:  P_l = quantize_{eta_l,mu_l}(P_h / 2^de),  X_l = X_h 2^de,
 *                      de = e_max(eta_h) - e_max(eta_l)
 *   Eq. 6  (Sec. 3.5)  W_A = Q_A(W_fp),  W_t = Q_{A->t}(W_A), straight-through gradients
 *   reconstruction (Sec. 3.3, Notation)  V^_i = X P_i
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers owned by the caller.  Tensor and code buffers
 *     (src, dst, codes, out_codes, grad_*) must be 32-byte aligned (the kernels use 256-bit
 *     global accesses); scale buffers must be 16-byte aligned.  The library enqueues work on
 *     `stream` and returns without synchronising.  Unless an entry point says otherwise it
 *     allocates nothing and copies nothing (mxq_slice_scale_batched_static copies its item table).
 *   - Work goes to the CURRENT device, which must be the one the pointers belong to.  Kernels
 *     are launched with programmatic stream serialization allowed, so that a kernel's blocks
 *     can become resident while the previous kernel of the stream drains; each kernel waits
 *     for that previous kernel to complete before its first load or store, so the ordering a
 *     stream guarantees is unchanged for every buffer.  (Before that wait a kernel may issue
 *     L2 prefetches for its input buffers, which return no data; the input pointers must
 *     therefore be valid device addresses when the call is made, as they must be anyway.)
 *   - `n` is the number of elements; it must be a multiple of `block`.  Blocks are runs
 *     of `block` consecutive elements of the flat array (for a row-major matrix whose inner
 *     dimension is a multiple of `block`: along the row).  n == 0 returns MXQ_OK at once.
 *     The entry points that read packed codes (mxq_slice_scale and its multi / batched forms,
 *     mxq_dequantize) also need n to be a multiple of 32, which only matters for block 16.
 *   - The return value is an mxq_status.  Errors detectable on the host (bad enum, null
 *     or misaligned pointer, bad size) are reported before anything is launched;
 *     MXQ_ERR_CUDA reports a failed launch (cudaGetLastError()).
 *   - Scales: uint8 scales[n / block], E8M0: byte = shared_exp + 127 with shared_exp
 *     clamped to [-127, 127]; an all-zero block stores 0; a block that holds a NaN or an
 *     infinity stores 0xFF with all-zero codes, stays 0xFF through mxq_slice_scale and
 *     reconstructs to quiet NaNs.
 *   - Codes: per block, the codes form a little-endian bitstream: element i of the tensor
 *     occupies bits [i*bits, (i+1)*bits) of the code buffer (4-bit: element 2j in the low
 *     nibble of byte j; 6-bit: 4 codes per 3 bytes; 8-bit: one byte each).  MXINT codes are
 *     two's-complement `bits`-bit integers in [-(2^(bits-1)-1), 2^(bits-1)-1]; MXFP codes
 *     are sign | exponent | mantissa with the sign in the top bit.  FP8 E4M3 follows the OCP
 *     encoding (S.1111.111 = NaN, never produced); the other MXFP element formats have no
 *     special codes.
 *   - e_max(MXINT b) = b - 2, e_max(MXFP eta) = 2^(eta-1).  MXINT rounding is to nearest
 *     with ties away from zero and a symmetric clip; MXFP rounding is to nearest even
 *     with saturation to the largest finite magnitude, subnormals kept, sign of zero kept.
 */
#ifndef MXQ_H
#define MXQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque here so that the header needs no CUDA include: pass a cudaStream_t. */
typedef void *mxq_stream;

typedef enum { MXQ_F32 = 0, MXQ_BF16 = 1 } mxq_dtype;

typedef enum {
    MXQ_INT8 = 0, MXQ_INT6 = 1, MXQ_INT4 = 2,
    MXQ_FP8_E4M3 = 3, MXQ_FP6_E3M2 = 4, MXQ_FP6_E2M3 = 5, MXQ_FP4_E2M1 = 6,
    MXQ_INT7 = 7, MXQ_INT5 = 8, MXQ_INT3 = 9, MXQ_INT2 = 10,
    MXQ_FP7_E3M3 = 11, MXQ_FP5_E2M2 = 12,
    MXQ_FORMAT_COUNT = 13
} mxq_format;

typedef enum { MXQ_FQ_DIRECT = 0, MXQ_FQ_VIA_ANCHOR = 1 } mxq_fq_mode;

typedef enum {
    MXQ_OK = 0,
    MXQ_ERR_NULL = -1,    /* a required pointer is null */
    MXQ_ERR_FORMAT = -2,  /* unknown format / dtype / mode enum */
    MXQ_ERR_BLOCK = -3,   /* unsupported block size */
    MXQ_ERR_SIZE = -4,    /* n is not a multiple of block, or a count is out of range */
    MXQ_ERR_ALIGN = -5,   /* a pointer is not aligned as required (32 bytes data, 16 bytes scales) */
    MXQ_ERR_PAIR = -6,    /* (src_fmt, dst_fmt) is not a same-family high-to-low pair */
    MXQ_ERR_CUDA = -7,    /* a CUDA call or launch failed */
    MXQ_ERR_TIMEOUT = -8  /* reserved: a bounded device-side wait gave up */
} mxq_status;

/* Human-readable name of a status code (static storage, never null). */
const char *mxq_status_string(int status);

/*
 * Debug builds of the library (compiled with -DMXQ_DEBUG; `python -m paper_2604_00529_b200.build --debug`
 * makes libmxq_debug.so) check every global-memory access of the kernels against the byte ranges of
 * the buffers the entry point was given -- computed from n, the format's width and the block size in
 * this layer, independently of the kernels' index arithmetic.  An access outside them is counted,
 * its address kept, and the access skipped: nothing traps.  (The paper has no counterpart; this is
 * the library's own sanitizer.)  Debug builds serve one stream at a time and are several times slower.
 *   mxq_debug_report      waits for the device, fills `out`, optionally clears the counters.
 *                         out->enabled is 0 in a release build (everything else stays 0).
 *   mxq_debug_trim_ranges test hook: from now on this thread registers every range `bytes` short, so
 *                         that the checker can be seen to catch the kernels' (legitimate) last accesses
 *                         without any access leaving its real buffer.  Returns 1 in a debug build, 0 otherwise.
 */
typedef struct mxq_debug_info {
    int enabled;                      /* 1: the library was built with -DMXQ_DEBUG */
    unsigned int checked_launches;    /* launches that ran with ranges registered */
    unsigned int violations;          /* accesses outside every registered range (each skipped) */
    unsigned long long first_address; /* address and size of the first one seen */
    unsigned int first_bytes;
} mxq_debug_info;

int mxq_debug_report(mxq_debug_info *out, int reset);
int mxq_debug_trim_ranges(size_t bytes);

/* Bits per element code of `fmt`, or 0 for an unknown format. */
int mxq_format_bits(int fmt);

/* Bytes of the packed code buffer for n elements (n * bits / 8), 0 for an unknown format. */
size_t mxq_codes_bytes(size_t n, int fmt);

/* Bytes of the scale buffer (n / block), 0 if block <= 0. */
size_t mxq_scales_bytes(size_t n, int block);

/* 1 if `block` is a supported scaling block size, else 0. */
int mxq_block_supported(int block);

/*
 * Q_f, Eq. 1-3: quantize `n` FP32 or BF16 elements at `src` into packed codes of element
 * format `fmt` plus one E8M0 scale per block.  Serves the 8-bit anchors (MXINT8, MXFP8
 * E4M3) and direct quantization to any lower format.
 *   src    [in]  device, n elements of `src_dtype`
 *   codes  [out] device, mxq_codes_bytes(n, fmt) bytes
 *   scales [out] device, n / block bytes
 */
int mxq_quantize(const void *src, int src_dtype, size_t n, int fmt, int block,
                 void *codes, uint8_t *scales, mxq_stream stream);

/*
 * Q_{h->l}, Eq. 4 (SSMXINT) and Eq. 5 (SSMXFP): convert packed codes + scales of `src_fmt`
 * into `dst_fmt` without reconstructing the full-precision tensor.  Both formats must
 * belong to the same family (MXINT or MXFP) with de = e_max(src) - e_max(dst) >= 0 and
 * bits(dst) <= bits(src); src_fmt == dst_fmt copies.  The output scale byte is
 * min(byte + de, 254), or 0xFF for a 0xFF input.
 *   codes, scales         [in]  device, layout as produced by mxq_quantize
 *   out_codes, out_scales [out] device, mxq_codes_bytes(n, dst_fmt) and n / block bytes;
 *                               must not overlap the inputs
 */
int mxq_slice_scale(const void *codes, const uint8_t *scales, size_t n, int block,
                    int src_fmt, int dst_fmt, void *out_codes, uint8_t *out_scales,
                    mxq_stream stream);

/*
 * Q_{h->l} for several targets at once (Sec. 3.5, Inference: one stored anchor, lower precisions
 * on demand): the same results as `ntargets` calls of mxq_slice_scale with the same source.
 * Consecutive targets (dst_fmts[0] with [1], [2] with [3]) that form one of the fused pairs --
 * MXINT8 -> {MXINT6, MXINT4}, MXFP8 E4M3 -> {E2M3, E2M1}, {E3M2, E2M1}, {E3M2, E2M3}, in either order
 * -- are produced by ONE pass over the anchor; any other legal target is produced by a pass of its own.
 *   dst_fmts, out_codes, out_scales  [in] HOST arrays of `ntargets` entries (0 <= ntargets <=
 *                                    MXQ_MULTI_TARGETS_MAX); the pointers inside are device pointers
 *                                    with the requirements of mxq_slice_scale; outputs must not
 *                                    overlap the inputs or one another
 */
#define MXQ_MULTI_TARGETS_MAX 8
int mxq_slice_scale_multi(const void *codes, const uint8_t *scales, size_t n, int block, int src_fmt,
                          int ntargets, const int *dst_fmts, void *const *out_codes,
                          uint8_t *const *out_scales, mxq_stream stream);

/*
 * Reconstruction V^_i = X P_i (Sec. 3.3, Notation) into FP32 or BF16, one
 * round-to-nearest-even rounding into the output type (exact unless the result falls
 * below the type's normal range; beyond its range it becomes +-Inf).  MXINT zero
 * reconstructs to +0; an MXFP zero keeps its sign.
 *   dst [out] device, n elements of `dst_dtype`
 */
int mxq_dequantize(const void *codes, const uint8_t *scales, size_t n, int fmt, int block,
                   void *dst, int dst_dtype, mxq_stream stream);

/*
 * Scales for the matrix multiply that consumes the converted weights (Sec. 3.5: W_t feeds the
 * layer's matmul).  Blackwell's block-scaled tensor-core multiply reads the E8M0 bytes of a
 * [rows, kblocks] scale matrix (kblocks = columns / 32, row-major as every entry point above
 * writes them) in tiles of 128 rows x 4 block-columns: a tile is 512 consecutive bytes, the byte
 * of row r and column c inside it sits at (r mod 32) * 16 + (r div 32) * 4 + c, and tiles follow
 * one another row-tile by row-tile.  mxq_tile_scales writes that order; rows and columns beyond
 * the matrix are filled with byte 0.  The element codes need no rearrangement: FP8 codes are
 * bytes, FP6 / FP4 codes are already the packed little-endian streams the hardware unpacks.
 *   scales [in]  device, rows * kblocks bytes, 16-byte aligned
 *   tiled  [out] device, mxq_tiled_scales_bytes(rows, kblocks) bytes, 16-byte aligned, no overlap
 */
size_t mxq_tiled_scales_bytes(size_t rows, size_t kblocks);
int mxq_tile_scales(const uint8_t *scales, size_t rows, size_t kblocks, uint8_t *tiled, mxq_stream stream);

/*
 * Q_f (Eq. 1-3) and Slice-and-Scale (Eq. 5) of a row-major [rows, cols] matrix with the scale bytes
 * written directly in the tiled order above, by the producing kernel: the same bytes as
 * mxq_quantize / mxq_slice_scale followed by mxq_tile_scales(rows, cols / 32), without the extra
 * pass.  The element codes are the same plain packed streams.  MXFP formats only (the formats the
 * block-scaled multiply takes; MXQ_ERR_FORMAT otherwise), block == 32 only (MXQ_ERR_BLOCK), cols a
 * multiple of 32 and rows * cols / 32 below 2^32 (MXQ_ERR_SIZE).  When rows is not a multiple of 128
 * or cols / 32 not a multiple of 4, the tiled buffer is first cleared on `stream`, so that the
 * uncovered part of the edge tiles reads 0.
 *   src / codes, scales   [in]  device, as for mxq_quantize / mxq_slice_scale (plain stored scales)
 *   codes / out_codes     [out] device, mxq_codes_bytes(rows * cols, fmt) bytes, 32-byte aligned
 *   tiled_scales          [out] device, mxq_tiled_scales_bytes(rows, cols / 32) bytes, 16-byte aligned
 */
int mxq_quantize_tiled(const void *src, int src_dtype, size_t rows, size_t cols, int fmt, int block,
                       void *codes, uint8_t *tiled_scales, mxq_stream stream);
int mxq_slice_scale_tiled(const void *codes, const uint8_t *scales, size_t rows, size_t cols, int block,
                          int src_fmt, int dst_fmt, void *out_codes, uint8_t *out_tiled_scales,
                          mxq_stream stream);

/*
 * Fused fake-quant forward, Eq. 6 in reconstructed form; nothing but the result leaves
 * the SM.  mode MXQ_FQ_DIRECT: dst = dequantize(Q_fmt(src)).  mode MXQ_FQ_VIA_ANCHOR:
 * dst = dequantize(Q_{A->fmt}(Q_A(src))) with A = MXINT8 for MXINT targets and MXFP8 E4M3
 * for MXFP targets.  dst has the type of src; dst == src (in place) is allowed, any other
 * overlap is not.
 */
int mxq_fake_quant(const void *src, int dtype, size_t n, int fmt, int block, int mode,
                   void *dst, mxq_stream stream);

/*
 * mxq_fake_quant over `count` tensors in one launch (Sec. 3.5, Training: every quantized weight of
 * the model goes through Eq. 6 in every step).  `items` is a HOST array, free to reuse when the call
 * returns; every pointer inside is a device pointer with the requirements of mxq_fake_quant, and
 * dst == src is allowed per item.  All tensors share dtype, format, block and mode.  The item table
 * travels in the kernel's parameter space, 512 tensors per launch; more are split over several
 * launches.  Nothing is allocated on the device.
 */
typedef struct mxq_fq_item {
    const void *src;
    void *dst;
    size_t n;
} mxq_fq_item;

int mxq_fake_quant_batched(const mxq_fq_item *items, int count, int dtype, int fmt, int block, int mode,
                           mxq_stream stream);

/*
 * mxq_quantize and mxq_dequantize over `count` tensors in one launch each: the anchor checkpoint of a
 * whole model (Sec. 3.5: W_A = Q_A(W_fp) for every quantized weight, Eq. 1-3) and the reconstruction
 * V^ = X P (Sec. 3.3, Notation) of a whole converted weight set.  `items` is a HOST array, free to
 * reuse when the call returns; every pointer inside is a device pointer with the requirements of the
 * single-tensor call, and the results are those of `count` single-tensor calls.  All tensors share
 * dtype, format and block.  The item table travels in the kernel's parameter space, 512 tensors per
 * launch (more: more launches); nothing is allocated on the device.
 */
typedef struct mxq_q_item {
    const void *src;      /* [in]  device, n elements of src_dtype */
    size_t n;
    void *codes;          /* [out] device, mxq_codes_bytes(n, fmt) bytes */
    uint8_t *scales;      /* [out] device, n / block bytes */
} mxq_q_item;

int mxq_quantize_batched(const mxq_q_item *items, int count, int src_dtype, int fmt, int block,
                         mxq_stream stream);

typedef struct mxq_dq_item {
    const void *codes;      /* [in]  device, packed codes of n elements */
    const uint8_t *scales;  /* [in]  device, n / block bytes */
    size_t n;
    void *dst;              /* [out] device, n elements of dst_dtype */
} mxq_dq_item;

int mxq_dequantize_batched(const mxq_dq_item *items, int count, int fmt, int block, int dst_dtype,
                           mxq_stream stream);

/*
 * Straight-through estimator backward of mxq_fake_quant (Sec. 3.5): grad_in = grad_out.
 * grad_in == grad_out is a no-op; otherwise n elements of `dtype` are copied.
 */
int mxq_fake_quant_bwd(const void *grad_out, int dtype, size_t n, void *grad_in,
                       mxq_stream stream);

/*
 * Whole-model on-the-fly conversion (Sec. 3.5, Inference): mxq_slice_scale over `count`
 * tensors in one launch.  `items` is a HOST array; every pointer inside is a device
 * pointer with the same requirements as in mxq_slice_scale; the host array may be freed
 * as soon as the call returns.  The item table travels in the kernel's own parameter
 * space, 512 non-empty tensors per launch (more tensors: more launches); nothing is
 * allocated or copied and no state is shared between calls.
 */
typedef struct mxq_ss_item {
    const void *codes;
    const uint8_t *scales;
    size_t n;
    void *out_codes;
    uint8_t *out_scales;
} mxq_ss_item;

int mxq_slice_scale_batched(const mxq_ss_item *items, int count, int block,
                            int src_fmt, int dst_fmt, mxq_stream stream);

/*
 * Whole-model conversion into TWO lower formats from one read of every anchor (Sec. 3.5, Inference: one
 * stored anchor checkpoint, several precisions served at once; Eq. 4-5 applied twice per element): the
 * results of mxq_slice_scale_batched to dst_fmt1 and to dst_fmt2.  For the fused pairs of
 * mxq_slice_scale_multi one launch covers 256 tensors and reads the anchors once (2.34 instead of
 * 3.375 bytes per element for 6-bit + 4-bit targets); any other legal pair of targets runs as two
 * single-target batched passes.  `items` is a HOST array; requirements per pointer as in mxq_slice_scale;
 * block must be 32, 64 or 128; outputs must not overlap the inputs or one another.  Nothing is allocated
 * on the device.
 */
typedef struct mxq_ss_pair_item {
    const void *codes;
    const uint8_t *scales;
    size_t n;
    void *out_codes1;        /* mxq_codes_bytes(n, dst_fmt1) bytes */
    uint8_t *out_scales1;
    void *out_codes2;        /* mxq_codes_bytes(n, dst_fmt2) bytes */
    uint8_t *out_scales2;
} mxq_ss_pair_item;

int mxq_slice_scale_pair_batched(const mxq_ss_pair_item *items, int count, int block, int src_fmt,
                                 int dst_fmt1, int dst_fmt2, mxq_stream stream);

/*
 * mxq_slice_scale_batched with every tensor's scale bytes written in the tiled order of
 * mxq_tile_scales (the whole-model conversion of Sec. 3.5 handed straight to block-scaled matrix
 * multiplies): item i is a row-major [rows, cols] matrix, and its results are those of
 * mxq_slice_scale_tiled on it.  MXFP formats and block == 32 only, as there.  The items travel in
 * the kernel's parameter space, 256 per launch (more items: more launches); nothing is allocated.
 * Tiled buffers of matrices that do not cover whole tiles are cleared on `stream` first.
 */
typedef struct mxq_ss_tiled_item {
    const void *codes;            /* [in]  device, anchor codes of rows * cols elements */
    const uint8_t *scales;        /* [in]  device, rows * cols / 32 plain scale bytes */
    size_t rows, cols;            /* cols a multiple of 32; rows * cols / 32 below 2^32 */
    void *out_codes;              /* [out] device, mxq_codes_bytes(rows * cols, dst_fmt) bytes */
    uint8_t *out_tiled_scales;    /* [out] device, mxq_tiled_scales_bytes(rows, cols / 32) bytes */
} mxq_ss_tiled_item;

int mxq_slice_scale_tiled_batched(const mxq_ss_tiled_item *items, int count, int block,
                                  int src_fmt, int dst_fmt, mxq_stream stream);

/*
 * The same conversion as mxq_slice_scale_batched for callers that cannot allocate device memory.
 * (The paper has no counterpart of this entry point; it exists for the library's users.)  Some
 * processes give all of HBM to a pool of their own at start-up, so a cudaMalloc made behind their
 * back fails or takes memory that was promised elsewhere; others run a loop that cannot take the
 * device-wide synchronisation that cudaMalloc / cudaFree imply.  For them the item table lives in a
 * fixed array inside the library image: MXQ_STATIC_BATCH_MAX items and a small index, 57 KiB,
 * present on every GPU that loads libmxq until the process exits.  The library makes no cudaMalloc,
 * cudaFree or other allocating call here, on the device or on the host heap, and converts up to
 * MXQ_STATIC_BATCH_MAX tensors in one launch.  (mxq_slice_scale_batched allocates nothing on the
 * device either, but it builds its launch tables on the host heap and needs one launch per 512 tensors.)
 * What the call does cost: it builds the table (57 KiB) on the caller's STACK, so a thread with a
 * small stack needs about 64 KiB free; it copies the used part of it (0.6 - 57 KiB) to the device
 * with a stream-ordered copy from that pageable memory, for which the CUDA runtime stages the bytes
 * and may make the host wait for earlier work on `stream`; and the first call on a device may load
 * the library's device code.  It is free of allocation, not free of host waits.
 *   - Arguments, checks and results are those of mxq_slice_scale_batched (block must be 32, 64 or
 *     128); in addition count > MXQ_STATIC_BATCH_MAX returns MXQ_ERR_SIZE and launches nothing.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and keeps it; make that first call before starting any stream capture.
 *   - A call on a stream that is being captured returns MXQ_ERR_CUDA and enqueues nothing: the table
 *     copy reads a buffer that no longer exists when the call has returned, so a recorded copy of it
 *     would feed every replay stale stack bytes.
 *   - All calls on one device share the one table.  Each call rewrites the entries it uses and the
 *     kernel reads no others, so stale contents of an earlier call are harmless.  Calls ordered by
 *     one stream are safe; two calls whose work can overlap on the GPU (different streams, no
 *     dependency between them) race on the table and give undefined results.
 */
#define MXQ_STATIC_BATCH_MAX 1024
int mxq_slice_scale_batched_static(const mxq_ss_item *items, int count, int block,
                                   int src_fmt, int dst_fmt, mxq_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* MXQ_H */
