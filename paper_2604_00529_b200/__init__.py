"""B200-native block-wise microscaling (MX) quantization for MF-QAT.

The compute lives in ``libmxq.so`` (hand-written CUDA for sm_100a behind the C ABI declared in
``include/mxq.h``).  This package is a thin ctypes binding with the same entry-point names; it
marshals arguments and nothing else.  There is no CPU fallback: every call fails loudly when
the library is missing or the tensors are not CUDA tensors.
"""
from .binding import (  # noqa: F401
    BF16, F32, FORMATS, FQ_DIRECT, FQ_VIA_ANCHOR, MxqError, codes_bytes, dequantize, fake_quant, fake_quant_batched,
    make_fq_items,
    fake_quant_bwd, fake_quant_ste, format_bits, library_path, load_library, make_items, quantize, scales_bytes, slice_scale,
    slice_scale_batched, slice_scale_batched_static, slice_scale_multi, quantize_tiled, slice_scale_tiled, slice_scale_tiled_batched, make_tiled_items, tile_scales, tiled_scales_bytes, status_string, STATIC_BATCH_MAX,
    slice_scale_pair_batched, make_pair_items,
    quantize_batched, make_q_items, dequantize_batched, make_dq_items,
    PreparedCall, prepare_quantize, prepare_slice_scale, prepare_dequantize, prepare_fake_quant, prepare_fake_quant_bwd,
)
