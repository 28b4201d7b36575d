"""ctypes binding of libmxq.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams: tensors are passed as raw device pointers and
the current CUDA stream's handle.  Code and scale buffers are ``torch.uint8`` tensors.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmxq.so")

F32, BF16 = 0, 1
FQ_DIRECT, FQ_VIA_ANCHOR = 0, 1

#: format name -> mxq_format enum value (include/mxq.h)
FORMATS = {
    "int8": 0, "int6": 1, "int4": 2, "e4m3": 3, "e3m2": 4, "e2m3": 5, "e2m1": 6,
    "int7": 7, "int5": 8, "int3": 9, "int2": 10, "e3m3": 11, "e2m2": 12,
}


class MxqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__("%s failed: %s" % (what, status_string(status)))


class _FqItem(ctypes.Structure):
    _fields_ = [("src", ctypes.c_void_p), ("dst", ctypes.c_void_p), ("n", ctypes.c_size_t)]


class _QItem(ctypes.Structure):
    _fields_ = [("src", ctypes.c_void_p), ("n", ctypes.c_size_t), ("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p)]


class _DqItem(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("n", ctypes.c_size_t), ("dst", ctypes.c_void_p)]


class _Item(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("n", ctypes.c_size_t),
                ("out_codes", ctypes.c_void_p), ("out_scales", ctypes.c_void_p)]


class _PairItem(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("n", ctypes.c_size_t),
                ("out_codes1", ctypes.c_void_p), ("out_scales1", ctypes.c_void_p),
                ("out_codes2", ctypes.c_void_p), ("out_scales2", ctypes.c_void_p)]


class _TiledItem(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("rows", ctypes.c_size_t),
                ("cols", ctypes.c_size_t), ("out_codes", ctypes.c_void_p), ("out_tiled_scales", ctypes.c_void_p)]


_lib: Optional[ctypes.CDLL] = None


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Load libmxq.so (built in-tree by ``python -m paper_2604_00529_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("libmxq.so is not built: run `python -m paper_2604_00529_b200.build` "
                          "(there is no fallback path)")
    L = ctypes.CDLL(_LIB_PATH)
    vp, sz, i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    L.mxq_status_string.argtypes = [i]
    L.mxq_status_string.restype = ctypes.c_char_p
    L.mxq_format_bits.argtypes = [i]
    L.mxq_format_bits.restype = i
    L.mxq_codes_bytes.argtypes = [sz, i]
    L.mxq_codes_bytes.restype = sz
    L.mxq_scales_bytes.argtypes = [sz, i]
    L.mxq_scales_bytes.restype = sz
    L.mxq_block_supported.argtypes = [i]
    L.mxq_block_supported.restype = i
    L.mxq_quantize.argtypes = [vp, i, sz, i, i, vp, vp, vp]
    L.mxq_slice_scale.argtypes = [vp, vp, sz, i, i, i, vp, vp, vp]
    L.mxq_dequantize.argtypes = [vp, vp, sz, i, i, vp, i, vp]
    L.mxq_slice_scale_multi.argtypes = [vp, vp, sz, i, i, i, ctypes.POINTER(i), ctypes.POINTER(vp), ctypes.POINTER(vp), vp]
    L.mxq_slice_scale_multi.restype = i
    L.mxq_fake_quant.argtypes = [vp, i, sz, i, i, i, vp, vp]
    L.mxq_fake_quant_batched.argtypes = [ctypes.POINTER(_FqItem), i, i, i, i, i, vp]
    L.mxq_fake_quant_batched.restype = i
    L.mxq_quantize_batched.argtypes = [ctypes.POINTER(_QItem), i, i, i, i, vp]
    L.mxq_quantize_batched.restype = i
    L.mxq_dequantize_batched.argtypes = [ctypes.POINTER(_DqItem), i, i, i, i, vp]
    L.mxq_dequantize_batched.restype = i
    L.mxq_tiled_scales_bytes.argtypes = [sz, sz]
    L.mxq_tiled_scales_bytes.restype = sz
    L.mxq_tile_scales.argtypes = [vp, sz, sz, vp, vp]
    L.mxq_tile_scales.restype = i
    L.mxq_quantize_tiled.argtypes = [vp, i, sz, sz, i, i, vp, vp, vp]
    L.mxq_quantize_tiled.restype = i
    L.mxq_slice_scale_tiled.argtypes = [vp, vp, sz, sz, i, i, i, vp, vp, vp]
    L.mxq_slice_scale_tiled.restype = i
    L.mxq_slice_scale_tiled_batched.argtypes = [ctypes.POINTER(_TiledItem), i, i, i, i, vp]
    L.mxq_slice_scale_tiled_batched.restype = i
    L.mxq_fake_quant_bwd.argtypes = [vp, i, sz, vp, vp]
    L.mxq_slice_scale_batched.argtypes = [ctypes.POINTER(_Item), i, i, i, i, vp]
    L.mxq_slice_scale_pair_batched.argtypes = [ctypes.POINTER(_PairItem), i, i, i, i, i, vp]
    L.mxq_slice_scale_pair_batched.restype = i
    L.mxq_slice_scale_batched_static.argtypes = [ctypes.POINTER(_Item), i, i, i, i, vp]
    L.mxq_slice_scale_batched_static.restype = i
    for name in ("mxq_quantize", "mxq_slice_scale", "mxq_dequantize", "mxq_fake_quant", "mxq_fake_quant_bwd",
                 "mxq_slice_scale_batched"):
        getattr(L, name).restype = i
    _lib = L
    return L


def status_string(status: int) -> str:
    return load_library().mxq_status_string(int(status)).decode()


def format_bits(fmt: str) -> int:
    return load_library().mxq_format_bits(FORMATS[fmt])


def codes_bytes(n: int, fmt: str) -> int:
    return load_library().mxq_codes_bytes(n, FORMATS[fmt])


def scales_bytes(n: int, block: int = 32) -> int:
    return load_library().mxq_scales_bytes(n, block)


def _dtype_id(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("mxq tensors are float32 or bfloat16, got %s" % t.dtype)


def _dev(t: torch.Tensor, what: str) -> int:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (libmxq has no CPU path)" % what)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % what)
    return t.data_ptr()


# torch.cuda.current_stream() builds a Stream object per call (about 3 us, more than the launch itself);
# the raw handle of the current device's current stream comes straight from the C layer when torch has it.
_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream) -> int:
    if stream is None:
        if _raw_stream is not None:
            return _raw_stream(torch.cuda.current_device())
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise MxqError(rc, what)


def quantize(src: torch.Tensor, fmt: str, block: int = 32, codes: Optional[torch.Tensor] = None,
             scales: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """mxq_quantize: returns (packed codes uint8[n*bits/8], scales uint8[n/block])."""
    L = load_library()
    n = src.numel()
    if codes is None:
        codes = torch.empty(codes_bytes(n, fmt), dtype=torch.uint8, device=src.device)
    if scales is None:
        scales = torch.empty(n // block if block > 0 else 0, dtype=torch.uint8, device=src.device)
    _check(L.mxq_quantize(_dev(src, "src"), _dtype_id(src), n, FORMATS[fmt], block, _dev(codes, "codes"),
                          _dev(scales, "scales"), _stream(stream)), "mxq_quantize")
    return codes, scales


def slice_scale(codes: torch.Tensor, scales: torch.Tensor, n: int, src_fmt: str, dst_fmt: str, block: int = 32,
                out_codes: Optional[torch.Tensor] = None, out_scales: Optional[torch.Tensor] = None,
                stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """mxq_slice_scale: anchor codes + scales -> lower-format codes + scales."""
    L = load_library()
    if out_codes is None:
        out_codes = torch.empty(codes_bytes(n, dst_fmt), dtype=torch.uint8, device=codes.device)
    if out_scales is None:
        out_scales = torch.empty(n // block if block > 0 else 0, dtype=torch.uint8, device=codes.device)
    _check(L.mxq_slice_scale(_dev(codes, "codes"), _dev(scales, "scales"), n, block, FORMATS[src_fmt],
                             FORMATS[dst_fmt], _dev(out_codes, "out_codes"), _dev(out_scales, "out_scales"),
                             _stream(stream)), "mxq_slice_scale")
    return out_codes, out_scales


def slice_scale_multi(codes: torch.Tensor, scales: torch.Tensor, n: int, src_fmt: str, dst_fmts: Sequence[str],
                      block: int = 32, outs: Optional[Sequence[Tuple[torch.Tensor, torch.Tensor]]] = None, stream=None):
    """mxq_slice_scale_multi: one anchor -> several lower formats; returns [(codes, scales), ...]."""
    L = load_library()
    k = len(dst_fmts)
    if outs is None:
        outs = [(torch.empty(codes_bytes(n, f), dtype=torch.uint8, device=codes.device),
                 torch.empty(n // block if block > 0 else 0, dtype=torch.uint8, device=codes.device)) for f in dst_fmts]
    fm = (ctypes.c_int * k)(*[FORMATS[f] for f in dst_fmts])
    oc = (ctypes.c_void_p * k)(*[_dev(c, "out_codes") for c, _ in outs])
    os_ = (ctypes.c_void_p * k)(*[_dev(s, "out_scales") for _, s in outs])
    _check(L.mxq_slice_scale_multi(_dev(codes, "codes"), _dev(scales, "scales"), n, block, FORMATS[src_fmt], k, fm, oc,
                                   os_, _stream(stream)), "mxq_slice_scale_multi")
    return list(outs)


def dequantize(codes: torch.Tensor, scales: torch.Tensor, n: int, fmt: str, block: int = 32,
               dtype: torch.dtype = torch.float32, dst: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """mxq_dequantize: V^ = X P as float32 or bfloat16."""
    L = load_library()
    if dst is None:
        dst = torch.empty(n, dtype=dtype, device=codes.device)
    _check(L.mxq_dequantize(_dev(codes, "codes"), _dev(scales, "scales"), n, FORMATS[fmt], block, _dev(dst, "dst"),
                            _dtype_id(dst), _stream(stream)), "mxq_dequantize")
    return dst


def tiled_scales_bytes(rows: int, kblocks: int) -> int:
    return load_library().mxq_tiled_scales_bytes(rows, kblocks)


def tile_scales(scales: torch.Tensor, rows: int, kblocks: int, tiled: Optional[torch.Tensor] = None,
                stream=None) -> torch.Tensor:
    """mxq_tile_scales: row-major [rows, kblocks] scale bytes -> the 128 x 4 tiled order a block-scaled
    tensor-core matmul reads."""
    L = load_library()
    if tiled is None:
        tiled = torch.empty(tiled_scales_bytes(rows, kblocks), dtype=torch.uint8, device=scales.device)
    _check(L.mxq_tile_scales(_dev(scales, "scales"), rows, kblocks, _dev(tiled, "tiled"), _stream(stream)),
           "mxq_tile_scales")
    return tiled


def quantize_tiled(src: torch.Tensor, fmt: str, block: int = 32, codes: Optional[torch.Tensor] = None,
                   tiled_scales: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """mxq_quantize_tiled: a 2-D [rows, cols] tensor -> (packed codes, scale bytes in the 128 x 4 tiled order)."""
    L = load_library()
    if src.dim() != 2:
        raise ValueError("quantize_tiled takes a [rows, cols] matrix")
    rows, cols = src.shape
    if codes is None:
        codes = torch.empty(codes_bytes(rows * cols, fmt), dtype=torch.uint8, device=src.device)
    if tiled_scales is None:
        tiled_scales = torch.empty(tiled_scales_bytes(rows, cols // 32), dtype=torch.uint8, device=src.device)
    _check(L.mxq_quantize_tiled(_dev(src, "src"), _dtype_id(src), rows, cols, FORMATS[fmt], block, _dev(codes, "codes"),
                                _dev(tiled_scales, "tiled_scales"), _stream(stream)), "mxq_quantize_tiled")
    return codes, tiled_scales


def slice_scale_tiled(codes: torch.Tensor, scales: torch.Tensor, rows: int, cols: int, src_fmt: str, dst_fmt: str,
                      block: int = 32, out_codes: Optional[torch.Tensor] = None,
                      out_tiled_scales: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """mxq_slice_scale_tiled: anchor codes + plain scales of a [rows, cols] matrix -> lower-format codes and
    scale bytes in the 128 x 4 tiled order."""
    L = load_library()
    if out_codes is None:
        out_codes = torch.empty(codes_bytes(rows * cols, dst_fmt), dtype=torch.uint8, device=codes.device)
    if out_tiled_scales is None:
        out_tiled_scales = torch.empty(tiled_scales_bytes(rows, cols // 32), dtype=torch.uint8, device=codes.device)
    _check(L.mxq_slice_scale_tiled(_dev(codes, "codes"), _dev(scales, "scales"), rows, cols, block, FORMATS[src_fmt],
                                   FORMATS[dst_fmt], _dev(out_codes, "out_codes"),
                                   _dev(out_tiled_scales, "out_tiled_scales"), _stream(stream)), "mxq_slice_scale_tiled")
    return out_codes, out_tiled_scales


def fake_quant(src: torch.Tensor, fmt: str, block: int = 32, mode: int = FQ_DIRECT,
               dst: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """mxq_fake_quant: quantize-dequantize in one pass (dst may be src)."""
    L = load_library()
    if dst is None:
        dst = torch.empty_like(src)
    _check(L.mxq_fake_quant(_dev(src, "src"), _dtype_id(src), src.numel(), FORMATS[fmt], block, mode,
                            _dev(dst, "dst"), _stream(stream)), "mxq_fake_quant")
    return dst


class FqTable:
    """A marshalled mxq_fq_item array for tensors that persist (e.g. a model's weights): build it once
    with ``make_fq_items`` and pass it to ``fake_quant_batched`` every step."""

    def __init__(self, pairs):
        self.tensors = [(s, d if d is not None else s) for s, d in pairs]
        if not self.tensors:
            raise ValueError("no tensors")
        self.dtype = _dtype_id(self.tensors[0][0])
        self.array = (_FqItem * len(self.tensors))()
        for k, (s, d) in enumerate(self.tensors):
            if _dtype_id(s) != self.dtype or d.dtype != s.dtype or d.numel() != s.numel():
                raise TypeError("all tensors of a batch share one dtype; dst matches src")
            self.array[k] = _FqItem(_dev(s, "src"), _dev(d, "dst"), s.numel())

    def __len__(self):
        return len(self.tensors)


def make_fq_items(pairs) -> FqTable:
    """Marshal (src, dst) tensor pairs (dst None = in place) into an mxq_fq_item array."""
    return FqTable(pairs)


def fake_quant_batched(pairs, fmt: str, block: int = 32, mode: int = FQ_DIRECT, stream=None) -> None:
    """mxq_fake_quant_batched over (src, dst) pairs or an FqTable made from them."""
    L = load_library()
    table = pairs if isinstance(pairs, FqTable) else FqTable(pairs)
    _check(L.mxq_fake_quant_batched(table.array, len(table), table.dtype, FORMATS[fmt], block, mode, _stream(stream)),
           "mxq_fake_quant_batched")


class QTable:
    """A marshalled mxq_q_item array over (src, codes, scales) tensor triples that persist (keeps them alive)."""

    def __init__(self, triples):
        self.tensors = list(triples)
        if not self.tensors:
            raise ValueError("no tensors")
        self.dtype = _dtype_id(self.tensors[0][0])
        self.array = (_QItem * len(self.tensors))()
        for k, (src, codes, scales) in enumerate(self.tensors):
            if _dtype_id(src) != self.dtype:
                raise TypeError("all tensors of a batch share one dtype")
            self.array[k] = _QItem(_dev(src, "src"), src.numel(), _dev(codes, "codes"), _dev(scales, "scales"))

    def __len__(self):
        return len(self.tensors)


def make_q_items(triples) -> QTable:
    """Marshal (src, codes, scales) tensor triples into an mxq_q_item array."""
    return QTable(triples)


def quantize_batched(triples, fmt: str, block: int = 32, stream=None) -> None:
    """mxq_quantize_batched over (src, codes, scales) triples or a QTable made from them."""
    L = load_library()
    table = triples if isinstance(triples, QTable) else QTable(triples)
    _check(L.mxq_quantize_batched(table.array, len(table), table.dtype, FORMATS[fmt], block, _stream(stream)),
           "mxq_quantize_batched")


class DqTable:
    """A marshalled mxq_dq_item array over (codes, scales, n, dst) tuples that persist (keeps them alive)."""

    def __init__(self, items):
        self.tensors = list(items)
        if not self.tensors:
            raise ValueError("no tensors")
        self.dtype = _dtype_id(self.tensors[0][3])
        self.array = (_DqItem * len(self.tensors))()
        for k, (codes, scales, n, dst) in enumerate(self.tensors):
            if _dtype_id(dst) != self.dtype or dst.numel() != n:
                raise TypeError("all outputs of a batch share one dtype and hold n elements")
            self.array[k] = _DqItem(_dev(codes, "codes"), _dev(scales, "scales"), n, _dev(dst, "dst"))

    def __len__(self):
        return len(self.tensors)


def make_dq_items(items) -> DqTable:
    """Marshal (codes, scales, n, dst) tuples into an mxq_dq_item array."""
    return DqTable(items)


def dequantize_batched(items, fmt: str, block: int = 32, stream=None) -> None:
    """mxq_dequantize_batched over (codes, scales, n, dst) tuples or a DqTable made from them."""
    L = load_library()
    table = items if isinstance(items, DqTable) else DqTable(items)
    _check(L.mxq_dequantize_batched(table.array, len(table), FORMATS[fmt], block, table.dtype, _stream(stream)),
           "mxq_dequantize_batched")


def fake_quant_bwd(grad_out: torch.Tensor, grad_in: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """mxq_fake_quant_bwd: straight-through gradient (identity)."""
    L = load_library()
    if grad_in is None:
        grad_in = torch.empty_like(grad_out)
    _check(L.mxq_fake_quant_bwd(_dev(grad_out, "grad_out"), _dtype_id(grad_out), grad_out.numel(),
                                _dev(grad_in, "grad_in"), _stream(stream)), "mxq_fake_quant_bwd")
    return grad_in


class PreparedCall:
    """One C-ABI call with its arguments already marshalled, for buffers that persist (a model's
    weights and their code buffers): ``prepare_*`` checks and converts the arguments once, calling the
    object enqueues the operation on the current stream (or on ``stream``).  It keeps the tensors alive.
    Per call this leaves the stream lookup and the foreign call itself (about 2 us instead of 5)."""

    __slots__ = ("fn", "args", "what", "keep")

    def __init__(self, fn, args, what, keep):
        self.fn, self.args, self.what, self.keep = fn, args, what, keep

    def __call__(self, stream=None) -> None:
        rc = self.fn(*self.args, _stream(stream))
        if rc != 0:
            raise MxqError(rc, self.what)


def prepare_quantize(src: torch.Tensor, fmt: str, block: int, codes: torch.Tensor, scales: torch.Tensor) -> PreparedCall:
    """mxq_quantize(src -> codes, scales) as a PreparedCall."""
    L = load_library()
    return PreparedCall(L.mxq_quantize, (_dev(src, "src"), _dtype_id(src), src.numel(), FORMATS[fmt], block,
                                         _dev(codes, "codes"), _dev(scales, "scales")), "mxq_quantize",
                        (src, codes, scales))


def prepare_slice_scale(codes: torch.Tensor, scales: torch.Tensor, n: int, src_fmt: str, dst_fmt: str, block: int,
                        out_codes: torch.Tensor, out_scales: torch.Tensor) -> PreparedCall:
    """mxq_slice_scale as a PreparedCall."""
    L = load_library()
    return PreparedCall(L.mxq_slice_scale, (_dev(codes, "codes"), _dev(scales, "scales"), n, block, FORMATS[src_fmt],
                                            FORMATS[dst_fmt], _dev(out_codes, "out_codes"),
                                            _dev(out_scales, "out_scales")), "mxq_slice_scale",
                        (codes, scales, out_codes, out_scales))


def prepare_dequantize(codes: torch.Tensor, scales: torch.Tensor, n: int, fmt: str, block: int,
                       dst: torch.Tensor) -> PreparedCall:
    """mxq_dequantize as a PreparedCall."""
    L = load_library()
    return PreparedCall(L.mxq_dequantize, (_dev(codes, "codes"), _dev(scales, "scales"), n, FORMATS[fmt], block,
                                           _dev(dst, "dst"), _dtype_id(dst)), "mxq_dequantize", (codes, scales, dst))


def prepare_fake_quant(src: torch.Tensor, fmt: str, block: int, mode: int, dst: torch.Tensor) -> PreparedCall:
    """mxq_fake_quant as a PreparedCall."""
    L = load_library()
    return PreparedCall(L.mxq_fake_quant, (_dev(src, "src"), _dtype_id(src), src.numel(), FORMATS[fmt], block, mode,
                                           _dev(dst, "dst")), "mxq_fake_quant", (src, dst))


def prepare_fake_quant_bwd(grad_out: torch.Tensor, grad_in: torch.Tensor) -> PreparedCall:
    """mxq_fake_quant_bwd as a PreparedCall."""
    L = load_library()
    return PreparedCall(L.mxq_fake_quant_bwd, (_dev(grad_out, "grad_out"), _dtype_id(grad_out), grad_out.numel(),
                                               _dev(grad_in, "grad_in")), "mxq_fake_quant_bwd", (grad_out, grad_in))


class _FakeQuantSTE(torch.autograd.Function):
    """Eq. 6 inside autograd: forward is mxq_fake_quant, backward the straight-through estimator."""

    @staticmethod
    def forward(ctx, x, fmt, block, mode, copy_grad):
        ctx.copy_grad = copy_grad
        return fake_quant(x.detach(), fmt, block, mode)

    @staticmethod
    def backward(ctx, grad_out):
        # identity: the incoming gradient itself, or a copy of it made by mxq_fake_quant_bwd
        g = fake_quant_bwd(grad_out.contiguous()) if ctx.copy_grad else grad_out
        return g, None, None, None, None


def fake_quant_ste(x: torch.Tensor, fmt: str, block: int = 32, mode: int = FQ_VIA_ANCHOR,
                   copy_grad: bool = False) -> torch.Tensor:
    """W_t of Eq. 6 as a differentiable function of W: the value is ``fake_quant(x, fmt, block, mode)``,
    the gradient passes straight through (``copy_grad`` hands autograd a fresh copy instead of the
    incoming tensor)."""
    return _FakeQuantSTE.apply(x, fmt, block, mode, copy_grad)


class ItemTable:
    """A marshalled mxq_ss_item array: build it once with ``make_items`` for buffers that persist and
    pass it to ``slice_scale_batched`` as often as needed (it keeps the tensors alive)."""

    def __init__(self, items):
        self.tensors = list(items)
        self.array = (_Item * len(self.tensors))()
        for k, (c, s, n, oc, os_) in enumerate(self.tensors):
            self.array[k] = _Item(_dev(c, "codes"), _dev(s, "scales"), n, _dev(oc, "out_codes"), _dev(os_, "out_scales"))

    def __len__(self):
        return len(self.tensors)


def make_items(items: Sequence[Tuple[torch.Tensor, torch.Tensor, int, torch.Tensor, torch.Tensor]]) -> ItemTable:
    """Marshal (codes, scales, n, out_codes, out_scales) tuples into an mxq_ss_item array."""
    return ItemTable(items)


def slice_scale_batched(items, src_fmt: str, dst_fmt: str, block: int = 32, stream=None) -> None:
    """mxq_slice_scale_batched over (codes, scales, n, out_codes, out_scales) tuples, or over an
    ItemTable made from them."""
    L = load_library()
    table = items if isinstance(items, ItemTable) else ItemTable(items)
    _check(L.mxq_slice_scale_batched(table.array, len(table), block, FORMATS[src_fmt], FORMATS[dst_fmt],
                                     _stream(stream)), "mxq_slice_scale_batched")


class PairItemTable:
    """A marshalled mxq_ss_pair_item array over (codes, scales, n, out_codes1, out_scales1, out_codes2,
    out_scales2) tuples that persist (keeps the tensors alive)."""

    def __init__(self, items):
        self.tensors = list(items)
        self.array = (_PairItem * len(self.tensors))()
        for k, (c, s, n, c1, s1, c2, s2) in enumerate(self.tensors):
            self.array[k] = _PairItem(_dev(c, "codes"), _dev(s, "scales"), n, _dev(c1, "out_codes1"), _dev(s1, "out_scales1"),
                                      _dev(c2, "out_codes2"), _dev(s2, "out_scales2"))

    def __len__(self):
        return len(self.tensors)


def make_pair_items(items) -> PairItemTable:
    """Marshal (codes, scales, n, out_codes1, out_scales1, out_codes2, out_scales2) tuples into an mxq_ss_pair_item array."""
    return PairItemTable(items)


def slice_scale_pair_batched(items, src_fmt: str, dst_fmt1: str, dst_fmt2: str, block: int = 32, stream=None) -> None:
    """mxq_slice_scale_pair_batched: every anchor of a set of tensors to two lower formats, one read of the anchor."""
    L = load_library()
    table = items if isinstance(items, PairItemTable) else PairItemTable(items)
    _check(L.mxq_slice_scale_pair_batched(table.array, len(table), block, FORMATS[src_fmt], FORMATS[dst_fmt1],
                                          FORMATS[dst_fmt2], _stream(stream)), "mxq_slice_scale_pair_batched")


class TiledItemTable:
    """A marshalled mxq_ss_tiled_item array (keeps the tensors alive), for buffers that persist."""

    def __init__(self, items):
        self.tensors = list(items)
        self.array = (_TiledItem * len(self.tensors))()
        for k, (c, s, rows, cols, oc, ot) in enumerate(self.tensors):
            self.array[k] = _TiledItem(_dev(c, "codes"), _dev(s, "scales"), rows, cols, _dev(oc, "out_codes"),
                                       _dev(ot, "out_tiled_scales"))

    def __len__(self):
        return len(self.tensors)


def make_tiled_items(items) -> TiledItemTable:
    """Marshal (codes, scales, rows, cols, out_codes, out_tiled_scales) tuples into an mxq_ss_tiled_item array."""
    return TiledItemTable(items)


def slice_scale_tiled_batched(items, src_fmt: str, dst_fmt: str, block: int = 32, stream=None) -> None:
    """mxq_slice_scale_tiled_batched over (codes, scales, rows, cols, out_codes, out_tiled_scales) tuples or a
    TiledItemTable made from them."""
    L = load_library()
    table = items if isinstance(items, TiledItemTable) else TiledItemTable(items)
    _check(L.mxq_slice_scale_tiled_batched(table.array, len(table), block, FORMATS[src_fmt], FORMATS[dst_fmt],
                                           _stream(stream)), "mxq_slice_scale_tiled_batched")


#: largest item count mxq_slice_scale_batched_static accepts (MXQ_STATIC_BATCH_MAX in include/mxq.h)
STATIC_BATCH_MAX = 1024


def slice_scale_batched_static(items: Sequence[Tuple[torch.Tensor, torch.Tensor, int, torch.Tensor, torch.Tensor]],
                               src_fmt: str, dst_fmt: str, block: int = 32, stream=None) -> None:
    """mxq_slice_scale_batched_static: slice_scale_batched for callers that may not allocate device
    memory (a process whose own pool owns all of HBM, or a loop that cannot afford the device-wide
    stall of cudaMalloc).  The item table is a fixed array inside libmxq, so at most STATIC_BATCH_MAX
    items fit, and calls that can overlap on the GPU must not share a device.  The marshalling here
    builds one small ctypes array on the host and touches no torch allocator."""
    L = load_library()
    arr = (_Item * len(items))()
    for k, (c, s, n, oc, os_) in enumerate(items):
        arr[k] = _Item(_dev(c, "codes"), _dev(s, "scales"), n, _dev(oc, "out_codes"), _dev(os_, "out_scales"))
    _check(L.mxq_slice_scale_batched_static(arr, len(items), block, FORMATS[src_fmt], FORMATS[dst_fmt],
                                            _stream(stream)), "mxq_slice_scale_batched_static")
