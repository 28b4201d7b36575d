"""numpy front end of the CPU oracle (``mxq_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the bench's
CPU-baseline legs.  Nothing here imports the CUDA package and the CUDA package never
imports this module.  All arithmetic lives in the C file; this module only compiles it
with gcc, marshals numpy arrays and names the element formats.

Formats are named by strings: ``int2`` .. ``int8`` for MXINT(b) and ``e4m3``, ``e3m3``,
``e3m2``, ``e2m3``, ``e2m2``, ``e2m1`` for MXFP(eta, mu).
Codes travel one code per byte unless a function says "packed".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# MXQ_ORACLE_SOURCE points the front end at another C file (the mutation test compiles copies of the
# oracle with one planted mistake each and checks that the pins catch it); its library is built beside it.
_SRC = os.environ.get("MXQ_ORACLE_SOURCE") or os.path.join(_HERE, "mxq_oracle.c")
_LIB = os.path.join(os.path.dirname(os.path.abspath(_SRC)), "libmxq_oracle.so")

F32, BF16 = 0, 1
FQ_DIRECT, FQ_VIA_ANCHOR = 0, 1

#: name -> (kind, a, m): kind 0 = MXINT(a bits), kind 1 = MXFP(eta=a, mu=m)
FORMATS = {
    "int8": (0, 8, 0), "int7": (0, 7, 0), "int6": (0, 6, 0), "int5": (0, 5, 0),
    "int4": (0, 4, 0), "int3": (0, 3, 0), "int2": (0, 2, 0),
    "e4m3": (1, 4, 3), "e3m3": (1, 3, 3), "e3m2": (1, 3, 2),
    "e2m3": (1, 2, 3), "e2m2": (1, 2, 2), "e2m1": (1, 2, 1),
}


def bits(fmt: str) -> int:
    kind, a, m = FORMATS[fmt]
    return a if kind == 0 else 1 + a + m


def anchor_of(fmt: str) -> str:
    """The 8-bit anchor of the format's family (Sec. 3.5: MXINT8 or MXFP8)."""
    return "int8" if FORMATS[fmt][0] == 0 else "e4m3"


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([
            "gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math",
            "-ffp-contract=off", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None
_lock = threading.Lock()


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            c_int, c_sz, c_vp, c_dbl, c_u = (ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p,
                                             ctypes.c_double, ctypes.c_uint)
            L.mxo_emax.argtypes = [c_int] * 3
            L.mxo_emax.restype = c_int
            L.mxo_max_value.argtypes = [c_int] * 3
            L.mxo_max_value.restype = c_dbl
            L.mxo_decode.argtypes = [c_int, c_int, c_int, c_u]
            L.mxo_decode.restype = c_dbl
            L.mxo_quantize_elem.argtypes = [c_int, c_int, c_int, c_dbl]
            L.mxo_quantize_elem.restype = c_u
            L.mxo_slice_scale_elem.argtypes = [c_int] * 5 + [c_u]
            L.mxo_slice_scale_elem.restype = c_u
            L.mxo_quantize.argtypes = [c_vp, c_int, c_sz, c_int, c_int, c_int, c_int, c_vp, c_vp]
            L.mxo_slice_scale.argtypes = [c_vp, c_vp, c_sz, c_int] + [c_int] * 5 + [c_vp, c_vp]
            L.mxo_dequantize.argtypes = [c_vp, c_vp, c_sz, c_int, c_int, c_int, c_int, c_vp, c_int]
            L.mxo_fake_quant.argtypes = [c_vp, c_int, c_sz, c_int, c_int, c_int, c_int, c_int, c_vp]
            L.mxo_fake_quant_bwd.argtypes = [c_vp, c_int, c_sz, c_vp]
            L.mxo_pack.argtypes = [c_vp, c_sz, c_int, c_vp]
            L.mxo_tile_scales.argtypes = [c_vp, c_sz, c_sz, c_vp]
            L.mxo_unpack.argtypes = [c_vp, c_sz, c_int, c_vp]
            _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def _src(x: np.ndarray):
    """FP32 arrays are float32; BF16 arrays are uint16 bit patterns."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:
        return x, BF16
    raise TypeError("oracle inputs are float32 or uint16 (BF16 bit patterns)")


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError("%s: oracle rejected the arguments (%d)" % (what, rc))


# ---- scalar helpers (used by the element-level pins) ----------------------------------

def emax(fmt: str) -> int:
    return lib().mxo_emax(*FORMATS[fmt])


def max_value(fmt: str) -> float:
    return lib().mxo_max_value(*FORMATS[fmt])


def decode(fmt: str, code: int) -> float:
    return lib().mxo_decode(*FORMATS[fmt], int(code))


def decode_table(fmt: str) -> np.ndarray:
    return np.array([decode(fmt, c) for c in range(1 << bits(fmt))], dtype=np.float64)


def quantize_elem(fmt: str, r: float) -> int:
    return lib().mxo_quantize_elem(*FORMATS[fmt], float(r))


def slice_scale_elem(src_fmt: str, dst_fmt: str, code: int) -> int:
    kh, ah, mh = FORMATS[src_fmt]
    kl, al, ml = FORMATS[dst_fmt]
    assert kh == kl
    return lib().mxo_slice_scale_elem(kh, ah, mh, al, ml, int(code))


# ---- array entry points ---------------------------------------------------------------

def quantize(x: np.ndarray, fmt: str, block: int = 32):
    """Q_f (Eq. 1-3): returns (codes uint8[n], one per byte; scales uint8[n/block])."""
    x, dt = _src(x)
    n = x.size
    codes = np.empty(n, np.uint8)
    scales = np.empty(n // block if block > 0 else 0, np.uint8)
    _check(lib().mxo_quantize(_ptr(x), dt, n, *FORMATS[fmt], block, _ptr(codes), _ptr(scales)),
           "quantize")
    return codes, scales


def slice_scale(codes: np.ndarray, scales: np.ndarray, src_fmt: str, dst_fmt: str,
                block: int = 32):
    """Q_{h->l} (Eq. 4-5) on one-code-per-byte arrays."""
    kh, ah, mh = FORMATS[src_fmt]
    kl, al, ml = FORMATS[dst_fmt]
    if kh != kl:
        raise ValueError("slice_scale: formats of different families")
    codes = np.ascontiguousarray(codes, np.uint8)
    scales = np.ascontiguousarray(scales, np.uint8)
    out_c = np.empty_like(codes)
    out_s = np.empty_like(scales)
    _check(lib().mxo_slice_scale(_ptr(codes), _ptr(scales), codes.size, block, kh, ah, mh, al, ml,
                                 _ptr(out_c), _ptr(out_s)), "slice_scale")
    return out_c, out_s


def dequantize(codes: np.ndarray, scales: np.ndarray, fmt: str, block: int = 32,
               out_dtype: int = F32) -> np.ndarray:
    """V^ = X P; float32 array, or uint16 BF16 bit patterns when out_dtype == BF16."""
    codes = np.ascontiguousarray(codes, np.uint8)
    scales = np.ascontiguousarray(scales, np.uint8)
    out = np.empty(codes.size, np.float32 if out_dtype == F32 else np.uint16)
    _check(lib().mxo_dequantize(_ptr(codes), _ptr(scales), codes.size, *FORMATS[fmt], block,
                                _ptr(out), out_dtype), "dequantize")
    return out


def fake_quant(x: np.ndarray, fmt: str, block: int = 32, mode: int = FQ_DIRECT) -> np.ndarray:
    """Eq. 6 forward in dequantized form; output has the input's type."""
    x, dt = _src(x)
    out = np.empty_like(x)
    _check(lib().mxo_fake_quant(_ptr(x), dt, x.size, *FORMATS[fmt], block, mode, _ptr(out)),
           "fake_quant")
    return out


def fake_quant_bwd(g: np.ndarray) -> np.ndarray:
    g, dt = _src(g)
    out = np.empty_like(g)
    lib().mxo_fake_quant_bwd(_ptr(g), dt, g.size, _ptr(out))
    return out


def tile_scales(scales: np.ndarray, rows: int, kblocks: int) -> np.ndarray:
    """Row-major [rows, kblocks] scale bytes in the 128 x 4 tiled order of a block-scaled matmul."""
    scales = np.ascontiguousarray(scales, np.uint8)
    assert scales.size == rows * kblocks
    out = np.empty(-(-rows // 128) * -(-kblocks // 4) * 512, np.uint8)
    lib().mxo_tile_scales(_ptr(scales), rows, kblocks, _ptr(out))
    return out


def pack(codes: np.ndarray, fmt_bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.uint8)
    out = np.empty(codes.size * fmt_bits // 8, np.uint8)
    _check(lib().mxo_pack(_ptr(codes), codes.size, fmt_bits, _ptr(out)), "pack")
    return out


def unpack(packed: np.ndarray, n: int, fmt_bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, np.uint8)
    out = np.empty(n, np.uint8)
    lib().mxo_unpack(_ptr(packed), n, fmt_bits, _ptr(out))
    return out
