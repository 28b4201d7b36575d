"""Helpers of the GPU parity tests: numpy <-> device marshalling through the C-ABI binding, with
guard bytes around every output buffer so that an out-of-range store fails the test."""
from __future__ import annotations

import numpy as np
import torch

import paper_2604_00529_b200 as mxq
from oracle import mxq_oracle as orc

GUARD = 256          # bytes on each side of an output buffer (keeps the 32-byte alignment)
PATTERN = 0xA5

INT_FORMATS = ["int8", "int7", "int6", "int5", "int4", "int3", "int2"]
FP_FORMATS = ["e4m3", "e3m3", "e3m2", "e2m3", "e2m2", "e2m1"]
ALL_FORMATS = INT_FORMATS + FP_FORMATS
MAIN_FORMATS = ["int8", "int6", "int4", "e4m3", "e3m2", "e2m3", "e2m1"]


def ss_pairs(all_pairs: bool = False):
    """(src, dst) pairs: from the 8-bit anchors, or every legal same-family pair."""
    out = []
    for fam in (INT_FORMATS, FP_FORMATS):
        for h in fam:
            if not all_pairs and h not in ("int8", "e4m3"):
                continue
            for l in fam:
                if orc.emax(h) >= orc.emax(l) and orc.bits(l) <= orc.bits(h):
                    out.append((h, l))
    return out


def to_dev(x: np.ndarray) -> torch.Tensor:
    """float32 array -> float32 tensor; uint16 BF16 bit patterns -> bfloat16 tensor; uint8 -> uint8."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(x).cuda()


def to_host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


class Guarded:
    """A device buffer of `nbytes` bytes (viewed as `dtype`) between two guard zones."""

    def __init__(self, nbytes: int, dtype=torch.uint8):
        self.raw = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.nbytes = nbytes
        self.view = self.raw[GUARD:GUARD + nbytes].view(dtype)

    def check(self):
        raw = self.raw.cpu().numpy()
        assert np.all(raw[:GUARD] == PATTERN), "store below the output buffer"
        assert np.all(raw[GUARD + self.nbytes:] == PATTERN), "store beyond the output buffer"


def gpu_quantize(x: np.ndarray, fmt: str, block: int = 32):
    n = x.size
    codes = Guarded(mxq.codes_bytes(n, fmt))
    scales = Guarded(n // block)
    mxq.quantize(to_dev(x), fmt, block, codes.view, scales.view)
    torch.cuda.synchronize()
    codes.check()
    scales.check()
    return to_host(codes.view), to_host(scales.view)


def gpu_slice_scale(packed: np.ndarray, scales: np.ndarray, n: int, src: str, dst: str, block: int = 32):
    oc = Guarded(mxq.codes_bytes(n, dst))
    os_ = Guarded(n // block)
    mxq.slice_scale(to_dev(packed), to_dev(scales), n, src, dst, block, oc.view, os_.view)
    torch.cuda.synchronize()
    oc.check()
    os_.check()
    return to_host(oc.view), to_host(os_.view)


def gpu_dequantize(packed: np.ndarray, scales: np.ndarray, n: int, fmt: str, block: int = 32, bf16: bool = False):
    dt = torch.bfloat16 if bf16 else torch.float32
    dst = Guarded(n * (2 if bf16 else 4), dt)
    mxq.dequantize(to_dev(packed), to_dev(scales), n, fmt, block, dst=dst.view)
    torch.cuda.synchronize()
    dst.check()
    return to_host(dst.view)


def gpu_fake_quant(x: np.ndarray, fmt: str, block: int = 32, mode: int = 0, inplace: bool = False):
    src = to_dev(x)
    if inplace:
        mxq.fake_quant(src, fmt, block, mode, dst=src)
        torch.cuda.synchronize()
        return to_host(src)
    dst = Guarded(x.size * x.itemsize, src.dtype)
    mxq.fake_quant(src, fmt, block, mode, dst=dst.view)
    torch.cuda.synchronize()
    dst.check()
    return to_host(dst.view)


def bits_equal(a: np.ndarray, b: np.ndarray) -> bool:
    """Bit-exact comparison (float32 compared as uint32, so NaN payloads and -0 count)."""
    if a.dtype == np.float32:
        a = a.view(np.uint32)
    if b.dtype == np.float32:
        b = b.view(np.uint32)
    return a.shape == b.shape and bool(np.array_equal(a, b))


def first_diff(a: np.ndarray, b: np.ndarray) -> str:
    if a.dtype == np.float32:
        a = a.view(np.uint32)
    if b.dtype == np.float32:
        b = b.view(np.uint32)
    idx = np.flatnonzero(a != b)
    if idx.size == 0:
        return "equal"
    i = int(idx[0])
    return "%d differences, first at %d: got %r want %r" % (idx.size, i, a[i], b[i])
