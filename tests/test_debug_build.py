"""The bounds-checked build of the library (libmxq_debug.so, -DMXQ_DEBUG): every entry point on the
sizes where index arithmetic goes wrong first -- one block, one warp's worth, ragged tails, several
tiles -- with exactly sized buffers.  With correct arguments the checker must have looked at every
launch and counted no violation, and the results must still be the oracle's.  The checker's teeth are
shown with the library's own test hook, which registers every range a few bytes short: the kernels'
last (legitimate) accesses are then counted and skipped, while no access ever leaves a real buffer."""
import ctypes
import os

import numpy as np
import pytest
import torch

from oracle import mxq_oracle as orc
from paper_2604_00529_b200 import inputs
from paper_2604_00529_b200.binding import FORMATS, _DqItem, _FqItem, _Item, _QItem

from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(os.path.dirname(HERE), "paper_2604_00529_b200", "libmxq_debug.so")


class Info(ctypes.Structure):
    _fields_ = [("enabled", ctypes.c_int), ("checked_launches", ctypes.c_uint), ("violations", ctypes.c_uint),
                ("first_address", ctypes.c_ulonglong), ("first_bytes", ctypes.c_uint)]


@pytest.fixture(scope="module")
def D():
    if not os.path.exists(LIB):
        pytest.fail("libmxq_debug.so is not built: python -m paper_2604_00529_b200.build --debug")
    L = ctypes.CDLL(LIB)
    vp, sz, i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    L.mxq_quantize.argtypes = [vp, i, sz, i, i, vp, vp, vp]
    L.mxq_slice_scale.argtypes = [vp, vp, sz, i, i, i, vp, vp, vp]
    L.mxq_dequantize.argtypes = [vp, vp, sz, i, i, vp, i, vp]
    L.mxq_fake_quant.argtypes = [vp, i, sz, i, i, i, vp, vp]
    L.mxq_fake_quant_bwd.argtypes = [vp, i, sz, vp, vp]
    L.mxq_slice_scale_batched.argtypes = [ctypes.POINTER(_Item), i, i, i, i, vp]
    L.mxq_slice_scale_batched_static.argtypes = [ctypes.POINTER(_Item), i, i, i, i, vp]
    L.mxq_quantize_batched.argtypes = [ctypes.POINTER(_QItem), i, i, i, i, vp]
    L.mxq_dequantize_batched.argtypes = [ctypes.POINTER(_DqItem), i, i, i, i, vp]
    L.mxq_fake_quant_batched.argtypes = [ctypes.POINTER(_FqItem), i, i, i, i, i, vp]
    L.mxq_quantize_tiled.argtypes = [vp, i, sz, sz, i, i, vp, vp, vp]
    L.mxq_tiled_scales_bytes.argtypes = [sz, sz]
    L.mxq_tiled_scales_bytes.restype = sz
    L.mxq_debug_report.argtypes = [ctypes.POINTER(Info), i]
    L.mxq_debug_trim_ranges.argtypes = [sz]
    return L


def report(L, reset=True):
    info = Info()
    assert L.mxq_debug_report(ctypes.byref(info), 1 if reset else 0) == 0
    return info


def u8(nbytes):
    return torch.empty(nbytes, dtype=torch.uint8, device="cuda")          # exactly sized: no slack behind the data


def P(t):
    return t.data_ptr()


SIZES = [32, 64, 32 * 31, 32 * 32, 32 * 33, 32 * 64, 32 * 65, 32 * 2051]   # one block ... tiles plus a ragged tail


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("anchor,low", [("int8", "int4"), ("int8", "int6"), ("e4m3", "e2m3"), ("e4m3", "e2m1"), ("int8", "int7")])
def test_single_tensor_entry_points_stay_inside_their_buffers(D, n, anchor, low):
    stream = torch.cuda.current_stream().cuda_stream
    x = inputs.to_bf16_bits((np.random.default_rng(n).standard_normal(n) * 0.3).astype(np.float32))
    xd = to_dev(x)
    report(D)
    codes, scales = u8(n), u8(n // 32)
    assert D.mxq_quantize(P(xd), 1, n, FORMATS[anchor], 32, P(codes), P(scales), stream) == 0
    b = orc.bits(low)
    lc, ls = u8(n * b // 8), u8(n // 32)
    assert D.mxq_slice_scale(P(codes), P(scales), n, 32, FORMATS[anchor], FORMATS[low], P(lc), P(ls), stream) == 0
    y = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    y32 = torch.empty(n, dtype=torch.float32, device="cuda")
    assert D.mxq_dequantize(P(lc), P(ls), n, FORMATS[low], 32, P(y), 1, stream) == 0
    assert D.mxq_dequantize(P(lc), P(ls), n, FORMATS[low], 32, P(y32), 0, stream) == 0
    f = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    g = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    assert D.mxq_fake_quant(P(xd), 1, n, FORMATS[low], 32, 1, P(f), stream) == 0
    assert D.mxq_fake_quant_bwd(P(f), 1, n, P(g), stream) == 0
    info = report(D)
    assert info.enabled == 1 and info.checked_launches == 6
    assert info.violations == 0, "first bad access: %#x (%d bytes)" % (info.first_address, info.first_bytes)
    wc, ws = orc.quantize(x, anchor)
    w4, s4 = orc.slice_scale(wc, ws, anchor, low)
    assert np.array_equal(to_host(codes), orc.pack(wc, 8)) and np.array_equal(to_host(scales), ws)
    assert np.array_equal(to_host(lc), orc.pack(w4, b)) and np.array_equal(to_host(ls), s4)
    want = orc.dequantize(w4, s4, low, out_dtype=orc.BF16)
    assert np.array_equal(to_host(y), want) and np.array_equal(to_host(f), want) and np.array_equal(to_host(g), want)
    assert np.array_equal(to_host(y32).view(np.uint32), orc.dequantize(w4, s4, low).view(np.uint32))


def test_batched_entry_points_stay_inside_their_buffers(D):
    stream = torch.cuda.current_stream().cuda_stream
    sizes = [32, 32 * 65, 64, 32 * 700, 32 * 33, 32 * 2051, 32 * 7]
    rng = np.random.default_rng(3)
    xs = [inputs.to_bf16_bits((rng.standard_normal(n) * 2.0 ** rng.integers(-8, 8)).astype(np.float32)) for n in sizes]
    xd = [to_dev(x) for x in xs]
    codes = [u8(n) for n in sizes]
    scales = [u8(n // 32) for n in sizes]
    lc = [u8(n // 2) for n in sizes]
    ls = [u8(n // 32) for n in sizes]
    lc2 = [u8(n // 2) for n in sizes]
    ls2 = [u8(n // 32) for n in sizes]
    y = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for n in sizes]
    f = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for n in sizes]
    k = len(sizes)
    report(D)
    q = (_QItem * k)(*[_QItem(P(xd[j]), sizes[j], P(codes[j]), P(scales[j])) for j in range(k)])
    assert D.mxq_quantize_batched(q, k, 1, FORMATS["e4m3"], 32, stream) == 0
    it = (_Item * k)(*[_Item(P(codes[j]), P(scales[j]), sizes[j], P(lc[j]), P(ls[j])) for j in range(k)])
    assert D.mxq_slice_scale_batched(it, k, 32, FORMATS["e4m3"], FORMATS["e2m1"], stream) == 0
    it2 = (_Item * k)(*[_Item(P(codes[j]), P(scales[j]), sizes[j], P(lc2[j]), P(ls2[j])) for j in range(k)])
    assert D.mxq_slice_scale_batched_static(it2, k, 32, FORMATS["e4m3"], FORMATS["e2m1"], stream) == 0
    dq = (_DqItem * k)(*[_DqItem(P(lc[j]), P(ls[j]), sizes[j], P(y[j])) for j in range(k)])
    assert D.mxq_dequantize_batched(dq, k, FORMATS["e2m1"], 32, 1, stream) == 0
    fq = (_FqItem * k)(*[_FqItem(P(xd[j]), P(f[j]), sizes[j]) for j in range(k)])
    assert D.mxq_fake_quant_batched(fq, k, 1, FORMATS["e2m1"], 32, 1, stream) == 0
    rows, cols = 130, 160                                   # edge tiles in both directions
    xm = to_dev(inputs.to_bf16_bits(rng.standard_normal(rows * cols).astype(np.float32)))
    tc, tt = u8(rows * cols), u8(D.mxq_tiled_scales_bytes(rows, cols // 32))
    assert D.mxq_quantize_tiled(P(xm), 1, rows, cols, FORMATS["e4m3"], 32, P(tc), P(tt), stream) == 0
    info = report(D)
    assert info.enabled == 1 and info.checked_launches == 6
    assert info.violations == 0, "first bad access: %#x (%d bytes)" % (info.first_address, info.first_bytes)
    for j, x in enumerate(xs):
        wc, ws = orc.quantize(x, "e4m3")
        w4, s4 = orc.slice_scale(wc, ws, "e4m3", "e2m1")
        assert np.array_equal(to_host(lc[j]), orc.pack(w4, 4)) and np.array_equal(to_host(ls[j]), s4), j
        assert np.array_equal(to_host(lc2[j]), orc.pack(w4, 4)) and np.array_equal(to_host(ls2[j]), s4), j
        want = orc.dequantize(w4, s4, "e2m1", out_dtype=orc.BF16)
        assert np.array_equal(to_host(y[j]), want) and np.array_equal(to_host(f[j]), want), j


def test_the_checker_counts_and_skips_what_leaves_a_registered_range(D):
    """Ranges registered 32 bytes short: the kernel's stores and loads of the last 32 bytes of each
    buffer are outside them, are counted, and are skipped (the output keeps its fill there)."""
    stream = torch.cuda.current_stream().cuda_stream
    n = 32 * 64
    x = inputs.to_bf16_bits(np.random.default_rng(1).standard_normal(n).astype(np.float32))
    xd = to_dev(x)
    y = torch.full((n,), 7.0, dtype=torch.bfloat16, device="cuda")
    report(D)
    assert D.mxq_debug_trim_ranges(32) == 1
    try:
        assert D.mxq_fake_quant(P(xd), 1, n, FORMATS["int8"], 32, 0, P(y), stream) == 0
        info = report(D)
    finally:
        D.mxq_debug_trim_ranges(0)
    assert info.checked_launches == 1 and info.violations == 2            # one load and one store of 32 bytes
    assert info.first_bytes == 32 and info.first_address in (P(xd) + 2 * n - 32, P(y) + 2 * n - 32)
    got = to_host(y)
    want = orc.fake_quant(x, "int8")
    assert np.array_equal(got[:-16], want[:-16])
    assert np.all(got[-16:] == 0x40E0)                                     # 7.0 in BF16: the store was skipped
    # and with whole ranges again the same call is clean
    assert D.mxq_fake_quant(P(xd), 1, n, FORMATS["int8"], 32, 0, P(y), stream) == 0
    info = report(D)
    assert info.violations == 0 and np.array_equal(to_host(y), want)


def test_release_build_reports_that_it_is_not_a_debug_build():
    import paper_2604_00529_b200 as mxq
    L = mxq.load_library()
    L.mxq_debug_report.argtypes = [ctypes.POINTER(Info), ctypes.c_int]
    info = Info()
    assert L.mxq_debug_report(ctypes.byref(info), 0) == 0 and info.enabled == 0 and info.violations == 0
    L.mxq_debug_trim_ranges.argtypes = [ctypes.c_size_t]
    assert L.mxq_debug_trim_ranges(64) == 0
