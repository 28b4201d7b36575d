"""The C-ABI library on a machine without a GPU: it loads, exports every function the public header
declares, and its host-side argument checks answer before anything is launched (no call here can
reach a kernel launch: each one is rejected on the host, or has n == 0)."""
import ctypes
import os
import re

import pytest

import paper_2604_00529_b200 as mxq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
OK, E_NULL, E_FORMAT, E_BLOCK, E_SIZE, E_ALIGN, E_PAIR = 0, -1, -2, -3, -4, -5, -6


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mxq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mxq_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def L():
    return mxq.load_library()


def test_every_declared_function_is_exported(L):
    names = _declared_functions()
    assert {"mxq_quantize", "mxq_slice_scale", "mxq_dequantize", "mxq_fake_quant", "mxq_fake_quant_bwd",
            "mxq_slice_scale_batched"} <= set(names)
    for name in names:
        assert hasattr(L, name), name


def test_size_helpers(L):
    assert [L.mxq_format_bits(f) for f in range(13)] == [8, 6, 4, 8, 6, 6, 4, 7, 5, 3, 2, 7, 5]
    assert L.mxq_format_bits(13) == 0 and L.mxq_format_bits(-1) == 0
    assert L.mxq_codes_bytes(64, mxq.FORMATS["int6"]) == 48
    assert L.mxq_codes_bytes(1 << 31, mxq.FORMATS["e2m1"]) == 1 << 30
    assert L.mxq_scales_bytes(4096, 32) == 128 and L.mxq_scales_bytes(4096, 0) == 0
    assert [L.mxq_block_supported(b) for b in (8, 16, 32, 48, 64, 128, 256)] == [0, 1, 1, 0, 1, 1, 0]
    assert b"MXQ_OK" in L.mxq_status_string(0) and b"unknown" in L.mxq_status_string(-99)
    for st in range(-8, 0):
        assert L.mxq_status_string(st).startswith(b"MXQ_ERR_")


def test_argument_checks_answer_on_the_host(L):
    A = 0x1000                       # an aligned, never dereferenced address
    q = L.mxq_quantize
    assert q(A, 0, 64, 99, 32, A, A, None) == E_FORMAT
    assert q(A, 7, 64, 0, 32, A, A, None) == E_FORMAT
    assert q(A, 0, 64, 0, 48, A, A, None) == E_BLOCK
    assert q(A, 0, 65, 0, 32, A, A, None) == E_SIZE
    assert q(None, 0, 64, 0, 32, A, A, None) == E_NULL
    assert q(A + 16, 0, 64, 0, 32, A, A, None) == E_ALIGN
    assert q(A, 0, 64, 0, 32, A, A + 8, None) == E_ALIGN
    assert q(None, 0, 0, 0, 32, None, None, None) == OK           # empty tensor: nothing to do
    ss = L.mxq_slice_scale
    F = mxq.FORMATS
    assert ss(A, A, 64, 32, F["int8"], F["e2m1"], A, A, None) == E_PAIR      # families differ
    assert ss(A, A, 64, 32, F["int4"], F["int8"], A, A, None) == E_PAIR      # low to high
    assert ss(A, A, 64, 32, F["e2m1"], F["e2m3"], A, A, None) == E_PAIR      # codes would widen
    assert ss(A, A, 64, 32, F["int8"], F["int4"], None, A, None) == E_NULL
    assert ss(A, A, 64, 32, F["int8"], F["int4"], A + 4, A, None) == E_ALIGN
    assert ss(A, A, 48, 16, F["int8"], F["int4"], A, A, None) == E_SIZE      # code units are 32 wide
    multi = L.mxq_slice_scale_multi
    import ctypes as C
    two = (C.c_int * 2)(F["int6"], F["int4"])
    bad = (C.c_int * 2)(F["int6"], F["e2m1"])
    ptrs = (C.c_void_p * 2)(A, A)
    nul = (C.c_void_p * 2)(A, None)
    assert multi(A, A, 64, 32, F["int8"], 2, bad, ptrs, ptrs, None) == E_PAIR
    assert multi(A, A, 64, 32, F["int8"], 2, two, nul, ptrs, None) == E_NULL
    assert multi(A, A, 64, 32, F["int8"], 9, two, ptrs, ptrs, None) == E_SIZE
    assert multi(A, A, 64, 32, F["int8"], 0, None, None, None, None) == OK
    assert multi(A, A, 65, 32, F["int8"], 2, two, ptrs, ptrs, None) == E_SIZE
    assert multi(A, A, 64, 32, F["int8"], 2, None, ptrs, ptrs, None) == E_NULL
    ts = L.mxq_tile_scales
    assert ts(None, 0, 4, None, None) == OK and ts(A, 128, 0, A, None) == OK
    assert ts(None, 128, 4, A, None) == E_NULL and ts(A, 128, 4, None, None) == E_NULL
    assert ts(A + 4, 128, 4, A, None) == E_ALIGN and ts(A, 128, 4, A + 8, None) == E_ALIGN
    assert L.mxq_tiled_scales_bytes(1, 1) == 512 and L.mxq_tiled_scales_bytes(129, 5) == 2 * 2 * 512
    assert L.mxq_tiled_scales_bytes(8192, 256) == 8192 * 256
    qt = L.mxq_quantize_tiled                       # (src, dtype, rows, cols, fmt, block, codes, tiled, stream)
    assert qt(None, 1, 0, 64, F["e4m3"], 32, None, None, None) == OK
    assert qt(A, 1, 2, 64, F["int8"], 32, A, A, None) == E_FORMAT            # MXFP formats only
    assert qt(A, 7, 2, 64, F["e4m3"], 32, A, A, None) == E_FORMAT
    assert qt(A, 1, 2, 64, F["e4m3"], 64, A, A, None) == E_BLOCK             # tiles are defined for block 32
    assert qt(A, 1, 2, 48, F["e4m3"], 32, A, A, None) == E_SIZE
    assert qt(A, 1, 1 << 31, 64, F["e4m3"], 32, A, A, None) == E_SIZE        # 2^32 blocks
    assert qt(A, 1, 2, 64, F["e4m3"], 32, A, None, None) == E_NULL
    assert qt(A, 1, 2, 64, F["e4m3"], 32, A, A + 8, None) == E_ALIGN
    st = L.mxq_slice_scale_tiled                    # (codes, scales, rows, cols, block, src, dst, out_codes, out_tiled, stream)
    assert st(None, None, 4, 0, 32, F["e4m3"], F["e2m1"], None, None, None) == OK
    assert st(A, A, 2, 64, 32, F["int8"], F["int4"], A, A, None) == E_FORMAT
    assert st(A, A, 2, 64, 32, F["e2m1"], F["e4m3"], A, A, None) == E_PAIR
    assert st(A, A, 2, 64, 16, F["e4m3"], F["e2m1"], A, A, None) == E_BLOCK
    assert st(A, A, 2, 80, 32, F["e4m3"], F["e2m1"], A, A, None) == E_SIZE
    assert st(A, None, 2, 64, 32, F["e4m3"], F["e2m1"], A, A, None) == E_NULL
    assert st(A, A, 2, 64, 32, F["e4m3"], F["e2m1"], A + 16, A, None) == E_ALIGN
    stb = L.mxq_slice_scale_tiled_batched           # (items, count, block, src, dst, stream)
    assert stb(None, 0, 32, F["e4m3"], F["e2m1"], None) == OK
    assert stb(None, 2, 32, F["e4m3"], F["e2m1"], None) == E_NULL
    assert stb(None, -1, 32, F["e4m3"], F["e2m1"], None) == E_SIZE
    assert stb(None, 2, 64, F["e4m3"], F["e2m1"], None) == E_BLOCK
    assert stb(None, 2, 32, F["int8"], F["int4"], None) == E_FORMAT
    assert stb(None, 2, 32, F["e2m1"], F["e4m3"], None) == E_PAIR
    from paper_2604_00529_b200.binding import _TiledItem
    one = (_TiledItem * 1)(_TiledItem(A, A, 2, 48, A, A))
    assert stb(one, 1, 32, F["e4m3"], F["e2m1"], None) == E_SIZE
    one = (_TiledItem * 1)(_TiledItem(A, A, 2, 64, A, None))
    assert stb(one, 1, 32, F["e4m3"], F["e2m1"], None) == E_NULL
    one = (_TiledItem * 1)(_TiledItem(A, A, 2, 64, A, A + 8))
    assert stb(one, 1, 32, F["e4m3"], F["e2m1"], None) == E_ALIGN
    one = (_TiledItem * 1)(_TiledItem(None, None, 0, 64, None, None))
    assert stb(one, 1, 32, F["e4m3"], F["e2m1"], None) == OK                 # an empty matrix: nothing to do
    dq = L.mxq_dequantize
    assert dq(A, A, 64, F["int4"], 32, A, 5, None) == E_FORMAT
    assert dq(A, None, 64, F["int4"], 32, A, 0, None) == E_NULL
    fq = L.mxq_fake_quant
    assert fq(A, 1, 64, F["e2m1"], 32, 2, A, None) == E_FORMAT               # unknown mode
    assert fq(A, 1, 64, F["e2m1"], 32, 1, None, None) == E_NULL
    fqb = L.mxq_fake_quant_batched
    assert fqb(None, 0, 1, F["e2m1"], 32, 0, None) == OK
    assert fqb(None, 3, 1, F["e2m1"], 32, 0, None) == E_NULL
    assert fqb(None, -2, 1, F["e2m1"], 32, 0, None) == E_SIZE
    assert fqb(None, 3, 1, F["e2m1"], 48, 0, None) == E_BLOCK
    assert fqb(None, 3, 1, 77, 32, 0, None) == E_FORMAT
    assert fqb(None, 3, 1, F["e2m1"], 32, 5, None) == E_FORMAT
    from paper_2604_00529_b200.binding import _DqItem, _QItem
    qb = L.mxq_quantize_batched                      # (items, count, dtype, fmt, block, stream)
    assert qb(None, 0, 1, F["int8"], 32, None) == OK
    assert qb(None, 3, 1, F["int8"], 32, None) == E_NULL
    assert qb(None, -1, 1, F["int8"], 32, None) == E_SIZE
    assert qb(None, 3, 1, F["int8"], 48, None) == E_BLOCK
    assert qb(None, 3, 7, F["int8"], 32, None) == E_FORMAT
    assert qb(None, 3, 1, 99, 32, None) == E_FORMAT
    assert qb((_QItem * 1)(_QItem(A, 48, A, A)), 1, 1, F["int8"], 32, None) == E_SIZE
    assert qb((_QItem * 1)(_QItem(A, 64, None, A)), 1, 1, F["int8"], 32, None) == E_NULL
    assert qb((_QItem * 1)(_QItem(A + 16, 64, A, A)), 1, 1, F["int8"], 32, None) == E_ALIGN
    assert qb((_QItem * 1)(_QItem(None, 0, None, None)), 1, 1, F["int8"], 32, None) == OK    # empty tensor: nothing to do
    dqb = L.mxq_dequantize_batched                   # (items, count, fmt, block, dtype, stream)
    assert dqb(None, 0, F["int4"], 32, 1, None) == OK
    assert dqb(None, 2, F["int4"], 32, 1, None) == E_NULL
    assert dqb(None, -1, F["int4"], 32, 1, None) == E_SIZE
    assert dqb(None, 2, F["int4"], 24, 1, None) == E_BLOCK
    assert dqb(None, 2, F["int4"], 32, 3, None) == E_FORMAT
    assert dqb((_DqItem * 1)(_DqItem(A, A, 16, A)), 1, F["int4"], 16, 1, None) == E_SIZE      # packed codes: multiples of 32
    assert dqb((_DqItem * 1)(_DqItem(A, None, 64, A)), 1, F["int4"], 32, 1, None) == E_NULL
    assert dqb((_DqItem * 1)(_DqItem(A, A + 8, 64, A)), 1, F["int4"], 32, 1, None) == E_ALIGN
    from paper_2604_00529_b200.binding import _PairItem
    pb = L.mxq_slice_scale_pair_batched             # (items, count, block, src, dst1, dst2, stream)
    assert pb(None, 0, 32, F["int8"], F["int6"], F["int4"], None) == OK
    assert pb(None, 2, 32, F["int8"], F["int6"], F["int4"], None) == E_NULL
    assert pb(None, -1, 32, F["int8"], F["int6"], F["int4"], None) == E_SIZE
    assert pb(None, 2, 16, F["int8"], F["int6"], F["int4"], None) == E_BLOCK
    assert pb(None, 2, 32, F["int8"], F["int6"], F["e2m1"], None) == E_PAIR
    assert pb(None, 2, 32, F["int8"], 44, F["int4"], None) == E_FORMAT
    assert pb((_PairItem * 1)(_PairItem(A, A, 65, A, A, A, A)), 1, 32, F["int8"], F["int6"], F["int4"], None) == E_SIZE
    assert pb((_PairItem * 1)(_PairItem(A, A, 64, A, A, None, A)), 1, 32, F["int8"], F["int6"], F["int4"], None) == E_NULL
    assert pb((_PairItem * 1)(_PairItem(A, A, 64, A, A, A, A + 8)), 1, 32, F["int8"], F["int6"], F["int4"], None) == E_ALIGN
    bw = L.mxq_fake_quant_bwd
    assert bw(A, 1, 64, A, None) == OK                                       # in place: no launch
    assert bw(A, 1, 64, None, None) == E_NULL
    for fn in (L.mxq_slice_scale_batched, L.mxq_slice_scale_batched_static):
        assert fn(None, 3, 32, F["int8"], F["int4"], None) == E_NULL
        assert fn(None, -1, 32, F["int8"], F["int4"], None) == E_SIZE
        assert fn(None, 0, 32, F["int8"], F["int4"], None) == OK
        assert fn(None, 3, 16, F["int8"], F["int4"], None) == E_BLOCK
        assert fn(None, 3, 32, F["int8"], F["e2m1"], None) == E_PAIR
    assert L.mxq_slice_scale_batched_static(None, 1025, 32, F["int8"], F["int4"], None) == E_SIZE


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError):
        mxq.quantize(torch.zeros(64), "int8")
    with pytest.raises((TypeError, ValueError)):
        mxq.fake_quant(torch.zeros(64, dtype=torch.float16), "int8")


def test_header_is_plain_c_and_links(tmp_path):
    """include/mxq.h compiled as C99 by gcc, every declared function referenced, linked against libmxq.so
    and run: the program only calls the size helpers and the host-side checks (no launch)."""
    import subprocess
    names = _declared_functions()
    refs = "\n".join("    p[%d] = (fn)%s;" % (i, n) for i, n in enumerate(names))
    src = tmp_path / "consumer.c"
    src.write_text("""
#include <stdio.h>
#include "mxq.h"
typedef void (*fn)(void);
int main(void)
{
    fn p[%d];
%s
    for (int i = 0; i < %d; ++i) if (!p[i]) return 2;
    if (mxq_format_bits(MXQ_FP6_E2M3) != 6 || mxq_codes_bytes(64, MXQ_INT4) != 32) return 3;
    if (mxq_quantize(0, MXQ_BF16, 64, MXQ_INT8, 32, 0, 0, 0) != MXQ_ERR_NULL) return 4;
    if (mxq_slice_scale(0, 0, 64, 32, MXQ_INT4, MXQ_INT8, 0, 0, 0) != MXQ_ERR_PAIR) return 5;
    printf("%%s\\n", mxq_status_string(MXQ_ERR_PAIR));
    return 0;
}
""" % (len(names), refs, len(names)))
    exe = tmp_path / "consumer"
    libdir = os.path.dirname(mxq.library_path())
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-l:libmxq.so", "-Wl,-rpath," + libdir])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stderr)
    assert "MXQ_ERR_PAIR" in out.stdout
