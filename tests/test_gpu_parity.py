"""GPU parity: every entry point of libmxq, called through the C-ABI binding, against the CPU
oracle on identical seeded inputs.  Codes, scales and reconstructed values must match bit for bit
(integer and byte work; floating point decides nothing here that both sides do not decide in the
same exact arithmetic, so the tolerance is zero)."""
import numpy as np
import pytest
import torch

import paper_2604_00529_b200 as mxq
from oracle import mxq_oracle as orc
from paper_2604_00529_b200 import inputs

from gpu_util import (ALL_FORMATS, FP_FORMATS, INT_FORMATS, MAIN_FORMATS, Guarded, bits_equal, first_diff, gpu_dequantize,
                      gpu_fake_quant, gpu_quantize, gpu_slice_scale, ss_pairs, to_dev, to_host)

pytestmark = pytest.mark.gpu


def _mixed_f32(nblk, seed, block=32):
    """Blocks at many magnitudes with outliers; spans several warp tiles plus a ragged tail."""
    rng = np.random.default_rng(seed)
    scale = 2.0 ** rng.integers(-30, 30, (nblk, 1))
    x = rng.standard_normal((nblk, block)) * scale
    x[rng.random((nblk, block)) < 0.02] *= 40
    x[rng.random((nblk, block)) < 0.05] = 0
    return x.astype(np.float32).reshape(-1)


def _oracle_packed(x, fmt, block=32):
    c, s = orc.quantize(x, fmt, block)
    return orc.pack(c, orc.bits(fmt)), s


# 64 lane units per warp tile: 2051 blocks of FP32 = 8204 units = 128 tiles + a ragged tail
NBLK = 2051


@pytest.mark.parametrize("fmt", ALL_FORMATS)
@pytest.mark.parametrize("bf16", [False, True])
def test_quantize_random(fmt, bf16):
    x = np.concatenate([_mixed_f32(NBLK, 1), inputs.adversarial_f32()])
    if bf16:
        x = inputs.to_bf16_bits(x)
    got_c, got_s = gpu_quantize(x, fmt)
    want_c, want_s = _oracle_packed(x, fmt)
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, want_c), first_diff(got_c, want_c)


@pytest.mark.parametrize("fmt", ALL_FORMATS)
def test_quantize_every_bf16_pattern(fmt):
    """All 65536 BF16 bit patterns as block elements, under pinned block maxima at several
    exponents (non-finite patterns poison their block, which is part of the contract)."""
    pats = np.arange(65536, dtype=np.uint16)
    blocks = []
    for k in (-126, -60, -9, 0, 3, 9, 90, 127):
        pin = inputs.to_bf16_bits(np.array([1.75 * 2.0 ** k], np.float32))[0]
        body = np.concatenate([pats, np.zeros((-65536) % 31, np.uint16)]).reshape(-1, 31)
        blk = np.concatenate([np.full((body.shape[0], 1), pin, np.uint16), body], axis=1)
        blocks.append(blk.reshape(-1))
    x = np.concatenate(blocks)
    got_c, got_s = gpu_quantize(x, fmt)
    want_c, want_s = _oracle_packed(x, fmt)
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, want_c), first_diff(got_c, want_c)


@pytest.mark.parametrize("fmt", ALL_FORMATS)
def test_quantize_f32_rounding_breakpoints(fmt):
    """FP32 inputs one ulp either side of every rounding breakpoint of the element format, at
    several block scales (the quantizer is a monotone step function: breakpoints suffice)."""
    tab = orc.decode_table(fmt)
    mags = np.unique(np.abs(tab[~np.isnan(tab)]))
    top = orc.max_value(fmt)
    mids = (mags[:-1] + mags[1:]) / 2
    pts = np.concatenate([mags, mids, [top + (mags[-1] - mags[-2]) / 2, top * 1.2]]).astype(np.float32)
    pts = np.concatenate([pts, np.nextafter(pts, np.float32(np.inf)), np.nextafter(pts, np.float32(-np.inf))])
    pts = pts[pts < 2.0 ** (orc.emax(fmt) + 1)]                 # must stay below the pinned maximum's binade
    pts = np.concatenate([pts, -pts])
    pin = np.float32(1.999 * 2.0 ** orc.emax(fmt))              # floor(log2) = e_max -> shared_exp = k
    xs = []
    for k in (-100, -17, 0, 5, 60):
        body = np.concatenate([pts, np.zeros((-pts.size) % 31, np.float32)]).reshape(-1, 31)
        blk = np.concatenate([np.full((body.shape[0], 1), pin, np.float32), body], axis=1)
        xs.append((blk * np.float32(2.0 ** k)).astype(np.float32).reshape(-1))
    x = np.concatenate(xs)
    got_c, got_s = gpu_quantize(x, fmt)
    want_c, want_s = _oracle_packed(x, fmt)
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, want_c), first_diff(got_c, want_c)


@pytest.mark.parametrize("block", [16, 64, 128])
@pytest.mark.parametrize("fmt", ["int8", "int4", "e4m3", "e2m1", "e3m2"])
@pytest.mark.parametrize("bf16", [False, True])
def test_quantize_other_block_sizes(fmt, block, bf16):
    x = _mixed_f32(777, 2, block)
    if bf16:
        x = inputs.to_bf16_bits(x)
    got_c, got_s = gpu_quantize(x, fmt, block)
    want_c, want_s = _oracle_packed(x, fmt, block)
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, want_c), first_diff(got_c, want_c)


# ---------------------------------------------------------------------------------------------
# Slice-and-Scale
# ---------------------------------------------------------------------------------------------

def _all_codes_input(src, nblk_extra=1000, seed=3):
    """Every code value of the source format (NaN codes and -2^(b-1) included) in every lane
    position, then random codes; scale bytes cover 0, the saturating range and 0xFF."""
    nb = orc.bits(src)
    rng = np.random.default_rng(seed)
    allc = np.arange(1 << nb, dtype=np.uint8)
    rolled = np.concatenate([np.roll(np.resize(allc, 256), r) for r in range(32)])
    codes = np.concatenate([rolled, rng.integers(0, 1 << nb, 32 * nblk_extra).astype(np.uint8)])
    nblk = codes.size // 32
    scales = rng.integers(0, 256, nblk).astype(np.uint8)
    scales[:8] = [0, 1, 248, 250, 252, 253, 254, 255]
    return codes, scales


@pytest.mark.parametrize("src,dst", ss_pairs(all_pairs=True), ids=lambda v: v)
def test_slice_scale_all_codes(src, dst):
    codes, scales = _all_codes_input(src)
    n = codes.size
    got_c, got_s = gpu_slice_scale(orc.pack(codes, orc.bits(src)), scales, n, src, dst)
    want_c, want_s = orc.slice_scale(codes, scales, src, dst)
    want_c = orc.pack(want_c, orc.bits(dst))
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, want_c), first_diff(got_c, want_c)


@pytest.mark.parametrize("src,dst", ss_pairs(), ids=lambda v: v)
def test_slice_scale_of_quantized_tensor(src, dst):
    """The paper's path: anchor = Q_A(V) on the GPU, then Q_{A->t}; both stages against the oracle."""
    x = inputs.to_bf16_bits(_mixed_f32(NBLK, 4))
    n = x.size
    a_c, a_s = gpu_quantize(x, src)
    got_c, got_s = gpu_slice_scale(a_c, a_s, n, src, dst)
    oc, os_ = orc.quantize(x, src)
    want_c, want_s = orc.slice_scale(oc, os_, src, dst)
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, orc.pack(want_c, orc.bits(dst))), first_diff(got_c, orc.pack(want_c, orc.bits(dst)))


@pytest.mark.parametrize("block", [16, 64, 128])
@pytest.mark.parametrize("src,dst", [("int8", "int4"), ("e4m3", "e2m3")])
def test_slice_scale_other_block_sizes(src, dst, block):
    rng = np.random.default_rng(block)
    n = 128 * 301
    codes = rng.integers(0, 255, n).astype(np.uint8)
    codes[codes == 0x7F] = 0x7E
    scales = rng.integers(0, 256, n // block).astype(np.uint8)
    got_c, got_s = gpu_slice_scale(codes, scales, n, src, dst, block)
    want_c, want_s = orc.slice_scale(codes, scales, src, dst, block)
    assert bits_equal(got_s, want_s), first_diff(got_s, want_s)
    assert bits_equal(got_c, orc.pack(want_c, orc.bits(dst)))


def test_slice_scale_batched_matches_oracle():
    """Tensors of very different sizes (one smaller than a tile) in one launch."""
    rng = np.random.default_rng(9)
    sizes = [32, 32 * 7, 32 * 64, 32 * 65, 32 * 4097, 32 * 1000, 32, 32 * 333]
    for src, dst in (("int8", "int6"), ("int8", "int4"), ("e4m3", "e2m3"), ("e4m3", "e3m2"), ("e4m3", "e2m1")):
        items, wants = [], []
        for n in sizes:
            codes = rng.integers(0, 256, n).astype(np.uint8)
            codes[(codes & 0x7F) == 0x7F] &= 0xFE
            scales = rng.integers(0, 256, n // 32).astype(np.uint8)
            oc = torch.full((mxq.codes_bytes(n, dst) + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            os_ = torch.full((n // 32 + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            items.append((to_dev(codes), to_dev(scales), n, oc, os_))
            wants.append(orc.slice_scale(codes, scales, src, dst))
        mxq.slice_scale_batched(items, src, dst)
        mxq.slice_scale_batched(items, src, dst)      # the item table is reused
        torch.cuda.synchronize()
        for (c, s, n, oc, os_), (wc, ws) in zip(items, wants):
            nb = mxq.codes_bytes(n, dst)
            assert bits_equal(to_host(oc[:nb]), orc.pack(wc, orc.bits(dst)))
            assert bits_equal(to_host(os_[:n // 32]), ws)
            assert np.all(to_host(oc[nb:]) == 0xA5) and np.all(to_host(os_[n // 32:]) == 0xA5)


@pytest.mark.parametrize("count", [64, 65, 512, 513, 700])
def test_slice_scale_batched_item_counts(count):
    """Item counts on both sides of the limits where the item table changes its way to the kernel
    (small and large kernel-parameter blocks, more than one launch)."""
    rng = np.random.default_rng(count)
    sizes = (64 * rng.integers(1, 8, count)).tolist()          # 64-element multiples keep every pointer 32-byte aligned
    total = int(sum(sizes))
    codes = rng.integers(0, 256, total).astype(np.uint8)
    scales = rng.integers(0, 256, total // 32).astype(np.uint8)
    # one arena per stream, tensors at 32-byte aligned offsets inside it
    d_codes, d_scales = to_dev(codes), to_dev(np.repeat(scales, 16))        # 16-byte stride keeps scale pointers aligned
    d_out = torch.full((total // 2,), 0xA5, dtype=torch.uint8, device="cuda")
    d_os = torch.full((total // 32 * 16,), 0xA5, dtype=torch.uint8, device="cuda")
    items, off = [], 0
    host_scales = np.repeat(scales, 16)
    for n in sizes:
        b0 = off // 32
        items.append((d_codes[off:off + n], d_scales[b0 * 16:b0 * 16 + n // 32], n, d_out[off // 2:(off + n) // 2],
                      d_os[b0 * 16:b0 * 16 + n // 32]))
        off += n
    mxq.slice_scale_batched(items, "int8", "int4")
    torch.cuda.synchronize()
    got_c, got_s = to_host(d_out), to_host(d_os)
    off = 0
    for n in sizes:
        b0 = off // 32
        sc = host_scales[b0 * 16:b0 * 16 + n // 32]
        wc, ws = orc.slice_scale(codes[off:off + n], sc, "int8", "int4")
        assert bits_equal(got_c[off // 2:(off + n) // 2], orc.pack(wc, 4)), (count, off)
        assert bits_equal(got_s[b0 * 16:b0 * 16 + n // 32], ws), (count, off)
        assert np.all(got_s[b0 * 16 + n // 32:b0 * 16 + 16] == 0xA5) or n // 32 >= 16
        off += n


@pytest.mark.parametrize("src,dsts", [
    ("int8", ["int6", "int4"]), ("int8", ["int4", "int6"]), ("e4m3", ["e2m3", "e2m1"]), ("e4m3", ["e2m1", "e3m2"]),
    ("e4m3", ["e3m2", "e2m3"]), ("e4m3", ["e2m3", "e2m1", "e3m2"]), ("int8", ["int7", "int2"]), ("int8", ["int4"]),
    ("e4m3", ["e3m2", "e2m3", "e2m1", "e2m2", "e3m3"]), ("int6", ["int4", "int3"]),
], ids=lambda v: v if isinstance(v, str) else "+".join(v))
@pytest.mark.parametrize("block", [32, 16, 128])
def test_slice_scale_multi_equals_single_target_conversions(src, dsts, block):
    """One read of the anchor, several targets: fused pairs in both orders, lists that mix fused and
    single passes, and pairs that have no fused kernel."""
    codes, scales32 = _all_codes_input(src, nblk_extra=301 * 4 - 256)
    n = codes.size - codes.size % 128
    codes = codes[:n]
    scales = np.resize(scales32, n // block)
    packed = orc.pack(codes, orc.bits(src))
    guards = [(Guarded(mxq.codes_bytes(n, d)), Guarded(n // block)) for d in dsts]
    mxq.slice_scale_multi(to_dev(packed), to_dev(scales), n, src, dsts, block, [(c.view, s.view) for c, s in guards])
    torch.cuda.synchronize()
    for d, (gc, gs) in zip(dsts, guards):
        gc.check()
        gs.check()
        wc, ws = orc.slice_scale(codes, scales, src, d, block)
        assert bits_equal(to_host(gs.view), ws), (d, first_diff(to_host(gs.view), ws))
        assert bits_equal(to_host(gc.view), orc.pack(wc, orc.bits(d))), d


# ---------------------------------------------------------------------------------------------
# Reconstruction
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("fmt", ALL_FORMATS)
@pytest.mark.parametrize("bf16", [False, True])
def test_dequantize_all_codes_all_scales(fmt, bf16):
    """Every code under every scale byte (subnormal results, overflow to infinity, 0xFF -> NaN)."""
    nb = orc.bits(fmt)
    allc = np.resize(np.arange(1 << nb, dtype=np.uint8), 256)
    codes = np.tile(allc, 256 * 2)                       # 8 blocks of 32 per sweep, two sweeps per scale byte
    n = codes.size
    scales = np.repeat(np.arange(256, dtype=np.uint8), n // 32 // 256)
    got = gpu_dequantize(orc.pack(codes, nb), scales, n, fmt, bf16=bf16)
    want = orc.dequantize(codes, scales, fmt, out_dtype=orc.BF16 if bf16 else orc.F32)
    assert bits_equal(got, want), first_diff(got, want)


@pytest.mark.parametrize("block", [16, 64, 128])
@pytest.mark.parametrize("fmt", ["int4", "e2m3", "e4m3"])
def test_dequantize_other_block_sizes(fmt, block):
    rng = np.random.default_rng(block + 1)
    n = 128 * 257
    codes = rng.integers(0, 1 << orc.bits(fmt), n).astype(np.uint8)
    scales = rng.integers(100, 160, n // block).astype(np.uint8)
    for bf16 in (False, True):
        got = gpu_dequantize(orc.pack(codes, orc.bits(fmt)), scales, n, fmt, block, bf16=bf16)
        want = orc.dequantize(codes, scales, fmt, block, orc.BF16 if bf16 else orc.F32)
        assert bits_equal(got, want), first_diff(got, want)


# ---------------------------------------------------------------------------------------------
# Fake-quant
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("fmt", ALL_FORMATS)
@pytest.mark.parametrize("mode", [orc.FQ_DIRECT, orc.FQ_VIA_ANCHOR])
@pytest.mark.parametrize("bf16", [False, True])
def test_fake_quant(fmt, mode, bf16):
    x = np.concatenate([_mixed_f32(NBLK, 5), inputs.adversarial_f32()])
    if bf16:
        x = inputs.to_bf16_bits(x)
    got = gpu_fake_quant(x, fmt, mode=mode)
    want = orc.fake_quant(x, fmt, mode=mode)
    assert bits_equal(got, want), first_diff(got, want)


@pytest.mark.parametrize("fmt", ["int6", "e2m3"])
def test_fake_quant_every_bf16_pattern(fmt):
    pats = np.arange(65536, dtype=np.uint16)
    blocks = []
    for k in (-126, -9, 0, 100):
        pin = inputs.to_bf16_bits(np.array([1.75 * 2.0 ** k], np.float32))[0]
        body = np.concatenate([pats, np.zeros((-65536) % 31, np.uint16)]).reshape(-1, 31)
        blocks.append(np.concatenate([np.full((body.shape[0], 1), pin, np.uint16), body], axis=1).reshape(-1))
    x = np.concatenate(blocks)
    for mode in (orc.FQ_DIRECT, orc.FQ_VIA_ANCHOR):
        got = gpu_fake_quant(x, fmt, mode=mode)
        want = orc.fake_quant(x, fmt, mode=mode)
        assert bits_equal(got, want), first_diff(got, want)


@pytest.mark.parametrize("block", [16, 64, 128])
def test_fake_quant_other_block_sizes(block):
    x = inputs.to_bf16_bits(_mixed_f32(501, 6, block))
    for fmt in ("int4", "e2m1"):
        for mode in (orc.FQ_DIRECT, orc.FQ_VIA_ANCHOR):
            got = gpu_fake_quant(x, fmt, block, mode)
            want = orc.fake_quant(x, fmt, block, mode)
            assert bits_equal(got, want), first_diff(got, want)


def test_fake_quant_in_place_and_backward():
    x = inputs.to_bf16_bits(_mixed_f32(513, 7))
    want = orc.fake_quant(x, "int4", mode=orc.FQ_VIA_ANCHOR)
    got = gpu_fake_quant(x, "int4", mode=orc.FQ_VIA_ANCHOR, inplace=True)
    assert bits_equal(got, want)
    # straight-through estimator: the gradient comes back unchanged, for any length
    for n in (1, 31, 4096, 4096 * 5 + 3):
        g = to_dev(inputs.to_bf16_bits(np.random.default_rng(n).standard_normal(n).astype(np.float32)))
        gi = mxq.fake_quant_bwd(g)
        torch.cuda.synchronize()
        assert torch.equal(gi.view(torch.int16), g.view(torch.int16))
        assert mxq.fake_quant_bwd(g, g) is g
    g32 = torch.randn(1000, device="cuda")
    assert torch.equal(mxq.fake_quant_bwd(g32), g32)


@pytest.mark.parametrize("copy_grad", [False, True])
def test_fake_quant_inside_autograd_is_straight_through(copy_grad):
    """Eq. 6 as a differentiable function: value = the oracle's fake-quant, dL/dW = dL/dW_t bit for bit."""
    w_bits = inputs.to_bf16_bits(_mixed_f32(257, 11))
    w = to_dev(w_bits).view(257, 32).requires_grad_(True)
    wt = mxq.fake_quant_ste(w, "e2m1", 32, mxq.FQ_VIA_ANCHOR, copy_grad=copy_grad)
    assert bits_equal(to_host(wt.detach().reshape(-1)), orc.fake_quant(w_bits, "e2m1", mode=orc.FQ_VIA_ANCHOR))
    up = to_dev(inputs.to_bf16_bits(np.random.default_rng(3).standard_normal(w_bits.size).astype(np.float32))).view(257, 32)
    wt.backward(up)
    torch.cuda.synchronize()
    assert torch.equal(w.grad.view(torch.int16), up.view(torch.int16))
    assert (w.grad.data_ptr() != up.data_ptr()) or not copy_grad


@pytest.mark.parametrize("count", [1, 7, 512, 513, 1100])
@pytest.mark.parametrize("bf16", [True, False])
def test_fake_quant_batched_matches_oracle(count, bf16):
    """Many tensors of different sizes (down to one block) in one call, some of them in place; counts on
    both sides of the 512-tensor launch limit."""
    rng = np.random.default_rng(count)
    nblks = rng.integers(1, 40, count)
    if count <= 7:
        nblks[0] = 3000                                          # one tensor of many tiles
    fmt, mode = ("e2m3", orc.FQ_VIA_ANCHOR) if bf16 else ("int4", orc.FQ_DIRECT)
    pairs, wants = [], []
    for k, nb in enumerate(nblks):
        x = _mixed_f32(int(nb), 1000 + k)
        if bf16:
            x = inputs.to_bf16_bits(x)
        src = to_dev(x)
        dst = None if k % 3 == 0 else torch.full_like(src, 7.0)
        pairs.append((src, dst))
        wants.append(orc.fake_quant(x, fmt, mode=mode))
    mxq.fake_quant_batched(pairs, fmt, 32, mode)
    torch.cuda.synchronize()
    for (src, dst), want in zip(pairs, wants):
        got = to_host(dst if dst is not None else src)
        assert bits_equal(got, want), first_diff(got, want)


@pytest.mark.parametrize("count", [1, 5, 256, 257, 600])
@pytest.mark.parametrize("src,dst1,dst2,block", [("int8", "int6", "int4", 32), ("e4m3", "e2m1", "e2m3", 32),
                                                  ("e4m3", "e3m2", "e2m1", 64), ("e4m3", "e2m3", "e3m2", 128),
                                                  ("int8", "int7", "int3", 32), ("e4m3", "e3m3", "e2m2", 32)])
def test_slice_scale_pair_batched_matches_oracle(count, src, dst1, dst2, block):
    """Two targets from one read of every anchor of a set of tensors: fused pairs (both orders of the
    targets) and pairs that fall back to two passes; counts on both sides of the 256-tensor launch limit;
    all byte values as codes and as scale bytes."""
    rng = np.random.default_rng(count * 7 + block)
    nblks = rng.integers(1, 30, count) * (block // 32)
    if count <= 5:
        nblks[0] = 2051 * (block // 32)
    ins, outs = [], []
    for nb in nblks:
        n = int(nb) * 32
        codes = rng.integers(0, 256, n).astype(np.uint8)
        scales = rng.integers(0, 256, n // block).astype(np.uint8)
        o = [Guarded(mxq.codes_bytes(n, dst1)), Guarded(n // block), Guarded(mxq.codes_bytes(n, dst2)), Guarded(n // block)]
        ins.append((codes, scales, n))
        outs.append(o)
    items = [(to_dev(c), to_dev(s), n, o[0].view, o[1].view, o[2].view, o[3].view) for (c, s, n), o in zip(ins, outs)]
    mxq.slice_scale_pair_batched(items, src, dst1, dst2, block)
    torch.cuda.synchronize()
    for k, ((c, s, n), o) in enumerate(zip(ins, outs)):
        for g in o:
            g.check()
        for dst, oc, os_ in ((dst1, o[0], o[1]), (dst2, o[2], o[3])):
            wc, ws = orc.slice_scale(c, s, src, dst, block)
            assert bits_equal(to_host(os_.view), ws), (k, dst)
            assert bits_equal(to_host(oc.view), orc.pack(wc, orc.bits(dst))), (k, dst, first_diff(to_host(oc.view), orc.pack(wc, orc.bits(dst))))


@pytest.mark.parametrize("count", [1, 6, 512, 513, 1030])
@pytest.mark.parametrize("fmt,bf16,block", [("int8", True, 32), ("e4m3", False, 32), ("int6", True, 64), ("e2m1", False, 16),
                                             ("int7", True, 32), ("e3m3", True, 128)])
def test_quantize_and_dequantize_batched_match_oracle(count, fmt, bf16, block):
    """Whole sets of tensors of different sizes (down to one block) in one call each: Q_f into codes and
    scales, then the reconstruction of those, both against the oracle per tensor; counts on both sides
    of the 512-tensor launch limit; guard zones around every output."""
    rng = np.random.default_rng(count * 131 + block)
    per = 128 // block if block < 32 else 1                    # keep n a multiple of 32 for the packed readers
    nblks = rng.integers(1, 24, count) * max(1, 32 // block) * per
    if count <= 6:
        nblks[0] = 2051 * max(1, 32 // block)                  # one tensor of many tiles and a ragged tail
    xs, triples, items, keep = [], [], [], []
    for k, nb in enumerate(nblks):
        x = _mixed_f32(int(nb), 2000 + k, block)
        if bf16:
            x = inputs.to_bf16_bits(x)
        n = x.size
        c, s = Guarded(mxq.codes_bytes(n, fmt)), Guarded(n // block)
        y = Guarded(n * (2 if k % 2 else 4), torch.bfloat16 if k % 2 else torch.float32)
        xs.append(x)
        triples.append((to_dev(x), c.view, s.view))
        keep.append((c, s, y))
    mxq.quantize_batched(triples, fmt, block)
    # reconstruction: the even tensors to FP32 in one call, the odd ones to BF16 in another
    for parity in (0, 1):
        sel = [(keep[k][0].view, keep[k][1].view, xs[k].size, keep[k][2].view) for k in range(count) if k % 2 == parity]
        if sel:
            mxq.dequantize_batched(sel, fmt, block)
    torch.cuda.synchronize()
    for k, x in enumerate(xs):
        c, s, y = keep[k]
        for g in (c, s, y):
            g.check()
        wc, ws = orc.quantize(x, fmt, block)
        assert bits_equal(to_host(s.view), ws), (k, first_diff(to_host(s.view), ws))
        assert bits_equal(to_host(c.view), orc.pack(wc, orc.bits(fmt))), k
        want = orc.dequantize(wc, ws, fmt, block, orc.BF16 if k % 2 else orc.F32)
        assert bits_equal(to_host(y.view), want), (k, first_diff(to_host(y.view), want))


# ---------------------------------------------------------------------------------------------
# chained entry points and degenerate sizes
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("fmt", MAIN_FORMATS)
def test_quantize_then_dequantize_equals_fake_quant(fmt):
    """The fused kernel and the two-kernel route agree with each other as well as with the oracle."""
    x = inputs.to_bf16_bits(_mixed_f32(300, 8))
    n = x.size
    c, s = gpu_quantize(x, fmt)
    v = gpu_dequantize(c, s, n, fmt, bf16=True)
    assert bits_equal(v, gpu_fake_quant(x, fmt))


@pytest.mark.parametrize("world", [2, 3, 8])
def test_sharded_conversion_stitches_to_the_unsharded_one(world):
    """The multi-GPU path: every rank converts its own run of whole blocks into its own byte range of
    the full outputs, with no exchange.  The ranks run here one after another on one GPU (independent
    launches that do not wait on one another); the stitched result must be the oracle's whole-tensor
    result, byte for byte, and nothing outside a rank's range may be touched by it."""
    from paper_2604_00529_b200.shard import block_range, quantize_shard, slice_scale_shard
    nblk = 5003                                          # 157 chunks of 32 blocks: a ragged split for every world size
    x = _mixed_f32(nblk, seed=77)
    n = x.size
    xd = to_dev(x)
    codes, scales = Guarded(n), Guarded(n // 32)
    lc, ls = Guarded(n // 2), Guarded(n // 32)
    covered = 0
    for rank in range(world):
        lo, hi = quantize_shard(xd, "int8", 32, codes.view, scales.view, rank, world)
        assert (lo, hi) == block_range(n, 32, rank, world) and lo == covered
        covered = hi
        torch.cuda.synchronize()
        got = to_host(codes.view)
        assert np.all(got[hi:] == 0xA5), "rank %d wrote beyond its range" % rank
    assert covered == n
    for rank in reversed(range(world)):                  # any order: the shards are independent
        slice_scale_shard(codes.view, scales.view, n, "int8", "int4", 32, lc.view, ls.view, rank, world)
    torch.cuda.synchronize()
    for g in (codes, scales, lc, ls):
        g.check()
    wc, ws = orc.quantize(x, "int8")
    assert bits_equal(to_host(codes.view), orc.pack(wc, 8)) and bits_equal(to_host(scales.view), ws)
    w4, s4 = orc.slice_scale(wc, ws, "int8", "int4")
    assert bits_equal(to_host(lc.view), orc.pack(w4, 4)), first_diff(to_host(lc.view), orc.pack(w4, 4))
    assert bits_equal(to_host(ls.view), s4)


def test_prepared_calls_give_the_same_bytes():
    """The pre-marshalled call objects of the binding enqueue the same operations as the plain functions."""
    x = _mixed_f32(700, seed=5)
    n = x.size
    xd = to_dev(x)
    c, s = Guarded(n), Guarded(n // 32)
    lc, ls = Guarded(n * 6 // 8), Guarded(n // 32)
    y, f, g = Guarded(4 * n, torch.float32), Guarded(4 * n, torch.float32), Guarded(4 * n, torch.float32)
    calls = [mxq.prepare_quantize(xd, "e4m3", 32, c.view, s.view),
             mxq.prepare_slice_scale(c.view, s.view, n, "e4m3", "e2m3", 32, lc.view, ls.view),
             mxq.prepare_dequantize(lc.view, ls.view, n, "e2m3", 32, y.view),
             mxq.prepare_fake_quant(xd, "e2m3", 32, mxq.FQ_VIA_ANCHOR, f.view),
             mxq.prepare_fake_quant_bwd(f.view, g.view)]
    for _ in range(2):                                   # a prepared call may be used any number of times
        for call in calls:
            call()
    torch.cuda.synchronize()
    for buf in (c, s, lc, ls, y, f, g):
        buf.check()
    wc, ws = orc.quantize(x, "e4m3")
    w6, s6 = orc.slice_scale(wc, ws, "e4m3", "e2m3")
    assert bits_equal(to_host(c.view), orc.pack(wc, 8)) and bits_equal(to_host(s.view), ws)
    assert bits_equal(to_host(lc.view), orc.pack(w6, 6)) and bits_equal(to_host(ls.view), s6)
    want = orc.dequantize(w6, s6, "e2m3")
    assert bits_equal(to_host(y.view), want) and bits_equal(to_host(f.view), want) and bits_equal(to_host(g.view), want)


def test_smallest_and_empty_inputs():
    x = np.array([1.0] + [0.25] * 31, np.float32)
    c, s = gpu_quantize(x, "int8")
    wc, ws = _oracle_packed(x, "int8")
    assert bits_equal(c, wc) and bits_equal(s, ws)
    empty = torch.empty(0, dtype=torch.float32, device="cuda")
    c, s = mxq.quantize(empty, "int8")
    assert c.numel() == 0 and s.numel() == 0
    assert mxq.fake_quant(empty, "e2m1").numel() == 0


# ---------------------------------------------------------------------------------------------
# The tensor-level study of Sec. 4.3 / App. C through the CUDA path
# ---------------------------------------------------------------------------------------------

def test_tensor_level_mse_study_on_gpu():
    """100 random tensors of shape (1, 1024): Slice-and-Scale against direct quantization over bit-widths
    at block 64 and over block sizes at 4 bits.  The GPU's reconstruction errors must equal the
    oracle's (the outputs are bit-identical) and show what the paper reports: SS tracks direct
    quantization closely, the gap being largest for MXFP at intermediate widths."""
    rng = np.random.default_rng(100)
    x = rng.standard_normal(100 * 1024).astype(np.float32)

    def mse(y):
        return float(np.mean((y.astype(np.float64) - x) ** 2))

    table = {}
    for fmt in ("int2", "int3", "int4", "int5", "int6", "int7", "int8", "e2m1", "e2m2", "e3m2", "e2m3", "e3m3", "e4m3"):
        for mode in (orc.FQ_DIRECT, orc.FQ_VIA_ANCHOR):
            got = gpu_fake_quant(x, fmt, 64, mode)
            want = orc.fake_quant(x, fmt, 64, mode)
            assert bits_equal(got, want), (fmt, mode, first_diff(got, want))
            table[(fmt, mode)] = mse(got)
    for fmt in ("int2", "int3", "int4", "int5", "int6", "int7", "e2m1", "e2m2", "e3m2", "e3m3"):
        r = table[(fmt, orc.FQ_VIA_ANCHOR)] / table[(fmt, orc.FQ_DIRECT)]
        assert 1.0 <= r < 2.0, (fmt, r)
    gap = {f: table[(f, orc.FQ_VIA_ANCHOR)] / table[(f, orc.FQ_DIRECT)] for f in ("e2m1", "e2m2", "e3m2", "e3m3")}
    assert min(gap["e2m2"], gap["e3m2"]) > max(gap["e2m1"], gap["e3m3"])
    for f in ("int8", "e4m3"):                                    # the anchor itself: both routes coincide
        assert table[(f, orc.FQ_VIA_ANCHOR)] == table[(f, orc.FQ_DIRECT)]
    by_block = []
    for block in (16, 32, 64, 128):
        d = gpu_fake_quant(x, "int4", block, orc.FQ_DIRECT)
        s = gpu_fake_quant(x, "int4", block, orc.FQ_VIA_ANCHOR)
        assert bits_equal(d, orc.fake_quant(x, "int4", block, orc.FQ_DIRECT))
        assert bits_equal(s, orc.fake_quant(x, "int4", block, orc.FQ_VIA_ANCHOR))
        by_block.append((mse(d), mse(s)))
    assert all(a[0] < b[0] and a[1] < b[1] for a, b in zip(by_block[:-1], by_block[1:]))   # smaller blocks, lower error
    assert all(1.0 <= s / d < 1.2 for d, s in by_block)


def test_two_streams_run_independent_conversions():
    """The same calls issued on two non-default streams at once give what they give alone (every
    entry point takes its stream from the caller; only the fixed-table batched entry point shares state)."""
    x1 = inputs.to_bf16_bits(_mixed_f32(4099, 21))
    x2 = inputs.to_bf16_bits(_mixed_f32(4099, 22))
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    d1, d2 = to_dev(x1), to_dev(x2)
    torch.cuda.synchronize()
    res = {}
    for rep in range(3):
        for name, st, d, fmt, low in (("a", s1, d1, "e4m3", "e2m1"), ("b", s2, d2, "int8", "int6")):
            with torch.cuda.stream(st):
                c, s = mxq.quantize(d, fmt)
                lc, ls = mxq.slice_scale(c, s, d.numel(), fmt, low)
                v = mxq.dequantize(lc, ls, d.numel(), low, dtype=torch.bfloat16)
                y = mxq.fake_quant(d, low, mode=mxq.FQ_VIA_ANCHOR)
                res[name] = (lc, ls, v, y)
    torch.cuda.synchronize()
    for name, x, fmt, low in (("a", x1, "e4m3", "e2m1"), ("b", x2, "int8", "int6")):
        lc, ls, v, y = res[name]
        oc, os_ = orc.quantize(x, fmt)
        wc, ws = orc.slice_scale(oc, os_, fmt, low)
        assert bits_equal(to_host(lc), orc.pack(wc, orc.bits(low))) and bits_equal(to_host(ls), ws)
        assert bits_equal(to_host(v), orc.dequantize(wc, ws, low, out_dtype=orc.BF16))
        assert bits_equal(to_host(y), orc.fake_quant(x, low, mode=orc.FQ_VIA_ANCHOR))


@pytest.mark.parametrize("nblk", [4096, 1 << 16, 1 << 19])
@pytest.mark.parametrize("anchor,low", [("e4m3", "e2m1"), ("e4m3", "e2m3"), ("int8", "int6"), ("int8", "int7")])
def test_dependent_chain_reusing_buffers_reads_fresh_data(nblk, anchor, low):
    """quantize -> slice_scale -> dequantize -> fake-quant in place, eight rounds back to back on ONE
    stream, every round with new input but the SAME intermediate buffers and no host synchronisation in
    between.  Each kernel starts while its producer is still running (programmatic dependent launch) and
    prefetches its input lines before it waits for the producer; what it then reads must be what the
    producer wrote in this round, not the previous round's bytes.  Sizes: less than one wave of CTAs, a
    few waves, many waves.  The 6- and 7-bit targets leave their kernel as bulk copies out of shared memory: the
    consumer must see those bytes too."""
    n = nblk * 32
    rounds = 8
    base = inputs.to_bf16_bits(_mixed_f32(nblk + rounds, 77))
    xs_host = [np.ascontiguousarray(base[32 * r:32 * r + n]) for r in range(rounds)]
    xs = [to_dev(x) for x in xs_host]
    codes = torch.empty(n, dtype=torch.uint8, device="cuda")
    scales = torch.empty(nblk, dtype=torch.uint8, device="cuda")
    bl = orc.bits(low)
    low_c = torch.empty(n * bl // 8, dtype=torch.uint8, device="cuda")
    low_s = torch.empty(nblk, dtype=torch.uint8, device="cuda")
    v = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    kept = []
    torch.cuda.synchronize()
    for r in range(rounds):
        mxq.quantize(xs[r], anchor, 32, codes, scales)
        mxq.slice_scale(codes, scales, n, anchor, low, 32, low_c, low_s)
        mxq.dequantize(low_c, low_s, n, low, 32, dst=v)
        mxq.fake_quant(v, "e2m3", 32, mxq.FQ_DIRECT, dst=v)                # in place, on what was just written
        kept.append((mxq.fake_quant_bwd(low_c.view(torch.bfloat16)), mxq.fake_quant_bwd(v)))   # stream-ordered copies
    torch.cuda.synchronize()
    for r in (0, 3, rounds - 1) if nblk > 4096 else range(rounds):
        oc, os_ = orc.quantize(xs_host[r], anchor)
        wc, ws = orc.slice_scale(oc, os_, anchor, low)
        want_v = orc.dequantize(wc, ws, low, out_dtype=orc.BF16)
        got_c, got_v = kept[r]
        assert bits_equal(to_host(got_c.view(torch.uint8)), orc.pack(wc, bl)), (r, "codes")
        assert bits_equal(to_host(got_v), orc.fake_quant(want_v, "e2m3", mode=orc.FQ_DIRECT)), (r, "values")


def test_randomized_cross_check_of_every_entry_point():
    """Seeded random cases: block size, source type, length, magnitudes (zeros, outliers, a NaN or an
    infinity now and then), tensors placed at 32-byte-aligned offsets inside larger buffers, a random
    anchor-to-lower pair and a chained pair; every result against the oracle, bit for bit."""
    rng = np.random.default_rng(20260411)
    ints = ["int8", "int7", "int6", "int5", "int4", "int3", "int2"]
    fps = ["e4m3", "e3m3", "e3m2", "e2m3", "e2m2", "e2m1"]

    def place(x, pad):
        if x.dtype == np.uint16:
            buf = torch.zeros(x.size + 16 * pad + 64, dtype=torch.int16, device="cuda")
            v = buf[16 * pad:16 * pad + x.size]
            v.copy_(torch.from_numpy(x.view(np.int16)))
            return v.view(torch.bfloat16)
        buf = torch.zeros(x.size + 8 * pad + 64, dtype=torch.float32, device="cuda")
        v = buf[8 * pad:8 * pad + x.size]
        v.copy_(torch.from_numpy(x))
        return v

    for case in range(150):
        block = int(rng.choice([16, 32, 32, 32, 64, 128]))
        bf16 = bool(rng.random() < 0.6)
        nblk = int(rng.choice([1, 2, 3, 5, 31, 33, 64, 127, 129, 257, 1000, 4097]))
        if block == 16 and nblk % 2:
            nblk += 1
        x = rng.standard_normal((nblk, block)) * 2.0 ** rng.integers(-40, 40, (nblk, 1))
        x[rng.random((nblk, block)) < 0.03] *= 64
        x[rng.random((nblk, block)) < 0.05] = 0
        x = x.astype(np.float32).reshape(-1)
        if rng.random() < 0.15:
            x[rng.integers(0, x.size)] = np.float32(rng.choice([np.inf, -np.inf, np.nan]))
        if bf16:
            x = inputs.to_bf16_bits(x)
        n = x.size
        xd = place(x, int(rng.integers(0, 4)))
        fam = ints if rng.random() < 0.5 else fps
        a, f = fam[0], str(rng.choice(fam))
        what = (case, block, bf16, nblk, a, f)
        ca, sa = mxq.quantize(xd, a, block)
        oa, osa = orc.quantize(x, a, block)
        assert bits_equal(to_host(ca), orc.pack(oa, 8)) and bits_equal(to_host(sa), osa), what
        cf, sf = mxq.quantize(xd, f, block)
        of, osf = orc.quantize(x, f, block)
        assert bits_equal(to_host(cf), orc.pack(of, orc.bits(f))) and bits_equal(to_host(sf), osf), what
        lc, ls = mxq.slice_scale(ca, sa, n, a, f, block)
        wc, ws = orc.slice_scale(oa, osa, a, f, block)
        assert bits_equal(to_host(lc), orc.pack(wc, orc.bits(f))) and bits_equal(to_host(ls), ws), what
        g = str(rng.choice([h for h in fam[fam.index(f):] if orc.bits(h) <= orc.bits(f)]))
        try:
            w2, ws2 = orc.slice_scale(wc, ws, f, g, block)
        except ValueError:
            w2 = None                                          # not a legal pair (the exponent range would grow)
        if w2 is not None:
            cc, cs = mxq.slice_scale(lc, ls, n, f, g, block)
            assert bits_equal(to_host(cc), orc.pack(w2, orc.bits(g))) and bits_equal(to_host(cs), ws2), what + (g,)
        for dt, od in ((torch.float32, orc.F32), (torch.bfloat16, orc.BF16)):
            v = mxq.dequantize(lc, ls, n, f, block, dtype=dt)
            assert bits_equal(to_host(v), orc.dequantize(wc, ws, f, block, od)), what + (dt,)
        for mode in (orc.FQ_DIRECT, orc.FQ_VIA_ANCHOR):
            y = mxq.fake_quant(xd, f, block, mode)
            assert bits_equal(to_host(y), orc.fake_quant(x, f, block, mode)), what + (mode,)
