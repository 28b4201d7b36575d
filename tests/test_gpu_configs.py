"""The five workloads at their full sizes, in the launch configuration the bench times, against the
CPU oracle.  Where the oracle finishes the whole tensor in seconds the comparison is element by
element over everything; otherwise it runs over sampled runs of blocks (every MX block is converted
on its own, so the oracle's output for a run of blocks is exactly the slice of the full result) --
the first and the last blocks always among them.  Tolerance: zero (bytes and bit patterns)."""
import numpy as np
import pytest
import torch

import paper_2604_00529_b200 as mxq
from oracle import mxq_oracle as orc
from paper_2604_00529_b200 import inputs

from gpu_util import bits_equal, first_diff, to_dev, to_host

pytestmark = pytest.mark.gpu
BLOCK = 32


def sample_runs(nblk: int, runs: int, run_blocks: int, seed: int):
    """Sorted, disjoint [lo, hi) block ranges: the first and last `run_blocks` blocks plus random runs."""
    run_blocks = min(run_blocks, nblk)
    if nblk <= runs * run_blocks:
        return [(0, nblk)]
    rng = np.random.default_rng(seed)
    starts = {0, nblk - run_blocks}
    slots = nblk // run_blocks
    for s in rng.choice(slots, size=min(runs, slots), replace=False):
        starts.add(int(s) * run_blocks)
    return [(s, s + run_blocks) for s in sorted(starts)]


def dev_slice(t: torch.Tensor, lo: int, hi: int) -> np.ndarray:
    return to_host(t[lo:hi])


def check_quantize(x_host, x_dev, fmt, runs, what):
    """GPU quantize of the whole tensor; compare the sampled block runs.  Returns device (codes, scales)."""
    n = x_dev.numel()
    codes, scales = mxq.quantize(x_dev, fmt, BLOCK)
    b = orc.bits(fmt)
    for lo, hi in runs:
        wc, ws = orc.quantize(x_host(lo * BLOCK, hi * BLOCK), fmt, BLOCK)
        got_s = dev_slice(scales, lo, hi)
        got_c = dev_slice(codes, lo * BLOCK * b // 8, hi * BLOCK * b // 8)
        assert bits_equal(got_s, ws), (what, fmt, lo, first_diff(got_s, ws))
        assert bits_equal(got_c, orc.pack(wc, b)), (what, fmt, lo, first_diff(got_c, orc.pack(wc, b)))
    assert codes.numel() == n * b // 8
    return codes, scales


def check_slice_scale(codes, scales, n, src, dst, runs, what, out=None):
    """GPU Slice-and-Scale of the whole tensor (or a given result); oracle on the anchor's sampled runs."""
    oc, os_ = out if out is not None else mxq.slice_scale(codes, scales, n, src, dst, BLOCK)
    bs, bd = orc.bits(src), orc.bits(dst)
    for lo, hi in runs:
        a_c = orc.unpack(dev_slice(codes, lo * BLOCK * bs // 8, hi * BLOCK * bs // 8), (hi - lo) * BLOCK, bs)
        a_s = dev_slice(scales, lo, hi)
        wc, ws = orc.slice_scale(a_c, a_s, src, dst, BLOCK)
        got_s = dev_slice(os_, lo, hi)
        got_c = dev_slice(oc, lo * BLOCK * bd // 8, hi * BLOCK * bd // 8)
        assert bits_equal(got_s, ws), (what, src, dst, lo, first_diff(got_s, ws))
        assert bits_equal(got_c, orc.pack(wc, bd)), (what, src, dst, lo, first_diff(got_c, orc.pack(wc, bd)))
    return oc, os_


def check_dequantize(codes, scales, n, fmt, dtype, runs, what):
    v = mxq.dequantize(codes, scales, n, fmt, BLOCK, dtype=dtype)
    b = orc.bits(fmt)
    for lo, hi in runs:
        c = orc.unpack(dev_slice(codes, lo * BLOCK * b // 8, hi * BLOCK * b // 8), (hi - lo) * BLOCK, b)
        want = orc.dequantize(c, dev_slice(scales, lo, hi), fmt, BLOCK, orc.BF16 if dtype == torch.bfloat16 else orc.F32)
        got = dev_slice(v, lo * BLOCK, hi * BLOCK)
        assert bits_equal(got, want), (what, fmt, lo, first_diff(got, want))
    return v


# ---------------------------------------------------------------------------------------------
# workload 1: FP32 4096 x 4096 N(0, 0.02), seed 0 -> MXINT8 -> MXINT4 -> reconstruction.  Everything compared.
# ---------------------------------------------------------------------------------------------

def test_workload1_fp32_weight_int8_int4_dequantize():
    x = inputs.weight_f32_normal(4096, 4096, seed=0)
    n = x.size
    runs = [(0, n // BLOCK)]
    xd = to_dev(x)
    codes, scales = check_quantize(lambda lo, hi: x[lo:hi], xd, "int8", runs, "w1")
    lc, ls = check_slice_scale(codes, scales, n, "int8", "int4", runs, "w1")
    check_dequantize(lc, ls, n, "int4", torch.float32, runs, "w1")
    check_dequantize(codes, scales, n, "int8", torch.float32, sample_runs(n // BLOCK, 8, 4096, 1), "w1")


# ---------------------------------------------------------------------------------------------
# workload 2: BF16 8192 x 8192 Student-t with outliers -> MXFP8 E4M3 -> MXFP6 E2M3, MXFP4 E2M1 (and E3M2)
# ---------------------------------------------------------------------------------------------

def test_workload2_bf16_student_t_e4m3_to_fp6_fp4():
    x = inputs.weight_bf16_student_t(8192, 8192, seed=1)
    n = x.size
    runs = [(0, n // BLOCK)]                                   # the whole tensor: ~10 s of oracle time
    xd = to_dev(x)
    codes, scales = check_quantize(lambda lo, hi: x[lo:hi], xd, "e4m3", runs, "w2")
    check_slice_scale(codes, scales, n, "e4m3", "e2m3", runs, "w2")
    lc, ls = check_slice_scale(codes, scales, n, "e4m3", "e2m1", runs, "w2")
    some = sample_runs(n // BLOCK, 32, 4096, 2)
    check_slice_scale(codes, scales, n, "e4m3", "e3m2", some, "w2")
    check_dequantize(lc, ls, n, "e2m1", torch.bfloat16, some, "w2")


# ---------------------------------------------------------------------------------------------
# workload 3: the 224 linear weights of an 8B Llama-shaped model, converted by ONE batched launch per
# target.  Four layers are drawn on the host (seeds 1000 layer + idx) and quantized on the GPU; the
# other layers' anchors are device copies of those four (Slice-and-Scale is a function of the anchor
# codes alone, and what is checked is the anchor -> target conversion of every one of the 224 items).
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("anchor,targets", [("int8", ("int6", "int4")), ("e4m3", ("e2m3", "e2m1"))])
def test_workload3_whole_model_batched_conversion(anchor, targets):
    drawn = (0, 13, 31, 7)                               # four of the 32 layers are fresh bits
    base = {}
    for li, layer in enumerate(drawn):
        for idx, (name, r, c) in enumerate(inputs.LLAMA8B_LAYER):
            x = inputs.llama8b_tensor(layer, idx)
            xd = to_dev(x)
            nblk = x.size // BLOCK
            base[(li, idx)] = check_quantize(lambda lo, hi, x=x: x[lo:hi], xd, anchor,
                                             sample_runs(nblk, 4, 2048, 100 * layer + idx), "w3 %s" % name)
            del xd
    shapes = inputs.llama8b_shapes()
    assert len(shapes) == 224 and sum(r * c for _, _, _, r, c in shapes) == 6979321856
    anchors = []
    for layer, idx, name, r, c in shapes:
        src_c, src_s = base[(layer % len(drawn), idx)]
        if layer < len(drawn):
            anchors.append((src_c, src_s, r * c))
        else:
            anchors.append((src_c.clone(), src_s.clone(), r * c))
    for dst in targets:
        b = orc.bits(dst)
        outs = [(torch.empty(n * b // 8, dtype=torch.uint8, device="cuda"),
                 torch.empty(n // BLOCK, dtype=torch.uint8, device="cuda")) for _, _, n in anchors]
        table = mxq.make_items([(c, s, n, oc, os_) for (c, s, n), (oc, os_) in zip(anchors, outs)])
        mxq.slice_scale_batched(table, anchor, dst, BLOCK)
        torch.cuda.synchronize()
        for k, ((c, s, n), out) in enumerate(zip(anchors, outs)):
            check_slice_scale(c, s, n, anchor, dst, sample_runs(n // BLOCK, 2, 1024, k), "w3 item %d" % k, out=out)
        del outs, table


def test_workload3_headline_step_in_the_launch_configuration_of_the_bench():
    """The ten launches of the bench's headline step, each over all 224 tensors of the weight set laid
    out in one arena per stream as the bench lays them out: quantize_batched to both anchors,
    slice_scale_batched to the 4-bit targets, dequantize_batched, fake_quant_batched (E2M3 through the
    anchor) and the straight-through copy of the whole arena.  Four layers are drawn on the host, the
    others are device copies of them in turn; every tensor is checked on sampled block runs (first and
    last blocks among them) against the oracle run on the host bits of the same elements."""
    drawn = (0, 13, 31, 7)
    shapes = inputs.llama8b_shapes()
    sizes = [r * c for *_, r, c in shapes]
    total = sum(sizes)
    layer_elems = sum(r * c for _, r, c in inputs.LLAMA8B_LAYER)
    host = [np.concatenate([inputs.llama8b_tensor(layer, idx) for idx in range(len(inputs.LLAMA8B_LAYER))]) for layer in drawn]
    w = torch.empty(total, dtype=torch.bfloat16, device="cuda")
    for li, bits in enumerate(host):
        w[li * layer_elems:(li + 1) * layer_elems].copy_(to_dev(bits))
    for l in range(len(drawn), inputs.LLAMA8B_LAYERS):
        src = (l % len(drawn)) * layer_elems
        w[l * layer_elems:(l + 1) * layer_elems].copy_(w[src:src + layer_elems])
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)

    def host_bits(k, lo, hi):                       # elements [lo, hi) of tensor k
        layer = shapes[k][0]
        base = int(offs[k]) - layer * layer_elems
        return host[layer % len(drawn)][base + lo:base + hi]

    u8 = dict(dtype=torch.uint8, device="cuda")
    T = range(len(sizes))
    sl = lambda buf, k, bits=8: buf[int(offs[k]) * bits // 8:int(offs[k + 1]) * bits // 8]
    ss = lambda buf, k: buf[int(offs[k]) // BLOCK:int(offs[k + 1]) // BLOCK]
    deq = torch.empty(total, dtype=torch.bfloat16, device="cuda")
    for anchor, low in (("int8", "int4"), ("e4m3", "e2m1")):
        ac, as_ = torch.empty(total, **u8), torch.empty(total // BLOCK, **u8)
        lc, ls = torch.empty(total // 2, **u8), torch.empty(total // BLOCK, **u8)
        mxq.quantize_batched([(w[int(offs[k]):int(offs[k + 1])], sl(ac, k), ss(as_, k)) for k in T], anchor, BLOCK)
        mxq.slice_scale_batched([(sl(ac, k), ss(as_, k), sizes[k], sl(lc, k, 4), ss(ls, k)) for k in T], anchor, low, BLOCK)
        mxq.dequantize_batched([(sl(lc, k, 4), ss(ls, k), sizes[k], deq[int(offs[k]):int(offs[k + 1])]) for k in T], low, BLOCK)
        torch.cuda.synchronize()
        for k in T:
            for lo, hi in sample_runs(sizes[k] // BLOCK, 1, 256, k):
                x = host_bits(k, lo * BLOCK, hi * BLOCK)
                wc, ws = orc.quantize(x, anchor, BLOCK)
                assert bits_equal(dev_slice(ss(as_, k), lo, hi), ws), (anchor, k, lo)
                assert bits_equal(dev_slice(sl(ac, k), lo * BLOCK, hi * BLOCK), orc.pack(wc, 8)), (anchor, k, lo)
                w4, s4 = orc.slice_scale(wc, ws, anchor, low, BLOCK)
                assert bits_equal(dev_slice(sl(lc, k, 4), lo * BLOCK // 2, hi * BLOCK // 2), orc.pack(w4, 4)), (low, k, lo)
                assert bits_equal(dev_slice(ss(ls, k), lo, hi), s4), (low, k, lo)
                want = orc.dequantize(w4, s4, low, BLOCK, orc.BF16)
                got = dev_slice(deq[int(offs[k]):int(offs[k + 1])], lo * BLOCK, hi * BLOCK)
                assert bits_equal(got, want), (low, k, lo, first_diff(got, want))
        del ac, as_, lc, ls
    fq = deq                                        # reuse the arena
    mxq.fake_quant_batched([(w[int(offs[k]):int(offs[k + 1])], fq[int(offs[k]):int(offs[k + 1])]) for k in T], "e2m3", BLOCK,
                           mxq.FQ_VIA_ANCHOR)
    torch.cuda.synchronize()
    for k in T:
        for lo, hi in sample_runs(sizes[k] // BLOCK, 1, 256, 1000 + k):
            want = orc.fake_quant(host_bits(k, lo * BLOCK, hi * BLOCK), "e2m3", BLOCK, orc.FQ_VIA_ANCHOR)
            got = dev_slice(fq[int(offs[k]):int(offs[k + 1])], lo * BLOCK, hi * BLOCK)
            assert bits_equal(got, want), ("fake_quant", k, lo, first_diff(got, want))
    grad = torch.empty_like(fq)
    mxq.fake_quant_bwd(fq, grad)                    # 6.98 G elements in one call
    torch.cuda.synchronize()
    for lo in (0, total // 3, total - (1 << 20)):
        assert torch.equal(grad[lo:lo + (1 << 20)].view(torch.int16), fq[lo:lo + (1 << 20)].view(torch.int16))


# ---------------------------------------------------------------------------------------------
# workload 4: BF16 activations [8 x 4096, 4096] with hot channels; per call a format sampled by seed,
# both routes (direct, through the anchor), and the straight-through backward
# ---------------------------------------------------------------------------------------------

def test_workload4_fake_quant_activations():
    x = inputs.activations_bf16(8, 4096, 4096, seed=4)
    n = x.size
    xd = to_dev(x)
    seen = set()
    for seed in range(200):                          # calls until every format of the list has come up
        fmt = inputs.fq_format_for_call(seed)
        if fmt in seen:
            continue
        seen.add(fmt)
        runs = sample_runs(n // BLOCK, 24, 2048, seed)
        for mode in (mxq.FQ_DIRECT, mxq.FQ_VIA_ANCHOR):
            y = mxq.fake_quant(xd, fmt, BLOCK, mode)
            for lo, hi in runs:
                want = orc.fake_quant(x[lo * BLOCK:hi * BLOCK], fmt, BLOCK, mode)
                got = dev_slice(y, lo * BLOCK, hi * BLOCK)
                assert bits_equal(got, want), (fmt, mode, lo, first_diff(got, want))
            del y
    assert seen == set(inputs.FQ_FORMATS)
    g = mxq.fake_quant_bwd(xd)
    torch.cuda.synchronize()
    assert torch.equal(g.view(torch.int16), xd.view(torch.int16))


# ---------------------------------------------------------------------------------------------
# workload 5: flat BF16 N(0,1) vectors of 2^16 .. 2^31 elements, every anchor-to-lower pair and direct
# quantization.  2^27 elements are drawn on the host (seed 5); longer vectors repeat them on the device.
# ---------------------------------------------------------------------------------------------

_W5_BASE = 1 << 27


@pytest.fixture(scope="module")
def w5_base():
    return inputs.flat_bf16_normal(_W5_BASE, seed=5)


# every size of the sweep up to 2^26 (whole tensors up to 2^20, sampled block runs above), then 2^28, the
# 2^31 end of the sweep, and 2^33: beyond the listed sizes, element and byte offsets past 2^32
@pytest.mark.parametrize("log2n", list(range(16, 27)) + [28, 31, 33])
def test_workload5_size_sweep(w5_base, log2n):
    n = 1 << log2n
    base = w5_base
    if n <= _W5_BASE:
        xd = to_dev(base[:n])
    else:
        xd = to_dev(base).repeat(n // _W5_BASE)

    def x_host(lo, hi):                              # elements [lo, hi) of the (possibly repeated) vector
        lo_m = lo % _W5_BASE
        assert lo_m + (hi - lo) <= _W5_BASE
        return base[lo_m:lo_m + (hi - lo)]

    nblk = n // BLOCK
    full = log2n <= 20
    runs = [(0, nblk)] if full else sample_runs(nblk, 12, 2048, log2n)
    for anchor, lows in (("int8", ("int6", "int4")), ("e4m3", ("e2m3", "e3m2", "e2m1"))):
        codes, scales = check_quantize(x_host, xd, anchor, runs, "w5 2^%d" % log2n)
        for dst in lows:
            check_slice_scale(codes, scales, n, anchor, dst, runs, "w5 2^%d" % log2n)
        del codes, scales
    for fmt in ("int6", "int4", "e2m3", "e2m1"):
        c, s = check_quantize(x_host, xd, fmt, runs, "w5 direct 2^%d" % log2n)
        del c, s
