"""The tiled scale order for block-scaled matrix multiplies: the oracle against a hand-worked case
and a second formulation (CPU), the CUDA entry point against the oracle, and -- the pin that counts --
a block-scaled tensor-core matmul of the library in use fed with our codes and tiled scales (GPU)."""
import numpy as np
import pytest
import torch

import paper_2604_00529_b200 as mxq
from oracle import mxq_oracle as orc
from paper_2604_00529_b200 import inputs


def _by_reshapes(s: np.ndarray) -> np.ndarray:
    """Second formulation: pad to whole tiles, split into (row tile, 128, column tile, 4), bring the two
    tile indices to the front, then reorder each 128 x 4 tile as (4 groups of 32 rows) -> (32, 4, 4)."""
    rows, kb = s.shape
    rt, ct = -(-rows // 128), -(-kb // 4)
    p = np.zeros((rt * 128, ct * 4), np.uint8)
    p[:rows, :kb] = s
    t = p.reshape(rt, 128, ct, 4).transpose(0, 2, 1, 3)            # [rt, ct, 128, 4]
    t = t.reshape(rt * ct, 4, 32, 4).transpose(0, 2, 1, 3)          # [tile, 32, 4 groups, 4 cols]
    return np.ascontiguousarray(t).reshape(-1)


def test_oracle_tiled_order_hand_worked():
    rows, kb = 33, 5
    s = (np.arange(rows * kb) % 251 + 1).astype(np.uint8).reshape(rows, kb)
    t = orc.tile_scales(s, rows, kb)
    assert t.size == 1 * 2 * 512
    assert t[0] == s[0, 0] and t[16] == s[1, 0] and t[4] == s[32, 0] and t[7] == s[32, 3]
    assert t[31 * 16 + 1] == s[31, 1] and t[512] == s[0, 4] and t[512 + 16 * 5] == s[5, 4]
    assert t[8] == 0 and t[512 + 1] == 0                             # rows 64.. and column 5 do not exist
    assert np.count_nonzero(t) == rows * kb


@pytest.mark.parametrize("rows,kb", [(1, 1), (128, 4), (129, 4), (128, 5), (300, 7), (4096, 128), (1000, 33)])
def test_oracle_tiled_order_second_formulation(rows, kb):
    s = np.random.default_rng(rows * 1000 + kb).integers(0, 256, (rows, kb)).astype(np.uint8)
    assert np.array_equal(orc.tile_scales(s, rows, kb), _by_reshapes(s))


@pytest.mark.gpu
@pytest.mark.parametrize("rows,kb", [(1, 1), (128, 4), (129, 4), (128, 5), (300, 7), (4096, 128), (1000, 33), (8192, 256)])
def test_gpu_tile_scales_matches_oracle(rows, kb):
    s = np.random.default_rng(rows + kb).integers(0, 256, (rows, kb)).astype(np.uint8)
    nbytes = mxq.tiled_scales_bytes(rows, kb)
    buf = torch.full((nbytes + 512,), 0xA5, dtype=torch.uint8, device="cuda")
    mxq.tile_scales(torch.from_numpy(s).cuda(), rows, kb, buf[256:256 + nbytes])
    torch.cuda.synchronize()
    got = buf.cpu().numpy()
    assert np.array_equal(got[256:256 + nbytes], orc.tile_scales(s, rows, kb))
    assert np.all(got[:256] == 0xA5) and np.all(got[256 + nbytes:] == 0xA5)


_FP = ("e4m3", "e3m3", "e3m2", "e2m3", "e2m2", "e2m1")
# row counts and row lengths (in blocks) that leave whole tiles, ragged tiles in either direction, rows
# shorter than a warp tile (so that one warp's blocks span several rows) and a non-power-of-two divisor
_SHAPES = [(1, 1), (3, 2), (128, 4), (129, 4), (128, 5), (300, 7), (257, 3), (1000, 33), (512, 128), (96, 448)]


def _bf16_matrix(rows, cols, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols)) * 2.0 ** rng.integers(-20, 21, (rows, cols // 32)).repeat(32, axis=1)
    return inputs.to_bf16_bits(x.astype(np.float32).reshape(-1))


def _guarded(nbytes):
    return torch.full((nbytes + 512,), 0xA5, dtype=torch.uint8, device="cuda")


@pytest.mark.gpu
@pytest.mark.parametrize("rows,kb", _SHAPES)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_gpu_quantize_tiled_equals_quantize_then_tile(rows, kb, dtype):
    """Fused entry point against the oracle's quantizer followed by the oracle's tiling, every MXFP format."""
    cols = kb * 32
    bits = _bf16_matrix(rows, cols, rows * 7 + kb)
    if dtype == "bf16":
        host = bits
        x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16).view(rows, cols)
    else:
        host = (bits.astype(np.uint32) << 16).view(np.float32)
        x = torch.from_numpy(host).cuda().view(rows, cols)
    nbytes = mxq.tiled_scales_bytes(rows, kb)
    for fmt in _FP:
        wc, ws = orc.quantize(host, fmt, 32)
        buf = _guarded(nbytes)
        codes, _ = mxq.quantize_tiled(x, fmt, 32, tiled_scales=buf[256:256 + nbytes])
        torch.cuda.synchronize()
        got = buf.cpu().numpy()
        assert np.array_equal(got[256:256 + nbytes], orc.tile_scales(ws.reshape(rows, kb), rows, kb)), fmt
        assert np.all(got[:256] == 0xA5) and np.all(got[256 + nbytes:] == 0xA5)
        assert np.array_equal(codes.cpu().numpy(), orc.pack(wc, orc.bits(fmt))), fmt


@pytest.mark.gpu
@pytest.mark.parametrize("rows,kb", _SHAPES)
def test_gpu_slice_scale_tiled_equals_slice_scale_then_tile(rows, kb):
    cols = kb * 32
    bits = _bf16_matrix(rows, cols, rows * 11 + kb)
    ac, as_ = orc.quantize(bits, "e4m3", 32)
    dc = torch.from_numpy(orc.pack(ac, 8)).cuda()
    ds = torch.from_numpy(as_).cuda()
    nbytes = mxq.tiled_scales_bytes(rows, kb)
    for dst in _FP:
        wc, ws = orc.slice_scale(ac, as_, "e4m3", dst, 32)
        buf = _guarded(nbytes)
        codes, _ = mxq.slice_scale_tiled(dc, ds, rows, cols, "e4m3", dst, 32, out_tiled_scales=buf[256:256 + nbytes])
        torch.cuda.synchronize()
        got = buf.cpu().numpy()
        assert np.array_equal(got[256:256 + nbytes], orc.tile_scales(ws.reshape(rows, kb), rows, kb)), dst
        assert np.all(got[:256] == 0xA5) and np.all(got[256 + nbytes:] == 0xA5)
        assert np.array_equal(codes.cpu().numpy(), orc.pack(wc, orc.bits(dst))), dst


@pytest.mark.gpu
@pytest.mark.parametrize("count", [1, 5, 256, 257, 600])
def test_gpu_slice_scale_tiled_batched_matches_oracle(count):
    """Many small matrices of assorted shapes in one call (more than one launch beyond 256 items), with an
    empty one among them; every output against the oracle's Slice-and-Scale followed by its tiling."""
    rng = np.random.default_rng(count)
    shapes = [(int(rng.integers(1, 200)), 32 * int(rng.integers(1, 12))) for _ in range(count)]
    if count > 3:
        shapes[2] = (0, 64)
    items, want = [], []
    for k, (rows, cols) in enumerate(shapes):
        kb = cols // 32
        n = rows * cols
        bits = _bf16_matrix(rows, cols, 1000 * count + k) if n else np.zeros(0, np.uint16)
        ac, as_ = orc.quantize(bits, "e4m3", 32) if n else (np.zeros(0, np.uint8), np.zeros(0, np.uint8))
        wc, ws = orc.slice_scale(ac, as_, "e4m3", "e2m1", 32) if n else (ac, as_)
        nbytes = mxq.tiled_scales_bytes(rows, kb) if n else 0
        # tensors are padded so that every device pointer keeps the 32-byte alignment inside one arena
        items.append((torch.from_numpy(orc.pack(ac, 8)).cuda() if n else torch.empty(32, dtype=torch.uint8, device="cuda"),
                      torch.from_numpy(as_).cuda() if n else torch.empty(32, dtype=torch.uint8, device="cuda"),
                      rows, cols,
                      torch.full((max(n // 2, 32),), 0xA5, dtype=torch.uint8, device="cuda"),
                      torch.full((max(nbytes, 32),), 0xA5, dtype=torch.uint8, device="cuda")))
        want.append((orc.pack(wc, 4), orc.tile_scales(ws.reshape(rows, kb), rows, kb) if n else None, n, nbytes))
    mxq.slice_scale_tiled_batched(items, "e4m3", "e2m1", 32)
    torch.cuda.synchronize()
    for k, ((_, _, rows, cols, oc, ot), (wc, wt, n, nbytes)) in enumerate(zip(items, want)):
        if n == 0:
            assert bool((oc == 0xA5).all()) and bool((ot == 0xA5).all()), k
            continue
        assert np.array_equal(oc.cpu().numpy()[:n // 2], wc), (k, rows, cols)
        assert np.array_equal(ot.cpu().numpy()[:nbytes], wt), (k, rows, cols)


@pytest.mark.gpu
def test_gpu_tiled_entry_points_full_size_workload():
    """BF16 8192 x 8192 (workload 2): the fused outputs equal the two-pass outputs byte for byte, and
    sampled bands of rows equal the oracle (Eq. 1-3, Eq. 5, then the oracle's own tiling): a band of
    128 rows is one row of scale tiles, so its codes, plain scales and tiled bytes are contiguous slices."""
    xb = inputs.weight_bf16_student_t(8192, 8192, seed=1)
    x = torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16).view(8192, 8192)
    codes, scales = mxq.quantize(x, "e4m3", 32)
    tc, ts = mxq.quantize_tiled(x, "e4m3", 32)
    assert torch.equal(tc, codes) and torch.equal(ts, mxq.tile_scales(scales, 8192, 256))
    fused = {}
    for dst in ("e2m3", "e2m1"):
        lc, ls = mxq.slice_scale(codes, scales, x.numel(), "e4m3", dst, 32)
        fc, fs = mxq.slice_scale_tiled(codes, scales, 8192, 8192, "e4m3", dst, 32)
        assert torch.equal(fc, lc) and torch.equal(fs, mxq.tile_scales(ls, 8192, 256))
        fused[dst] = (fc, fs)
    cols, kb = 8192, 256
    for band in (0, 17, 63):                                  # first, one in the middle, last
        r0 = band * 128
        xs = xb[r0 * cols:(r0 + 128) * cols]
        wc, ws = orc.quantize(xs, "e4m3")
        assert np.array_equal(tc[r0 * cols:(r0 + 128) * cols].cpu().numpy(), orc.pack(wc, 8)), band
        assert np.array_equal(ts[band * 128 * kb:(band + 1) * 128 * kb].cpu().numpy(), orc.tile_scales(ws, 128, kb)), band
        for dst, (fc, fs) in fused.items():
            b = orc.bits(dst)
            lc, ls = orc.slice_scale(wc, ws, "e4m3", dst)
            assert np.array_equal(fc[r0 * cols * b // 8:(r0 + 128) * cols * b // 8].cpu().numpy(), orc.pack(lc, b)), (band, dst)
            assert np.array_equal(fs[band * 128 * kb:(band + 1) * 128 * kb].cpu().numpy(), orc.tile_scales(ls, 128, kb)), (band, dst)


def _mixed_matrix(rows, cols, seed):
    """Rows and 32-wide blocks at very different magnitudes, so that a misplaced scale is a gross error."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols))
    x *= 2.0 ** rng.integers(-6, 7, (rows, 1))
    x *= 2.0 ** rng.integers(-4, 5, (rows, cols // 32)).repeat(32, axis=1)
    return inputs.to_bf16_bits(x.astype(np.float32).reshape(-1))


@pytest.mark.gpu
@pytest.mark.parametrize("fmt", ["e4m3", "e2m1"])
def test_block_scaled_matmul_consumes_codes_and_tiled_scales(fmt):
    """A = [M, K], B = [N, K] quantized along K with block 32; the library's block-scaled matmul on our
    codes and tiled scales must equal dequantize(A) @ dequantize(B)^T."""
    try:
        from torch.nn.functional import ScalingType, SwizzleType, scaled_mm
    except ImportError:
        pytest.skip("this torch has no scaled_mm")
    M, N, K = 256, 384, 1024
    qa = {}
    for name, rows, seed in (("a", M, 1), ("b", N, 2)):
        bits = _mixed_matrix(rows, K, seed)
        x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        codes, scales = mxq.quantize(x, fmt, 32)
        deq = mxq.dequantize(codes, scales, rows * K, fmt, 32, dtype=torch.float32).view(rows, K)
        if name == "a":                              # one operand by the separate pass, the other by the fused kernel
            tiled = mxq.tile_scales(scales, rows, K // 32)
        else:
            codes, tiled = mxq.quantize_tiled(x.view(rows, K), fmt, 32)
        qa[name] = (codes, tiled, deq)
    ref = qa["a"][2].double() @ qa["b"][2].double().t()
    if fmt == "e4m3":
        a = qa["a"][0].view(torch.float8_e4m3fn).view(M, K)
        b = qa["b"][0].view(torch.float8_e4m3fn).view(N, K)
    else:
        a = qa["a"][0].view(torch.float4_e2m1fn_x2).view(M, K // 2)
        b = qa["b"][0].view(torch.float4_e2m1fn_x2).view(N, K // 2)
    sa = qa["a"][1].view(torch.float8_e8m0fnu)
    sb = qa["b"][1].view(torch.float8_e8m0fnu)
    try:
        out = scaled_mm(a, b.t(), sa, ScalingType.BlockWise1x32, sb, ScalingType.BlockWise1x32,
                        swizzle_a=SwizzleType.SWIZZLE_32_4_4, swizzle_b=SwizzleType.SWIZZLE_32_4_4,
                        output_dtype=torch.bfloat16)
    except (RuntimeError, NotImplementedError, ValueError) as e:
        pytest.skip("block-scaled matmul not available for %s here: %s" % (fmt, str(e).splitlines()[0][:200]))
    torch.cuda.synchronize()
    err = (out.double() - ref).abs()
    # BF16 output (8 significant bits) of an FP32 accumulation: a few 2^-8 relative to the row's scale
    tol = 2.0 ** -6 * ref.abs().max(dim=1, keepdim=True).values + 1e-30
    assert bool((err <= tol).all()), "max error / tolerance = %.3g" % float((err / tol).max())
    # and the result is not trivially small: the check has teeth
    assert float(ref.abs().max()) > 0
