"""Seeded synthetic inputs shared by the tests, the bench and the oracle checks.

This module holds NO quantization arithmetic: it only draws numbers with
``numpy.random.default_rng`` on the host and narrows FP32 to BF16 bit patterns, so the
CUDA path and the CPU oracle can be fed identical bits.  The tensors take the shapes and
rough value statistics of LLM linear-layer weights and activations (the paper's workload,
Sec. 3.1-3.2); they stand in for the pretrained weights, which are not needed to exercise
the conversion path.

FP32 tensors are ``float32`` arrays; BF16 tensors are ``uint16`` arrays of bit patterns.
"""
from __future__ import annotations

import numpy as np

#: the six element formats a fake-quant call samples from, in the order the workload lists them
FQ_FORMATS = ("int8", "int6", "int4", "e4m3", "e2m3", "e2m1")

#: (name, rows, cols) of the linear weights of one 8B Llama-shaped decoder layer
LLAMA8B_LAYER = (
    ("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
    ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336),
)
LLAMA8B_LAYERS = 32


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """FP32 -> BF16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    return ((u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def weight_f32_normal(rows: int = 4096, cols: int = 4096, seed: int = 0, std: float = 0.02) -> np.ndarray:
    """FP32 weight matrix, N(0, std^2) (workload 1: 4096 x 4096, seed 0)."""
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)).reshape(-1)


def weight_bf16_student_t(rows: int = 8192, cols: int = 8192, seed: int = 1, std: float = 0.02,
                          outlier_frac: float = 0.001, outlier_gain: float = 50.0) -> np.ndarray:
    """BF16 weight matrix: Student-t (nu = 4) scaled to `std`, a fraction of the entries
    multiplied by `outlier_gain` (workload 2)."""
    rng = np.random.default_rng(seed)
    t = rng.standard_t(4, size=(rows, cols)).astype(np.float32)
    t *= np.float32(std / np.sqrt(2.0))  # Var(t_4) = 2
    mask = rng.random((rows, cols), dtype=np.float32) < outlier_frac
    t[mask] *= np.float32(outlier_gain)
    return to_bf16_bits(t.reshape(-1))


def weight_bf16_normal(rows: int, cols: int, seed: int, std: float = 0.02) -> np.ndarray:
    """BF16 weight matrix N(0, std^2) (one tensor of workload 3)."""
    rng = np.random.default_rng(seed)
    return to_bf16_bits((rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)).reshape(-1))


def llama8b_tensor(layer: int, idx: int) -> np.ndarray:
    """Tensor `idx` (order of LLAMA8B_LAYER) of decoder layer `layer`, seed 1000*layer + idx."""
    _, r, c = LLAMA8B_LAYER[idx]
    return weight_bf16_normal(r, c, seed=1000 * layer + idx)


def llama8b_shapes():
    """All (layer, idx, name, rows, cols) of the 224-tensor weight set."""
    return [(l, i, n, r, c) for l in range(LLAMA8B_LAYERS) for i, (n, r, c) in enumerate(LLAMA8B_LAYER)]


def activations_bf16(batch: int = 8, tokens: int = 4096, hidden: int = 4096, seed: int = 4,
                     hot_frac: float = 0.01, hot_gain: float = 20.0) -> np.ndarray:
    """BF16 activations N(0,1) with a fraction of the channels (last dim) scaled up (workload 4)."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((batch * tokens, hidden), dtype=np.float32)
    hot = rng.choice(hidden, max(1, int(round(hidden * hot_frac))), replace=False)
    x[:, hot] *= np.float32(hot_gain)
    return to_bf16_bits(x.reshape(-1))


def fq_format_for_call(seed: int) -> str:
    """The element format a fake-quant call uses, sampled by seed (workload 4)."""
    return FQ_FORMATS[int(np.random.default_rng(seed).integers(0, len(FQ_FORMATS)))]


def flat_bf16_normal(n: int, seed: int = 5) -> np.ndarray:
    """Flat BF16 N(0,1) vector of n elements (workload 5); drawn in chunks to bound host memory."""
    rng = np.random.default_rng(seed)
    out = np.empty(n, np.uint16)
    step = 1 << 24
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = to_bf16_bits(rng.standard_normal(hi - lo, dtype=np.float32))
    return out


def adversarial_f32(block: int = 32) -> np.ndarray:
    """A few dozen hand-built FP32 blocks: zeros, signed zeros, subnormals, exact ties on the
    integer grid, power-of-two maxima, values one ulp either side of them, FLT_MAX, a block
    whose scale clamps at the bottom of E8M0, NaN and Inf."""
    f = np.float32
    blocks = []

    def blk(vals, fill=0.0):
        a = np.full(block, fill, np.float32)
        a[:len(vals)] = np.asarray(vals, np.float32)
        blocks.append(a)

    blk([])                                                   # all +0
    blk([-0.0] * block)                                       # all -0
    blk([1.0] * block)                                        # all equal, power of two
    blk([1.0, -1.0, 0.5, -0.5, 0.25, 0.75, 1.5, -1.75])
    blk([np.nextafter(f(1.0), f(0.0)), 0.3, -0.3])            # amax just below 2^0
    blk([np.nextafter(f(1.0), f(2.0)), 0.3, -0.3])            # amax just above 2^0
    blk([64.0] + [(i + 0.5) for i in range(31)])              # exact .5 ties for INT8 (X = 1)
    blk([-64.0] + [-(i + 0.5) for i in range(31)])
    blk([127.5, 127.4999, 126.5, -127.5])                     # top-bin clipping for INT8
    blk([448.0, 464.0, 465.0, 479.0, 480.0, 20.0, 18.0, 17.0, -464.0])  # E4M3 saturation/ties (X=1)
    blk([255.0, 254.0, 253.0, 240.0, 7.75, 7.5, 7.25, 6.5, 5.0, 3.5, 2.5, 1.25, 0.75, 0.25])
    blk([6.0, 5.0, 4.5, 3.5, 2.5, 1.75, 1.25, 0.75, 0.25, 0.26, 0.24, -0.25, -5.0, -7.0])
    blk([1000.0] + [0.001] * 31)                              # one outlier
    blk([np.float32(2.0 ** -149)] * 3)                        # smallest subnormal
    blk([np.float32(2.0 ** -127), np.float32(2.0 ** -128), np.float32(-2.0 ** -140)])
    blk([np.float32(2.0 ** -126), np.float32(2.0 ** -127 * 1.5)])
    blk([np.float32(2.0 ** -120), np.float32(2.0 ** -121), np.float32(2.0 ** -126)])
    blk([np.finfo(np.float32).max, -np.finfo(np.float32).max, 1.0])
    blk([np.float32(2.0 ** 127), np.float32(2.0 ** 126 * 1.5), np.float32(2.0 ** 120)])
    blk([np.float32(1e-30), np.float32(-3e-31), np.float32(7e-32)])
    blk([np.nan, 1.0, 2.0])
    blk([1.0, np.inf, 2.0])
    blk([1.0, 2.0, -np.inf] + [0.0] * 28 + [3.0])
    rng = np.random.default_rng(12345)
    for e in (-140, -100, -30, -1, 0, 5, 60, 120):
        blocks.append((rng.standard_normal(block) * 2.0 ** e).astype(np.float32))
    # every lane position holds the maximum once
    for p in range(0, block, 5):
        a = (rng.standard_normal(block) * 0.01).astype(np.float32)
        a[p] = 3.0
        blocks.append(a)
    return np.concatenate(blocks)
