"""Host-side partition of a tensor over ranks for the MX conversion path.

Every MX block is converted on its own (Eq. 1-5 of the MF-QAT paper read one block and write one
block), so a tensor shards over GPUs by contiguous runs of whole blocks and the ranks exchange
nothing: rank r converts elements [lo, hi), writes code bytes [lo*bits/8, hi*bits/8) and scale bytes
[lo/block, hi/block) of the full outputs.  Shard boundaries are kept on multiples of 32 blocks so
that every rank's code, scale and tensor pointers keep the 32-byte alignment the kernels need.
"""
from __future__ import annotations

from typing import Tuple

#: shard boundaries fall on multiples of this many blocks (32 scale bytes = one aligned scale chunk)
BLOCKS_PER_CHUNK = 32


def block_range(n: int, block: int, rank: int, world: int) -> Tuple[int, int]:
    """Element range [lo, hi) of `rank` out of `world` for a tensor of `n` elements.

    n must be a multiple of block.  Chunks of BLOCKS_PER_CHUNK blocks are dealt out as evenly as
    possible, the first ranks taking one more; the ragged last chunk goes to the last rank that has
    work.  Ranges are contiguous, disjoint and cover [0, n).
    """
    if block <= 0 or n % block:
        raise ValueError("n must be a multiple of block")
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    nblk = n // block
    nchunk = -(-nblk // BLOCKS_PER_CHUNK)
    base, extra = divmod(nchunk, world)
    c_lo = rank * base + min(rank, extra)
    c_hi = c_lo + base + (1 if rank < extra else 0)
    lo = min(c_lo * BLOCKS_PER_CHUNK, nblk) * block
    hi = min(c_hi * BLOCKS_PER_CHUNK, nblk) * block
    return lo, hi


def output_ranges(lo: int, hi: int, bits: int, block: int):
    """Byte ranges ((codes_lo, codes_hi), (scales_lo, scales_hi)) of the packed outputs that the
    element range [lo, hi) owns."""
    return (lo * bits // 8, hi * bits // 8), (lo // block, hi // block)


def quantize_shard(src, fmt: str, block: int, codes, scales, rank: int, world: int, stream=None):
    """Rank `rank`'s part of mxq_quantize(src -> codes, scales): converts the rank's run of whole blocks
    of the full tensor `src` into the matching byte ranges of the full output buffers (all of them
    device tensors of the FULL size; with one process per GPU each rank passes its own copies or
    views).  Returns the element range [lo, hi) it converted."""
    from . import binding
    lo, hi = block_range(src.numel(), block, rank, world)
    if hi > lo:
        (c_lo, c_hi), (s_lo, s_hi) = output_ranges(lo, hi, binding.format_bits(fmt), block)
        binding.quantize(src.reshape(-1)[lo:hi], fmt, block, codes[c_lo:c_hi], scales[s_lo:s_hi], stream)
    return lo, hi


def slice_scale_shard(codes, scales, n: int, src_fmt: str, dst_fmt: str, block: int, out_codes, out_scales,
                      rank: int, world: int, stream=None):
    """Rank `rank`'s part of mxq_slice_scale over full-size buffers (see quantize_shard)."""
    from . import binding
    lo, hi = block_range(n, block, rank, world)
    if hi > lo:
        (a_lo, a_hi), (s_lo, s_hi) = output_ranges(lo, hi, binding.format_bits(src_fmt), block)
        (c_lo, c_hi), _ = output_ranges(lo, hi, binding.format_bits(dst_fmt), block)
        binding.slice_scale(codes[a_lo:a_hi], scales[s_lo:s_hi], hi - lo, src_fmt, dst_fmt, block,
                            out_codes[c_lo:c_hi], out_scales[s_lo:s_hi], stream)
    return lo, hi
