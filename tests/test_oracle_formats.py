"""Pins for the oracle's element formats: code tables and the element quantizers.

The paper prints no code table or worked example, so the oracle is pinned to what the
formats' published definitions and independent implementations fix: the ml_dtypes / torch
casts for the OCP element types, published value sets, and an exact-rational brute-force
nearest-neighbour search written here (sharing nothing with the oracle's arithmetic).
"""
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest
import torch

from oracle import mxq_oracle as orc

INT_FORMATS = ["int8", "int7", "int6", "int5", "int4", "int3", "int2"]
FP_FORMATS = ["e4m3", "e3m3", "e3m2", "e2m3", "e2m2", "e2m1"]
ML = {"e4m3": ml_dtypes.float8_e4m3fn, "e3m2": ml_dtypes.float6_e3m2fn,
      "e2m3": ml_dtypes.float6_e2m3fn, "e2m1": ml_dtypes.float4_e2m1fn}

# largest magnitude, smallest non-zero magnitude, e_max -- from the OCP MX element definitions
FP_FACTS = {"e4m3": (448.0, 2.0 ** -9, 8), "e3m3": (30.0, 2.0 ** -5, 4), "e3m2": (28.0, 2.0 ** -4, 4),
            "e2m3": (7.5, 0.125, 2), "e2m2": (7.0, 0.25, 2), "e2m1": (6.0, 0.5, 2)}


# ----------------------------------------------------------------------------------------
# decode tables
# ----------------------------------------------------------------------------------------

@pytest.mark.parametrize("fmt", list(ML))
def test_decode_matches_ml_dtypes(fmt):
    """Every code decodes to the value the ml_dtypes implementation of the same OCP type gives."""
    nb = orc.bits(fmt)
    codes = np.arange(1 << nb, dtype=np.uint8)
    want = codes.view(ML[fmt]).astype(np.float64)
    got = orc.decode_table(fmt)
    assert np.array_equal(np.isnan(want), np.isnan(got))
    ok = ~np.isnan(want)
    assert np.array_equal(want[ok], got[ok])
    assert np.array_equal(np.signbit(want[ok]), np.signbit(got[ok]))  # -0 keeps its sign


def test_decode_e4m3_matches_torch():
    codes = torch.arange(256, dtype=torch.uint8)
    want = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = orc.decode_table("e4m3")
    assert np.array_equal(np.isnan(want), np.isnan(got))
    assert np.array_equal(want[~np.isnan(want)], got[~np.isnan(got)])


def test_e2m1_value_set():
    """FP4 E2M1 represents exactly +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}."""
    t = orc.decode_table("e2m1")
    assert list(t[:8]) == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    assert list(t[8:]) == [-0.0, -0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -6.0]


@pytest.mark.parametrize("fmt", FP_FORMATS)
def test_fp_table_structure(fmt):
    nb = orc.bits(fmt)
    t = orc.decode_table(fmt)
    half = 1 << (nb - 1)
    pos, neg = t[:half], t[half:]
    n_nan = int(np.isnan(t).sum())
    assert n_nan == (2 if fmt == "e4m3" else 0)        # E4M3: S.1111.111 only; no other specials
    finite = pos[~np.isnan(pos)]
    assert np.all(np.diff(finite) > 0)                 # magnitude codes are strictly increasing
    assert np.array_equal(-finite, neg[~np.isnan(neg)])
    vmax, vmin, emax = FP_FACTS[fmt]
    assert finite[-1] == vmax == orc.max_value(fmt)
    assert finite[1] == vmin
    assert orc.emax(fmt) == emax == int(np.floor(np.log2(vmax)))
    assert not np.any(np.isinf(t))


@pytest.mark.parametrize("fmt", INT_FORMATS)
def test_int_table(fmt):
    b = orc.bits(fmt)
    t = orc.decode_table(fmt)
    want = np.array([c if c < (1 << (b - 1)) else c - (1 << b) for c in range(1 << b)], float)
    assert np.array_equal(t, want)                      # two's complement
    assert orc.max_value(fmt) == 2 ** (b - 1) - 1
    # e_max(b) = exponent of the largest magnitude, so that de = b_h - b_l (Sec. 3.3)
    assert orc.emax(fmt) == b - 2 == int(np.floor(np.log2(2 ** (b - 1) - 1))) or b == 2
    assert orc.emax("int8") - orc.emax(fmt) == 8 - b


# ----------------------------------------------------------------------------------------
# element quantizer against an exact-rational brute force
# ----------------------------------------------------------------------------------------

def _finite_table(fmt):
    """[(code, Fraction value)] of the non-negative finite codes, from the decode table."""
    nb = orc.bits(fmt)
    out = []
    for c in range(1 << (nb - 1)):
        v = orc.decode(fmt, c)
        if not np.isnan(v):
            out.append((c, Fraction(v)))
    return out


def brute_force_quantize(fmt, r):
    """Nearest representable value by exhaustive search on exact rationals.
    Ties: MXFP -> the candidate whose code is even (round-half-to-even on the mantissa),
    MXINT -> the larger magnitude (away from zero).  Values beyond the largest magnitude
    saturate.  MXINT uses the symmetric range."""
    kind = orc.FORMATS[fmt][0]
    nb = orc.bits(fmt)
    neg = np.signbit(r)
    a = abs(Fraction(r))
    tab = _finite_table(fmt)
    best = None
    for c, v in tab:
        d = abs(v - a)
        if best is None or d < best[0]:
            best = (d, c, v)
        elif d == best[0]:
            if kind == 0:
                if v > best[2]:
                    best = (d, c, v)
            elif c % 2 == 0:
                best = (d, c, v)
    code = best[1]
    if kind == 0:
        q = -code if neg else code
        return q & ((1 << nb) - 1)
    return code | ((1 << (nb - 1)) if neg else 0)


def _breakpoints(fmt):
    """Every representable magnitude, every midpoint of neighbours, and their float neighbours."""
    tab = [float(v) for _, v in _finite_table(fmt)]
    pts = set()
    top = tab[-1]
    step = tab[-1] - tab[-2]
    grid = tab + [top + step / 2, top + step, top * 4]
    for lo, hi in zip(grid[:-1], grid[1:]):
        for p in (lo, (lo + hi) / 2, hi):
            pts.update((p, np.nextafter(p, np.inf), np.nextafter(p, -np.inf)))
    pts.update((0.0, 2.0 ** -40, 2.0 ** -200))
    return sorted(pts)


@pytest.mark.parametrize("fmt", INT_FORMATS + FP_FORMATS)
def test_quantize_elem_breakpoints(fmt):
    for p in _breakpoints(fmt):
        for r in (p, -p):
            assert orc.quantize_elem(fmt, r) == brute_force_quantize(fmt, r), (fmt, r)


@pytest.mark.parametrize("fmt", INT_FORMATS + FP_FORMATS)
def test_quantize_elem_random(fmt):
    rng = np.random.default_rng(7)
    top = orc.max_value(fmt)
    xs = np.concatenate([rng.uniform(-1.2 * top, 1.2 * top, 1500),
                         rng.standard_normal(1500) * top / 8,
                         rng.standard_normal(500) * 2.0 ** -6])
    for r in xs:
        assert orc.quantize_elem(fmt, float(r)) == brute_force_quantize(fmt, float(r)), (fmt, r)


@pytest.mark.parametrize("fmt", INT_FORMATS + FP_FORMATS)
def test_quantize_is_idempotent_on_codes(fmt):
    """quantize_f(decode_f(c)) == c for every finite code (MXINT: every code but -2^(b-1))."""
    nb = orc.bits(fmt)
    for c in range(1 << nb):
        v = orc.decode(fmt, c)
        if np.isnan(v):
            continue
        if orc.FORMATS[fmt][0] == 0 and c == 1 << (nb - 1):
            assert orc.quantize_elem(fmt, v) == (c + 1)      # -2^(b-1) clips to -(2^(b-1)-1)
            continue
        assert orc.quantize_elem(fmt, v) == c, (fmt, c)


@pytest.mark.parametrize("fmt", list(ML))
def test_quantize_elem_matches_ml_dtypes_cast(fmt):
    """In range, the element quantizer is the round-to-nearest-even cast of an independent library."""
    rng = np.random.default_rng(11)
    top = orc.max_value(fmt)
    xs = np.concatenate([rng.uniform(-top, top, 20000), rng.standard_normal(20000) * top / 16])
    # FP32 inputs (the library narrows float64 through float32, which would round twice)
    b32 = np.array(_breakpoints(fmt), np.float32)
    xs = np.concatenate([xs, b32, np.nextafter(b32, np.float32(np.inf)),
                         np.nextafter(b32, np.float32(-np.inf))]).astype(np.float32)
    xs = xs[np.abs(xs) <= top]
    want = xs.astype(ML[fmt]).view(np.uint8)
    mask = (1 << orc.bits(fmt)) - 1
    got = np.array([orc.quantize_elem(fmt, float(x)) for x in xs], np.uint8)
    assert np.array_equal(want & mask, got)


def test_quantize_elem_matches_torch_e4m3_cast():
    rng = np.random.default_rng(13)
    xs = np.concatenate([rng.uniform(-448, 448, 20000), rng.standard_normal(20000) * 0.01]).astype(np.float32)
    want = torch.from_numpy(xs).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([orc.quantize_elem("e4m3", float(x)) for x in xs], np.uint8)
    assert np.array_equal(want, got)


def test_int_round_is_away_from_zero_and_symmetric():
    for b in (2, 3, 4, 6, 8):
        fmt = "int%d" % b
        lim = 2 ** (b - 1) - 1
        mask = (1 << b) - 1
        for k in range(0, lim):
            assert orc.quantize_elem(fmt, k + 0.5) == (k + 1) & mask
            assert orc.quantize_elem(fmt, -(k + 0.5)) == (-(k + 1)) & mask
        assert orc.quantize_elem(fmt, 1e9) == lim
        assert orc.quantize_elem(fmt, -1e9) == (-lim) & mask          # never -2^(b-1)
        assert orc.quantize_elem(fmt, np.nextafter(0.5, 0)) == 0


# ----------------------------------------------------------------------------------------
# E8M0 scale byte and the packed layout
# ----------------------------------------------------------------------------------------

def test_scale_byte_is_e8m0():
    """dequantize(P = 1, byte) is 2^(byte-127): the same value ml_dtypes gives the E8M0 code."""
    bytes_ = np.arange(0, 255, dtype=np.uint8)
    want = bytes_.view(ml_dtypes.float8_e8m0fnu).astype(np.float64)
    codes = np.ones(255, np.uint8)
    got = orc.dequantize(codes, bytes_, "int8", block=1).astype(np.float64)
    assert np.array_equal(want[1:], got[1:])
    assert got[0] == 2.0 ** -127           # FP32 subnormal, exact
    assert np.isnan(orc.dequantize(np.ones(1, np.uint8), np.array([255], np.uint8), "int8", block=1))[0]


@pytest.mark.parametrize("nb", [2, 3, 4, 5, 6, 7, 8])
def test_pack_layout(nb):
    """Element i occupies bits [i*nb, (i+1)*nb) of a little-endian bitstream."""
    rng = np.random.default_rng(nb)
    n = 96
    codes = rng.integers(0, 1 << nb, n).astype(np.uint8)
    packed = orc.pack(codes, nb)
    big = sum(int(c) << (i * nb) for i, c in enumerate(codes))
    assert bytes(packed) == big.to_bytes(n * nb // 8, "little")
    assert np.array_equal(orc.unpack(packed, n, nb), codes)
    if nb == 4:
        assert packed[0] == (codes[0] | (codes[1] << 4))
    if nb == 8:
        assert np.array_equal(packed, codes)


def test_ssmxint_other_tie_rules_would_differ_on_these_codes():
    """What the reading of Eq. 4's Round is worth: how many of the 255 anchor codes would convert
    differently under round-half-to-even or under round-half-up (toward +infinity), per exponent
    difference.  Only exact ties differ -- 32 / 8 / 2 codes for ties-to-even (every second tie) and
    31 / 7 / 1 for half-up (every negative tie that the clip does not absorb) -- so the oracle's rule
    is pinned against both alternatives by those codes and by nothing else."""
    for (src, dst), (want_even, want_up) in {("int8", "int6"): (32, 31), ("int8", "int4"): (8, 7),
                                             ("int8", "int2"): (2, 1)}.items():
        de = 8 - orc.bits(dst)
        top = 2 ** (orc.bits(dst) - 1) - 1
        even = up = 0
        for p in range(-127, 128):
            got = orc.slice_scale_elem(src, dst, p & 0xFF)
            got = got - (1 << orc.bits(dst)) if got >> (orc.bits(dst) - 1) else got
            x = Fraction(p, 1 << de)
            lo = x.numerator // x.denominator
            frac = x - lo
            rne = lo + (1 if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2) else 0)
            hup = (x + Fraction(1, 2)).numerator // (x + Fraction(1, 2)).denominator
            clip = lambda q: max(-top, min(top, q))
            even += clip(rne) != got
            up += clip(hup) != got
            if frac != Fraction(1, 2):
                assert clip(rne) == got == clip(hup), (src, dst, p)
        assert (even, up) == (want_even, want_up), (src, dst, even, up)
