"""The oracle's pins must fail when the oracle is wrong.  Each case plants ONE plausible mistake in a
copy of the oracle's C source (a dropped term, a wrong constant, another tie rule, a reversed bit
order ...), builds it, and runs the pin tests against it in a child process: they have to fail.
The mistakes are planted on the CPU, in the oracle only; nothing here touches the CUDA path."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "mxq_oracle.c")

# (name, text in the oracle, replacement)
MUTANTS = [
    ("mxint_emax_off_by_one", "return kind == MXO_INT ? a - 2 : (1 << (a - 1));", "return kind == MXO_INT ? a - 1 : (1 << (a - 1));"),
    ("mxfp_emax_off_by_one", "return kind == MXO_INT ? a - 2 : (1 << (a - 1));", "return kind == MXO_INT ? a - 2 : (1 << (a - 1)) - 1;"),
    ("mxint_ties_toward_zero", "if (a - q >= 0.5) q += 1.0;", "if (a - q > 0.5) q += 1.0;"),
    ("mxint_asymmetric_clip", "double lim = (double)((1 << (b - 1)) - 1);", "double lim = (double)(1 << (b - 1));"),
    ("mxfp_ties_away", "double m = nearbyint(ldexp(a, mu - ea));    /* a / ulp, ulp = 2^(ea-mu); ties to even */",
     "double m = floor(ldexp(a, mu - ea) + 0.5);"),
    ("mxfp_no_subnormals", "if (ea < 1 - bias) ea = 1 - bias;           /* subnormal range shares one ulp */", ""),
    ("mxfp_no_saturation", "if (v > vmax) v = vmax;                     /* clamping */", ""),
    ("mxfp_bias_off_by_one", "static int fp_bias(mxo_fmt f) { return (1 << (f.a - 1)) - 1; }",
     "static int fp_bias(mxo_fmt f) { return (1 << (f.a - 1)); }"),
    ("floor_log2_is_ceil", "    return E - 1;\n", "    return E;\n"),
    ("ssmxint_truncates", "int q = de > 0 ? (mag + (1 << (de - 1))) >> de : mag;", "int q = de > 0 ? mag >> de : mag;"),
    ("ssmxint_no_clip", "        if (q > lim) q = lim;\n        if (p < 0) q = -q;", "        if (p < 0) q = -q;"),
    ("ss_scale_not_adjusted", "unsigned sl = sh == 0xFF ? 0xFF : (sh + (unsigned)de > 254 ? 254 : sh + (unsigned)de);",
     "unsigned sl = sh;"),
    ("ssmxfp_wrong_divisor", "return quantize_fp(fl, ldexp(x, -de));", "return quantize_fp(fl, ldexp(x, -de + 1));"),
    ("dequantize_exponent_off_by_one", "v = ldexp(mxo_decode(kind, a, m, codes[j]), (int)scales[b] - 127);",
     "v = ldexp(mxo_decode(kind, a, m, codes[j]), (int)scales[b] - 126);"),
    ("scale_byte_bias", "*scale = (uint8_t)(shared_exp + 127);", "*scale = (uint8_t)(shared_exp + 128);"),
    ("pack_bits_reversed_in_byte", "out[bit >> 3] |= (uint8_t)(1u << (bit & 7));", "out[bit >> 3] |= (uint8_t)(1u << (7 - (bit & 7)));"),
    ("fake_quant_ignores_anchor_route", "if (mode == MXO_FQ_VIA_ANCHOR) {", "if (0) {"),
    ("e4m3_nan_code_is_a_number", "static int fp_has_nan(mxo_fmt f) { return f.kind == MXO_FP && f.a == 4 && f.m == 3; }",
     "static int fp_has_nan(mxo_fmt f) { (void)f; return 0; }"),
    ("poisoned_block_not_flagged", "            *scale = 0xFF;\n", "            *scale = 0;\n"),
    ("bf16_store_truncates", "double m = nearbyint(ldexp(a, 7 - e));      /* in units of 2^(e-7) */", "double m = floor(ldexp(a, 7 - e));"),
]


def test_every_planted_text_exists_once():
    text = open(SRC).read()
    for name, old, new in MUTANTS:
        assert text.count(old) == 1, name


def _run_mutant(args):
    tmp, name, old, new = args
    d = os.path.join(tmp, name)
    os.makedirs(d)
    src = os.path.join(d, "mxq_oracle.c")
    with open(src, "w") as f:
        f.write(open(SRC).read().replace(old, new))
    env = dict(os.environ, MXQ_ORACLE_SOURCE=src)
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_formats.py"),
                        os.path.join(ROOT, "tests", "test_oracle_blocks.py")],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    return name, r.returncode, r.stdout[-800:]


def test_pins_catch_every_planted_mistake(tmp_path):
    """All mutants at once (one child process each, run side by side to keep the suite short)."""
    from concurrent.futures import ThreadPoolExecutor
    workers = max(2, min(len(MUTANTS), os.cpu_count() or 2))
    with ThreadPoolExecutor(max_workers=workers) as ex:
        results = list(ex.map(_run_mutant, [(str(tmp_path), n, o, w) for n, o, w in MUTANTS]))
    survived = [(n, rc, out) for n, rc, out in results if rc != 1 or " failed" not in out]
    assert not survived, "the pins did not fail with these mistakes planted: %s" % [(n, rc) for n, rc, _ in survived]
