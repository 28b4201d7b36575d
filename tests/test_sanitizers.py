"""Host code under AddressSanitizer and UBSan (no GPU): the CPU oracle on exactly sized heap buffers
over every format, pair and block size, and the argument checks of the C ABI (the layer that walks
the callers' item arrays) on the paths that return before any CUDA call.  An out-of-bounds access,
a signed overflow or a bad shift aborts the program under test."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NATIVE = os.path.join(ROOT, "tests", "native")
SAN = ["-fsanitize=address", "-fsanitize=undefined", "-fno-sanitize-recover=all"]
ENV = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1")


def _run(cmd, **kw):
    r = subprocess.run(cmd, capture_output=True, text=True, **kw)
    assert r.returncode == 0, "%s\n%s\n%s" % (" ".join(cmd), r.stdout[-2000:], r.stderr[-4000:])
    return r.stdout


def test_oracle_is_clean_under_asan_and_ubsan(tmp_path):
    exe = str(tmp_path / "oracle_sanitize")
    _run(["gcc", "-O1", "-g", "-std=c11", *SAN, "-fno-fast-math", "-ffp-contract=off", "-o", exe,
          os.path.join(NATIVE, "oracle_sanitize.c"), os.path.join(ROOT, "oracle", "mxq_oracle.c"), "-lm"])
    assert _run([exe], env=ENV).strip().endswith("ok")


@pytest.mark.skipif(shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"), reason="needs nvcc")
def test_abi_argument_checks_are_clean_under_asan_and_ubsan(tmp_path):
    from paper_2604_00529_b200 import build
    build.build()                                           # the kernel objects the sanitized ABI layer links against
    nvcc = build._nvcc()
    xsan = [x for f in SAN for x in ("-Xcompiler", f)]
    units = ["mxq_api", "mxq_static_batch", "mxq_layout"]   # every translation unit with extern "C" entry points
    objs = []
    for u in units:
        obj = str(tmp_path / (u + ".o"))
        _run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++20", "-O1", "-g", "-Xcompiler", "-fPIC", *xsan,
              "-c", os.path.join(build.CSRC, u + ".cu"), "-o", obj])
        objs.append(obj)
    others = [os.path.join(build.OBJ_DIR, u + ".o") for u in build.UNITS if u not in units]
    lib = str(tmp_path / "libmxq.so")
    _run([nvcc, "-shared", "-o", lib, *objs, *others, "-gencode", "arch=compute_100a,code=sm_100a", *xsan])
    exe = str(tmp_path / "abi_sanitize")
    _run(["gcc", "-O1", "-g", "-std=c11", *SAN, "-o", exe, os.path.join(NATIVE, "abi_sanitize.c"),
          "-L" + str(tmp_path), "-lmxq", "-Wl,-rpath," + str(tmp_path)])
    assert _run([exe], env=ENV).strip().endswith("ok")
