"""Bandwidth sweep of libmxq on one GPU.

    python -m paper_2604_00529_b200.sweep [--min-log2 16] [--max-log2 31] [--model] [--all-formats] [--tiled] [--graph] [--warm] [--json out.json]

`--graph` times CUDA-graph replays instead of direct launches.  For flat BF16 N(0,1) vectors of 2^k elements: direct quantization to each format, Slice-and-Scale
for every anchor-to-lower pair, reconstruction and the fused fake-quant, timed with CUDA events over
back-to-back launches that rotate over enough buffer copies to exceed the 126 MB L2 (small sizes
therefore show launch-bound, not cache-resident, figures).  GB/s counts algorithmic bytes (read +
written).  `--model` adds the whole-model conversion of an 8B Llama-shaped weight set (224 tensors,
6.98 G elements) through one batched launch per target.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

import paper_2604_00529_b200 as mxq
from paper_2604_00529_b200 import inputs

BLOCK = 32
L2_BYTES = 126 << 20


def _peak():
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


WARM = False      # --warm: one buffer set for every launch, so that sizes below the L2 capacity run out of L2
GRAPH = False     # --graph: time the replay of a CUDA graph that holds the launches (no host cost per launch)


def _time(launch, copies: int, reps: int) -> float:
    """Average microseconds per launch; launch(j) must use buffer copy j."""
    if GRAPH:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for j in range(min(3, copies)):
                launch(j)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(reps):
                launch(i % copies)
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / reps
    for j in range(min(3, copies)):
        launch(j)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(reps):
        launch(i % copies)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / reps


def sweep_size(n: int, base_dev: torch.Tensor, reps: int):
    """All ops at n elements; returns {op: (us, GB/s)}."""
    bits = {"int8": 8, "int6": 6, "int4": 4, "e4m3": 8, "e3m2": 6, "e2m3": 6, "e2m1": 4}
    # enough rotating copies that a buffer is not found in L2 again (at least 2, at most 2048)
    copies = int(min(2048, max(2, -(-2 * L2_BYTES // (2 * n)))))
    if n * 2 * copies > 24 << 30:
        copies = 2
    if WARM:
        copies = 1
    xs = [base_dev[:n].clone() if n <= base_dev.numel() else base_dev.repeat(n // base_dev.numel()) for _ in range(copies)]
    u8 = dict(dtype=torch.uint8, device="cuda")
    out = {}

    def rec(name, us, bytes_per_elem):
        out[name] = (us, bytes_per_elem * n / us / 1e3)

    anchors = {}
    for fmt in ("int8", "e4m3", "int6", "int4", "e2m3", "e2m1"):
        cs = [(torch.empty(n * bits[fmt] // 8, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
        us = _time(lambda j: mxq.quantize(xs[j], fmt, BLOCK, *cs[j]), copies, reps)
        rec("quantize_bf16_" + fmt, us, 2 + bits[fmt] / 8 + 1 / BLOCK)
        if fmt in ("int8", "e4m3"):
            anchors[fmt] = cs
        else:
            del cs
    for src, dsts in (("int8", ("int6", "int4")), ("e4m3", ("e2m3", "e3m2", "e2m1"))):
        for dst in dsts:
            os_ = [(torch.empty(n * bits[dst] // 8, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
            us = _time(lambda j: mxq.slice_scale(*anchors[src][j], n, src, dst, BLOCK, *os_[j]), copies, reps)
            rec("slice_scale_%s_%s" % (src, dst), us, 1 + bits[dst] / 8 + 2 / BLOCK)
            if dst in ("int4", "e2m1"):
                ys = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(copies)]
                us = _time(lambda j: mxq.dequantize(*os_[j], n, dst, BLOCK, dst=ys[j]), copies, reps)
                rec("dequantize_%s_bf16" % dst, us, bits[dst] / 8 + 1 / BLOCK + 2)
                del ys
            del os_
    two = [[(torch.empty(n * 6 // 8, **u8), torch.empty(n // BLOCK, **u8)), (torch.empty(n // 2, **u8), torch.empty(n // BLOCK, **u8))]
           for _ in range(copies)]
    us = _time(lambda j: mxq.slice_scale_multi(*anchors["e4m3"][j], n, "e4m3", ("e2m3", "e2m1"), BLOCK, two[j]), copies, reps)
    rec("slice_scale_multi_e4m3_e2m3+e2m1", us, 1 + 6 / 8 + 4 / 8 + 3 / BLOCK)
    del two, anchors
    ys = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(copies)]
    for fmt, mode, tag in (("e2m3", mxq.FQ_VIA_ANCHOR, "via_anchor"), ("int4", mxq.FQ_DIRECT, "direct"),
                           ("int4", mxq.FQ_VIA_ANCHOR, "via_anchor"), ("e2m1", mxq.FQ_VIA_ANCHOR, "via_anchor")):
        us = _time(lambda j: mxq.fake_quant(xs[j], fmt, BLOCK, mode, dst=ys[j]), copies, reps)
        rec("fake_quant_bf16_%s_%s" % (fmt, tag), us, 4.0)
    return out, copies


def sweep_f32(n: int, reps: int):
    """The FP32 entry points at one size (workload 1's element type)."""
    x = torch.from_numpy(inputs.weight_f32_normal(n // 4096, 4096, seed=0)).cuda()
    copies = 6
    xs = [x.clone() for _ in range(copies)]
    u8 = dict(dtype=torch.uint8, device="cuda")
    cs = [(torch.empty(n, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
    ys = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(copies)]
    out = {}
    for fmt in ("int8", "e4m3"):
        us = _time(lambda j: mxq.quantize(xs[j], fmt, BLOCK, *cs[j]), copies, reps)
        out["quantize_f32_" + fmt] = (us, (4 + 1 + 1 / BLOCK) * n / us / 1e3)
        us = _time(lambda j: mxq.dequantize(*cs[j], n, fmt, BLOCK, dst=ys[j]), copies, reps)
        out["dequantize_%s_f32" % fmt] = (us, (1 + 1 / BLOCK + 4) * n / us / 1e3)
        us = _time(lambda j: mxq.fake_quant(xs[j], fmt, BLOCK, mxq.FQ_DIRECT, dst=ys[j]), copies, reps)
        out["fake_quant_f32_" + fmt] = (us, 8.0 * n / us / 1e3)
    # the anchors reconstructed to BF16 (the 8-bit line of the algorithmic-bytes table)
    yb = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(copies)]
    for fmt in ("int8", "e4m3"):
        us = _time(lambda j: mxq.dequantize(*cs[j], n, fmt, BLOCK, dst=yb[j]), copies, reps)
        out["dequantize_%s_bf16" % fmt] = (us, (1 + 1 / BLOCK + 2) * n / us / 1e3)
    return out


def all_formats(n: int, reps: int = 20):
    """Every element format of the paper (MXINT2..8, MXFP4..8) at one size: Slice-and-Scale from the
    anchor, direct quantization, reconstruction and the fused fake-quant through the anchor."""
    bits = {"int8": 8, "int7": 7, "int6": 6, "int5": 5, "int4": 4, "int3": 3, "int2": 2,
            "e4m3": 8, "e3m3": 7, "e3m2": 6, "e2m3": 6, "e2m2": 5, "e2m1": 4}
    g = torch.Generator(device="cuda").manual_seed(1)
    copies = 4
    u8 = dict(dtype=torch.uint8, device="cuda")
    codes = [torch.randint(0, 127, (n,), generator=g, **u8) for _ in range(copies)]           # no E4M3 NaN codes
    scales = [torch.randint(100, 140, (n // BLOCK,), generator=g, **u8) for _ in range(copies)]
    x = [torch.randn(n, device="cuda", generator=g).to(torch.bfloat16) for _ in range(copies)]
    y = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(copies)]
    out = {}
    for src, dsts in (("int8", ("int7", "int6", "int5", "int4", "int3", "int2")),
                      ("e4m3", ("e3m3", "e3m2", "e2m3", "e2m2", "e2m1"))):
        for d in dsts:
            b = bits[d]
            oc = [torch.empty(n * b // 8, **u8) for _ in range(copies)]
            os_ = [torch.empty(n // BLOCK, **u8) for _ in range(copies)]
            row = {}
            us = _time(lambda j: mxq.slice_scale(codes[j], scales[j], n, src, d, BLOCK, oc[j], os_[j]), copies, reps)
            row["slice_scale_from_anchor"] = (us, n * (1 + b / 8 + 2 / BLOCK) / us / 1e3)
            us = _time(lambda j: mxq.quantize(x[j], d, BLOCK, oc[j], os_[j]), copies, reps)
            row["quantize_bf16"] = (us, n * (2 + b / 8 + 1 / BLOCK) / us / 1e3)
            us = _time(lambda j: mxq.dequantize(oc[j], os_[j], n, d, BLOCK, dst=y[j]), copies, reps)
            row["dequantize_bf16"] = (us, n * (2 + b / 8 + 1 / BLOCK) / us / 1e3)
            us = _time(lambda j: mxq.fake_quant(x[j], d, BLOCK, mxq.FQ_VIA_ANCHOR, dst=y[j]), copies, reps)
            row["fake_quant_bf16_via_anchor"] = (us, n * 4.0 / us / 1e3)
            out[d] = row
            del oc, os_
    return out


def tiled_scales(rows: int = 8192, cols: int = 8192, reps: int = 50):
    """Scale bytes in the tiled order of a block-scaled matmul: the producing kernel writing them
    itself (quantize_tiled, slice_scale_tiled) against the plain kernel followed by tile_scales."""
    n = rows * cols
    g = torch.Generator(device="cuda").manual_seed(2)
    copies = 4
    u8 = dict(dtype=torch.uint8, device="cuda")
    x = [(torch.randn(rows, cols, device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(copies)]
    anchor = [mxq.quantize(x[j], "e4m3", BLOCK) for j in range(copies)]
    oc = [torch.empty(n, **u8) for _ in range(copies)]
    plain = [torch.empty(n // BLOCK, **u8) for _ in range(copies)]
    tiled = [torch.empty(mxq.tiled_scales_bytes(rows, cols // BLOCK), **u8) for _ in range(copies)]
    out = {}
    for fmt in ("e4m3", "e2m1"):
        out["quantize_bf16_" + fmt] = {
            "plain_us": _time(lambda j: mxq.quantize(x[j], fmt, BLOCK, oc[j], plain[j]), copies, reps),
            "plain_then_tile_us": _time(lambda j: (mxq.quantize(x[j], fmt, BLOCK, oc[j], plain[j]),
                                                   mxq.tile_scales(plain[j], rows, cols // BLOCK, tiled[j])), copies, reps),
            "fused_us": _time(lambda j: mxq.quantize_tiled(x[j], fmt, BLOCK, oc[j], tiled[j]), copies, reps)}
    for dst in ("e2m3", "e2m1"):
        out["slice_scale_e4m3_" + dst] = {
            "plain_us": _time(lambda j: mxq.slice_scale(*anchor[j], n, "e4m3", dst, BLOCK, oc[j], plain[j]), copies, reps),
            "plain_then_tile_us": _time(lambda j: (mxq.slice_scale(*anchor[j], n, "e4m3", dst, BLOCK, oc[j], plain[j]),
                                                   mxq.tile_scales(plain[j], rows, cols // BLOCK, tiled[j])), copies, reps),
            "fused_us": _time(lambda j: mxq.slice_scale_tiled(*anchor[j], rows, cols, "e4m3", dst, BLOCK, oc[j], tiled[j]),
                              copies, reps)}
    return {k: {a: round(b, 2) for a, b in v.items()} for k, v in out.items()}


def whole_model(reps: int = 5):
    """Anchor -> target for the 224 tensors of the 8B Llama-shaped set, one batched launch per target.
    Anchors hold seeded random codes (the conversion's speed does not depend on the values)."""
    shapes = inputs.llama8b_shapes()
    total = sum(r * c for *_, r, c in shapes)
    g = torch.Generator(device="cuda").manual_seed(3)
    out = {}
    for anchor, dsts in (("int8", (("int6", 6), ("int4", 4))), ("e4m3", (("e2m3", 6), ("e2m1", 4)))):
        codes = torch.randint(0, 127, (total,), dtype=torch.uint8, device="cuda", generator=g)   # no E4M3 NaN codes
        scales = torch.randint(100, 140, (total // BLOCK,), dtype=torch.uint8, device="cuda", generator=g)
        for dst, b in dsts:
            oc = torch.empty(total * b // 8, dtype=torch.uint8, device="cuda")
            os_ = torch.empty(total // BLOCK, dtype=torch.uint8, device="cuda")
            items, off = [], 0
            for *_, r, c in shapes:
                n = r * c
                items.append((codes[off:off + n], scales[off // BLOCK:(off + n) // BLOCK], n,
                              oc[off * b // 8:(off + n) * b // 8], os_[off // BLOCK:(off + n) // BLOCK]))
                off += n
            table = mxq.make_items(items)
            us = _time(lambda j: mxq.slice_scale_batched(table, anchor, dst, BLOCK), 1, reps)
            per = _time(lambda j: [mxq.slice_scale(c_, s_, n_, anchor, dst, BLOCK, oc_, os2) for c_, s_, n_, oc_, os2 in items], 1, reps)
            bytes_ = total * (1 + b / 8 + 2 / BLOCK)
            out["model_%s_%s" % (anchor, dst)] = {"batched_ms": us / 1e3, "batched_gbs": bytes_ / us / 1e3,
                                                  "per_tensor_launches_ms": per / 1e3, "per_tensor_gbs": bytes_ / per / 1e3,
                                                  "elements": total, "tensors": len(items)}
            if anchor == "e4m3":
                # the same conversion with every tensor's scales written in the matmul's tiled order
                t_items, off = [], 0
                tiled = torch.empty(total // BLOCK, dtype=torch.uint8, device="cuda")   # every shape covers whole tiles
                for *_, r, c in shapes:
                    n = r * c
                    t_items.append((codes[off:off + n], scales[off // BLOCK:(off + n) // BLOCK], r, c,
                                    oc[off * b // 8:(off + n) * b // 8], tiled[off // BLOCK:(off + n) // BLOCK]))
                    off += n
                t_table = mxq.make_tiled_items(t_items)
                tus = _time(lambda j: mxq.slice_scale_tiled_batched(t_table, anchor, dst, BLOCK), 1, reps)
                out["model_%s_%s" % (anchor, dst)].update({"tiled_batched_ms": tus / 1e3, "tiled_batched_gbs": bytes_ / tus / 1e3})
                del t_table, t_items, tiled
            del oc, os_, table, items
        del codes, scales
    # the QAT side of the same weight set: the fused fake-quant of all 224 BF16 weights (Eq. 6)
    w = torch.randn(total, device="cuda", generator=g, dtype=torch.float32).mul_(0.02).to(torch.bfloat16)
    y = torch.empty_like(w)
    pairs, off = [], 0
    for *_, r, c in shapes:
        pairs.append((w[off:off + r * c], y[off:off + r * c]))
        off += r * c
    table = mxq.make_fq_items(pairs)
    for fmt, mode, tag in (("e2m3", mxq.FQ_VIA_ANCHOR, "via_anchor"), ("int4", mxq.FQ_VIA_ANCHOR, "via_anchor")):
        us = _time(lambda j: mxq.fake_quant_batched(table, fmt, BLOCK, mode), 1, reps)
        per = _time(lambda j: [mxq.fake_quant(a, fmt, BLOCK, mode, dst=b) for a, b in pairs], 1, reps)
        out["model_fake_quant_%s_%s" % (fmt, tag)] = {"batched_ms": us / 1e3, "batched_gbs": 4.0 * total / us / 1e3,
                                                      "per_tensor_launches_ms": per / 1e3, "per_tensor_gbs": 4.0 * total / per / 1e3,
                                                      "elements": total, "tensors": len(pairs)}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--min-log2", type=int, default=16)
    ap.add_argument("--max-log2", type=int, default=31)
    ap.add_argument("--model", action="store_true")
    ap.add_argument("--all-formats", action="store_true", help="every element format of the paper at 2^26 elements")
    ap.add_argument("--tiled", action="store_true", help="tiled scale order at 8192 x 8192: fused against two passes")
    ap.add_argument("--warm", action="store_true",
                    help="reuse one buffer set for every launch (L2-resident figures for sizes that fit the 126 MB L2; "
                         "the default rotates over enough copies to be cold)")
    ap.add_argument("--json", default=None)
    ap.add_argument("--graph", action="store_true",
                    help="capture each timed loop in a CUDA graph and time its replay: the figures then exclude the "
                         "host's cost of enqueuing a launch (about 8 us through this binding)")
    args = ap.parse_args()
    global GRAPH, WARM
    GRAPH = args.graph
    WARM = args.warm
    mxq.load_library()
    peak, kind = _peak()
    base = torch.from_numpy(inputs.flat_bf16_normal(1 << 27, seed=5).view(np.int16)).cuda().view(torch.bfloat16)
    result = {"peak_gbs": peak, "peak_kind": kind, "graph": GRAPH, "warm": WARM, "sizes": {}, "f32": {}, "model": {}}
    for k in range(args.min_log2, args.max_log2 + 1):
        n = 1 << k
        reps = 200 if k <= 22 else (50 if k <= 27 else 10)
        ops, copies = sweep_size(n, base, reps)
        result["sizes"][k] = {name: {"us": round(us, 3), "gbs": round(g, 1)} for name, (us, g) in ops.items()}
        print("2^%d elements (%d buffer copies)" % (k, copies))
        for name, (us, g) in ops.items():
            print("  %-36s %10.2f us %8.1f GB/s  %5.1f %% of %s peak  %5.1f %% of 8000" % (name, us, g, 100 * g / peak, kind, g / 80))
        torch.cuda.empty_cache()
    f32 = sweep_f32(1 << 26, 50)
    result["f32"] = {name: {"us": round(us, 3), "gbs": round(g, 1)} for name, (us, g) in f32.items()}
    print("FP32 entry points and anchor reconstruction, 2^26 elements")
    for name, (us, g) in f32.items():
        print("  %-36s %10.2f us %8.1f GB/s  %5.1f %% of %s peak" % (name, us, g, 100 * g / peak, kind))
    if args.all_formats:
        fm = all_formats(1 << 26)
        result["formats"] = {f: {op: {"us": round(us, 3), "gbs": round(g, 1)} for op, (us, g) in row.items()}
                             for f, row in fm.items()}
        print("all formats, 2^26 elements: GB/s (us)")
        for f, row in fm.items():
            print("  %-5s " % f + "  ".join("%s %6.0f (%5.1f)" % (op, g, us) for op, (us, g) in row.items()))
    if args.tiled:
        result["tiled"] = tiled_scales()
        print("scales in the tiled order, BF16 8192 x 8192: us per call")
        for name, r in result["tiled"].items():
            print("  %-24s plain %6.2f | plain then tile_scales %6.2f | fused %6.2f" %
                  (name, r["plain_us"], r["plain_then_tile_us"], r["fused_us"]))
    if args.model:
        result["model"] = whole_model()
        for name, r in result["model"].items():
            if "tiled_batched_ms" in r:
                print("  %-20s batched, scales in the tiled order %.3f ms %7.1f GB/s" % (name, r["tiled_batched_ms"], r["tiled_batched_gbs"]))
            print("  %-20s batched %.3f ms %7.1f GB/s | %d separate launches %.3f ms %7.1f GB/s" %
                  (name, r["batched_ms"], r["batched_gbs"], r["tensors"], r["per_tensor_launches_ms"], r["per_tensor_gbs"]))
    if args.json:
        json.dump(result, open(args.json, "w"), indent=1)


if __name__ == "__main__":
    main()
