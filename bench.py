#!/usr/bin/env python
"""Benchmark of the MX (re)quantization hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mxq|reference]

A *step* is one pass of the whole hot path over one tensor of the headline workload (a
BF16 8192 x 8192 weight matrix, Student-t with outliers): quantize to the MXFP8 (E4M3) and
MXINT8 anchors, Slice-and-Scale to MXFP6 (E2M3) / MXFP4 (E2M1) / MXINT6 / MXINT4, the same
conversion through the batched entry point, both MXFP targets from one read of the anchor, reconstruction to BF16, the fused fake-quant
forward through the anchor and its straight-through backward.  Consumers read what the
*previous* step produced (four buffer sets, each with its own copy of the input), so no kernel finds its input in L2.

Prints ONE JSON line on stdout: whole-step algorithmic GB/s (`value`), the end-to-end figure
with host buffers (`e2e`), the roofline record of the dominant kernel, per-kernel figures,
the CPU oracle timed on a bounded sample (`cpu_baseline`) and the clocks seen under load.
`--impl reference` times the CPU oracle alone.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_00529_b200 import inputs  # noqa: E402  (no quantization arithmetic in there)

BLOCK = 32
WORKLOAD = "bf16_8192x8192_student_t_outliers"
ROWS = COLS = 8192
SCALE_B = 1.0 / BLOCK                       # scale bytes per element


def code_b(bits: int) -> float:
    return bits / 8.0


# name -> algorithmic bytes per element (read + write), the numerators of every GB/s below
OP_BYTES = {
    "quantize_bf16_e4m3": 2 + code_b(8) + SCALE_B,
    "quantize_bf16_int8": 2 + code_b(8) + SCALE_B,
    "ss_e4m3_e2m3": code_b(8) + SCALE_B + code_b(6) + SCALE_B,
    "ss_e4m3_e2m1": code_b(8) + SCALE_B + code_b(4) + SCALE_B,
    "ss_int8_int6": code_b(8) + SCALE_B + code_b(6) + SCALE_B,
    "ss_int8_int4": code_b(8) + SCALE_B + code_b(4) + SCALE_B,
    "ss_batched_e4m3_e2m1": code_b(8) + SCALE_B + code_b(4) + SCALE_B,
    "ss_multi_e4m3_e2m3_e2m1": code_b(8) + SCALE_B + code_b(6) + SCALE_B + code_b(4) + SCALE_B,
    "dequantize_e2m1_bf16": code_b(4) + SCALE_B + 2,
    "dequantize_int4_bf16": code_b(4) + SCALE_B + 2,
    "fake_quant_bf16_via_anchor": 4.0,
    "fake_quant_bwd_bf16": 4.0,
}
STEP_BYTES_PER_ELEM = sum(OP_BYTES.values())


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised under
# profiles/ (same workload, same launch configuration).  Valid only for the kernel sources the
# capture was taken from: when their digest differs the bench reports traffic = null.
NCU_TRAFFIC = {
    "fake_quant_bf16_via_anchor": 218676992,
    "fake_quant_bwd_bf16": 213681024,
}   # profiles/fake_quant_and_copy_kernels_bf16_8192x8192_full.md
NCU_TRAFFIC_SOURCES = "14104d515423b57f"


def kernel_sources_digest() -> str:
    """sha256 over the CUDA sources of the library (file names and contents, sorted)."""
    import hashlib
    d = os.path.join(ROOT, "paper_2604_00529_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(d)):
        if name.endswith((".cu", ".cuh", ".h")):
            h.update(name.encode())
            h.update(open(os.path.join(d, name), "rb").read())
    return h.hexdigest()[:16]


def peaks():
    """Measured HBM peak of this machine (generated file), else the documented fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi every 200 ms while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------------------------

class HotPath:
    """Device buffers and the op list of one step.  NSETS buffer sets (each with its own copy of
    the input tensor): set j is written by the producers of step j (mod NSETS) and read by the
    consumers of the following step, so a buffer is touched again only after about NSETS x 0.9 GB
    of other traffic has gone through the 126 MB L2."""

    NSETS = 4

    def __init__(self, x_host_bits: np.ndarray, device, nsets: int = 4):
        import torch
        self.NSETS = nsets
        import paper_2604_00529_b200 as mxq
        self.torch, self.mxq = torch, mxq
        self.n = n = int(x_host_bits.size)
        x0 = torch.from_numpy(x_host_bits.view(np.int16)).to(device).view(torch.bfloat16)
        self.xs = [x0] + [x0.clone() for _ in range(self.NSETS - 1)]
        u8 = dict(dtype=torch.uint8, device=device)
        nb = n // BLOCK
        self.sets = []
        for _ in range(self.NSETS):
            s = {}
            for name, bits in (("e4m3", 8), ("int8", 8), ("e2m3", 6), ("e2m1", 4), ("int6", 6), ("int4", 4),
                               ("e2m1_b", 4), ("e2m3_m", 6), ("e2m1_m", 4)):
                s[name] = (torch.empty(n * bits // 8, **u8), torch.empty(nb, **u8))
            s["deq_e2m1"] = torch.empty(n, dtype=torch.bfloat16, device=device)
            s["deq_int4"] = torch.empty(n, dtype=torch.bfloat16, device=device)
            s["fq"] = torch.empty(n, dtype=torch.bfloat16, device=device)
            s["grad"] = torch.empty(n, dtype=torch.bfloat16, device=device)
            self.sets.append(s)
        self.parts = 8                          # the batched entry point sees the tensor as 8 row bands
        self.op_names = list(OP_BYTES)
        # item lists of the batched conversion: read set j-1, write set j
        self.items = [mxq.make_items(self.batched_items(self.sets[(j - 1) % self.NSETS]["e4m3"], self.sets[j]["e2m1_b"]))
                      for j in range(self.NSETS)]

    def batched_items(self, src, dst):
        n, p = self.n, self.parts
        m = n // p
        items = []
        for k in range(p):
            items.append((src[0][k * m:(k + 1) * m], src[1][k * m // BLOCK:(k + 1) * m // BLOCK], m,
                          dst[0][k * m // 2:(k + 1) * m // 2], dst[1][k * m // BLOCK:(k + 1) * m // BLOCK]))
        return items

    def step(self, i: int, mark=None, only=None):
        """Runs the ops of step i (or just op `only`); `mark(k)` is called before op k and after
        the last one."""
        mxq, n = self.mxq, self.n
        j = i % self.NSETS
        cur, prev, x = self.sets[j], self.sets[(j - 1) % self.NSETS], self.xs[j]
        ops = [
            lambda: mxq.quantize(x, "e4m3", BLOCK, *cur["e4m3"]),
            lambda: mxq.quantize(x, "int8", BLOCK, *cur["int8"]),
            lambda: mxq.slice_scale(*prev["e4m3"], n, "e4m3", "e2m3", BLOCK, *cur["e2m3"]),
            lambda: mxq.slice_scale(*prev["e4m3"], n, "e4m3", "e2m1", BLOCK, *cur["e2m1"]),
            lambda: mxq.slice_scale(*prev["int8"], n, "int8", "int6", BLOCK, *cur["int6"]),
            lambda: mxq.slice_scale(*prev["int8"], n, "int8", "int4", BLOCK, *cur["int4"]),
            lambda: mxq.slice_scale_batched(self.items[j], "e4m3", "e2m1", BLOCK),
            lambda: mxq.slice_scale_multi(*prev["e4m3"], n, "e4m3", ("e2m3", "e2m1"), BLOCK,
                                          (cur["e2m3_m"], cur["e2m1_m"])),
            lambda: mxq.dequantize(*prev["e2m1"], n, "e2m1", BLOCK, dst=cur["deq_e2m1"]),
            lambda: mxq.dequantize(*prev["int4"], n, "int4", BLOCK, dst=cur["deq_int4"]),
            lambda: mxq.fake_quant(x, "e2m3", BLOCK, mxq.FQ_VIA_ANCHOR, dst=cur["fq"]),
            lambda: mxq.fake_quant_bwd(prev["fq"], cur["grad"]),
        ]
        if only is not None:
            ops[only]()
            return 1
        for k, op in enumerate(ops):
            if mark:
                mark(k)
            op()
        if mark:
            mark(len(ops))
        return len(ops)


def run_cuda(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    import paper_2604_00529_b200 as mxq
    mxq.load_library()

    # weak scaling: every rank converts its own tensor of the workload's shape (blocks are
    # independent, so ranks exchange nothing); seed 1 on rank 0 is the documented workload
    x_bits = inputs.weight_bf16_student_t(ROWS, COLS, seed=1 + rank)
    hp = HotPath(x_bits, device, args.buffer_sets)
    n = hp.n
    nops = len(hp.op_names)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        hp.step(i)
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # keep the GPU under load long enough for the sampler to see it (not part of the timing)
    t_end = time.time() + 0.7
    i = args.warmup
    while time.time() < t_end:
        hp.step(i)
        i += 1
        torch.cuda.synchronize()
    barrier()

    stream = torch.cuda.current_stream()
    base = i                                # continue the rotation of buffer sets where the warm-up stopped
    # timed region 1 -- the headline: K steps back to back between two events, nothing else in the stream
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record(stream)
    for s in range(args.steps):
        hp.step(base + s)
    t1.record(stream)
    barrier()
    total_ms = t0.elapsed_time(t1)
    # timed region 2 -- the same K steps with an event between consecutive launches, for the
    # per-kernel durations (an event costs a few microseconds of stream time, so these K steps are
    # slower than region 1 and are not what `value` is computed from)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(nops + 1)] for _ in range(args.steps)]
    for s in range(args.steps):
        ev = events[s]
        hp.step(base + s, mark=lambda k, ev=ev: ev[k].record(stream))
    barrier()
    op_ms = [sum(events[s][k].elapsed_time(events[s][k + 1]) for s in range(args.steps)) / args.steps
             for k in range(nops)]
    # timed region 3 -- every op on its own: K launches of the same kernel back to back between two
    # events, rotating over the buffer sets; this is the average launch duration the roofline uses
    iso_ms, host_ms = [], []
    for k in range(nops):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for s in range(3):
            hp.step(base + s, only=k)
        torch.cuda.synchronize()
        h0 = time.perf_counter()
        a.record(stream)
        for s in range(args.steps):
            hp.step(base + s, only=k)
        b.record(stream)
        host_ms.append((time.perf_counter() - h0) * 1e3 / args.steps)   # host time to enqueue one launch
        torch.cuda.synchronize()
        iso_ms.append(a.elapsed_time(b) / args.steps)
    if world > 1:
        t = torch.tensor([total_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = total_ms / args.steps

    # end to end through the public API with host buffers: every step copies its input from pinned host
    # memory, runs, and copies the converted tensors (the four lower-format code + scale sets) back to
    # pinned host memory.  Three streams (copy in, compute, copy out) let the copies of neighbouring
    # steps overlap the kernels; events keep a buffer set from being rewritten before its last reader
    # has finished.  The timed region runs from the first host-to-device copy to the last device-to-host one.
    e2e_steps = max(8, args.steps // 4)
    host_in = torch.from_numpy(x_bits.view(np.int16)).pin_memory()
    outs = ["e2m3", "e2m1", "int6", "int4"]
    host_out = {k: (torch.empty_like(hp.sets[0][k][0], device="cpu").pin_memory(),
                    torch.empty_like(hp.sets[0][k][1], device="cpu").pin_memory()) for k in outs}
    h2d = host_in.numel() * 2
    d2h = sum(a.numel() + b.numel() for a, b in host_out.values())
    s_in, s_cmp, s_out = torch.cuda.Stream(device), torch.cuda.Stream(device), torch.cuda.Stream(device)

    def e2e_pipeline(first, count):
        ev_in = [torch.cuda.Event() for _ in range(count)]
        ev_cmp = [torch.cuda.Event() for _ in range(count)]
        ev_out = [torch.cuda.Event() for _ in range(count)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s_in)
        for k in range(count):
            i = first + k
            j = i % hp.NSETS
            with torch.cuda.stream(s_in):
                if k >= hp.NSETS:
                    s_in.wait_event(ev_cmp[k - hp.NSETS])        # the step that last read this input copy
                hp.xs[j].view(torch.int16).copy_(host_in, non_blocking=True)
                ev_in[k].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in[k])
                if k >= hp.NSETS:
                    s_cmp.wait_event(ev_out[k - hp.NSETS])       # this set's previous results are on the host
                hp.step(i)
                ev_cmp[k].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[k])
                cur = hp.sets[j]
                for name in outs:
                    host_out[name][0].copy_(cur[name][0], non_blocking=True)
                    host_out[name][1].copy_(cur[name][1], non_blocking=True)
                ev_out[k].record(s_out)
        e1.record(s_out)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / count

    barrier()
    e2e_pipeline(base, hp.NSETS)                                 # untimed: page in the pinned buffers
    barrier()
    e2e_ms = e2e_pipeline(base, e2e_steps)
    barrier()
    if world > 1:
        t = torch.tensor([e2e_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = peaks()
    step_bytes = STEP_BYTES_PER_ELEM * n
    value = step_bytes * world / (ms_per_step * 1e-3) / 1e9
    per_op = {}
    for name, ms, ms_in_step, ms_host in zip(hp.op_names, iso_ms, op_ms, host_ms):
        gbs = OP_BYTES[name] * n / (ms * 1e-3) / 1e9
        per_op[name] = {"ms": round(ms, 5), "ms_in_step_with_events": round(ms_in_step, 5),
                        "host_enqueue_ms": round(ms_host, 5), "gbs": round(gbs, 1),
                        "gelem_s": round(n / (ms * 1e-3) / 1e9, 2),
                        "frac_of_%s_peak" % peak_kind: round(gbs / peak, 4), "frac_of_8000": round(gbs / 8000.0, 4)}
    top = max(range(nops), key=lambda k: iso_ms[k])
    top_name = hp.op_names[top]
    top_gbs = OP_BYTES[top_name] * n / (iso_ms[top] * 1e-3) / 1e9
    traffic = NCU_TRAFFIC.get(top_name) if kernel_sources_digest() == NCU_TRAFFIC_SOURCES else None

    # the oracle is timed beside the one-GPU run only: at N > 1 every rank's GPU would be held meanwhile
    cpu = cpu_baseline(x_bits) if world == 1 else None
    line = {
        "metric": "mx_requant_hot_path_hbm_gbs", "value": round(value, 1), "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "impl": "mxq",
        "config": {"workload": WORKLOAD, "elements_per_gpu": n, "block": BLOCK, "ops_per_step": hp.op_names,
                   "bytes_per_step_per_gpu": int(step_bytes), "l2": "inputs larger than L2; consumers read the "
                   "previous step's buffers", "timing": "value: K steps between two events; kernels/roofline: K "
                   "launches of one kernel back to back between two events, rotating over 4 buffer sets; "
                   "ms_in_step_with_events: K steps with an event between launches", "gelem_per_s": round(n * nops * world / (ms_per_step * 1e-3) / 1e9, 2)},
        "e2e": {"value": round(step_bytes * world / (e2e_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                "ms_per_step": round(e2e_ms, 4)},
        "gpu_launches": nops * args.steps,
        "roofline": {"bound": "hbm", "kernel": top_name, "achieved": round(top_gbs, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(top_gbs / peak, 4), "peak_kind": peak_kind, "traffic": traffic,
                     "bytes_per_launch": int(OP_BYTES[top_name] * n)},
        "kernels": per_op,
        "cpu_baseline": cpu,
        "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------
# the CPU oracle arm (reported baseline; also `--impl reference`)
# ----------------------------------------------------------------------------------------------

def oracle_step(x_bits: np.ndarray):
    """The same op list on the CPU oracle (single thread, as it stands)."""
    from oracle import mxq_oracle as orc
    ca, sa = orc.quantize(x_bits, "e4m3", BLOCK)
    ci, si = orc.quantize(x_bits, "int8", BLOCK)
    orc.slice_scale(ca, sa, "e4m3", "e2m3", BLOCK)
    c4, s4 = orc.slice_scale(ca, sa, "e4m3", "e2m1", BLOCK)
    orc.slice_scale(ci, si, "int8", "int6", BLOCK)
    c4i, s4i = orc.slice_scale(ci, si, "int8", "int4", BLOCK)
    orc.slice_scale(ca, sa, "e4m3", "e2m1", BLOCK)
    orc.slice_scale(ca, sa, "e4m3", "e2m3", BLOCK)           # the two-target conversion: both targets again
    orc.slice_scale(ca, sa, "e4m3", "e2m1", BLOCK)
    orc.dequantize(c4, s4, "e2m1", BLOCK, orc.BF16)
    orc.dequantize(c4i, s4i, "int4", BLOCK, orc.BF16)
    g = orc.fake_quant(x_bits, "e2m3", BLOCK, orc.FQ_VIA_ANCHOR)
    orc.fake_quant_bwd(g)


def cpu_baseline(x_bits: np.ndarray, sample_elems: int = 1 << 24):
    """Oracle throughput on the first `sample_elems` elements of the workload, one thread."""
    from oracle import mxq_oracle as orc
    orc.lib()
    sample = np.ascontiguousarray(x_bits[:sample_elems])
    t0 = time.perf_counter()
    oracle_step(sample)
    dt = time.perf_counter() - t0
    gbs = STEP_BYTES_PER_ELEM * sample.size / dt / 1e9
    return {"value": round(gbs, 4), "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": "first %d elements of the workload tensor, all %d ops of the step, %.1f s" %
                      (sample.size, len(OP_BYTES), dt),
            "host_cores_available": len(os.sched_getaffinity(0))}


def run_reference(args):
    """`--impl reference`: the CPU oracle timed on the machine's host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import mxq_oracle as orc
    orc.lib()
    sample_elems = 1 << 20
    x_bits = inputs.weight_bf16_student_t(ROWS, COLS, seed=1)[:sample_elems].copy()
    for _ in range(args.warmup):
        oracle_step(x_bits)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(x_bits)
    dt = (time.perf_counter() - t0) / args.steps
    gbs = STEP_BYTES_PER_ELEM * sample_elems / dt / 1e9
    sample = "each step = the first %d elements of the workload tensor through all %d ops" % (sample_elems,
                                                                                              len(OP_BYTES))
    line = {
        "metric": "mx_requant_hot_path_hbm_gbs", "value": round(gbs, 4), "unit": "GB/s", "impl": "reference",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "block": BLOCK, "ops_per_step": list(OP_BYTES), "sample": sample},
        "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="mxq", choices=["mxq", "reference"])
    ap.add_argument("--buffer-sets", type=int, default=4,
                    help="rotating buffer sets (>= 2); profiling captures use 2 to hold less device memory")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.buffer_sets = max(args.buffer_sets, 2)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
