#!/usr/bin/env python
"""Benchmark of the MX (re)quantization hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mxq|reference] [--workloads w1,w2,w3,w4,w5]

One invocation times all five workloads of the method and prints ONE JSON line on stdout.

Headline (`value`, `config.workload`): the whole-model workload -- the 224 BF16 linear weights of an 8B
Llama-shaped decoder (6.98 G elements).  A *step* is one pass of the whole hot path over that weight
set, ten launches that each cover all 224 tensors: quantize to the MXINT8 and the MXFP8 (E4M3) anchor (Eq. 1-3), Slice-and-Scale both
anchors to MXINT6 / MXINT4 and MXFP6 (E2M3) / MXFP4 (E2M1) (Eq. 4-5,
the on-the-fly conversion of Sec. 3.5), reconstruct the two 4-bit sets to BF16, run the fused fake-quant
of all weights through the anchor (Eq. 6) and its straight-through backward.  180 GB of algorithmic
traffic per step, every buffer far larger than L2.  K steps run back to back between two CUDA events;
events between the steps and between the op groups give the spread and the per-kernel durations.

`workloads` in the line carries the other four (and the per-target conversion times of the headline
one): w1 the FP32 4096 x 4096 matrix (quantize -> MXINT8 -> MXINT4 -> reconstruct), w2 the BF16
8192 x 8192 Student-t matrix through a 12-launch step, w4 the fake-quant of a [8, 4096, 4096]
activation tensor with the format sampled by seed, w5 the size sweep 2^16 ... 2^31.  Every figure there
is the median of 15 timed regions with its minimum and maximum, in microseconds per launch, with the SM
clock seen meanwhile; small tensors rotate over enough buffer copies to stay out of L2.

`e2e` is the headline step with the weights copied from pinned host memory and the four converted
sets copied back inside the timed region.  `cpu_baseline` is the CPU oracle on a bounded sample (one
thread, and split over all host cores).  `--impl reference` times the CPU oracle alone.
`--gpus N` (N > 1, not under torchrun) starts N ranks, one per device; every rank converts its own
replica of the workload (blocks are independent: no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
SCALE_B = 1.0 / BLOCK                       # scale bytes per element
BITS = {"int8": 8, "int6": 6, "int4": 4, "e4m3": 8, "e3m2": 6, "e2m3": 6, "e2m1": 4}
METRIC = "mx_requant_hot_path_hbm_gbs"
HEADLINE = "llama8b_linear_weights_bf16_224_tensors"
REGIONS = 15                                # timed regions per figure of the `workloads` record
L2_BYTES = 126 << 20


# algorithmic bytes per element (read + write): the numerators of every GB/s below
def b_quantize(src_bytes: int, fmt: str) -> float:
    return src_bytes + BITS[fmt] / 8 + SCALE_B


def b_slice_scale(dst: str) -> float:
    return 1 + SCALE_B + BITS[dst] / 8 + SCALE_B


def b_dequantize(fmt: str, dst_bytes: int) -> float:
    return BITS[fmt] / 8 + SCALE_B + dst_bytes


# the op groups of the headline step, in order, with their algorithmic bytes per element
STEP_OPS = [
    ("quantize_batched_bf16_int8", b_quantize(2, "int8")),
    ("quantize_batched_bf16_e4m3", b_quantize(2, "e4m3")),
    ("ss_batched_int8_int6", b_slice_scale("int6")),
    ("ss_batched_int8_int4", b_slice_scale("int4")),
    ("ss_batched_e4m3_e2m3", b_slice_scale("e2m3")),
    ("ss_batched_e4m3_e2m1", b_slice_scale("e2m1")),
    ("dequantize_batched_int4_bf16", b_dequantize("int4", 2)),
    ("dequantize_batched_e2m1_bf16", b_dequantize("e2m1", 2)),
    ("fake_quant_batched_bf16_e2m3_via_anchor", 4.0),
    ("fake_quant_bwd_bf16", 4.0),
]
STEP_BYTES_PER_ELEM = sum(b for _, b in STEP_OPS)

# the 12-launch step of workload 2 (unchanged between releases, so that its figures stay comparable)
W2_OPS = {
    "quantize_bf16_e4m3": b_quantize(2, "e4m3"),
    "quantize_bf16_int8": b_quantize(2, "int8"),
    "ss_e4m3_e2m3": b_slice_scale("e2m3"),
    "ss_e4m3_e2m1": b_slice_scale("e2m1"),
    "ss_int8_int6": b_slice_scale("int6"),
    "ss_int8_int4": b_slice_scale("int4"),
    "ss_batched_e4m3_e2m1": b_slice_scale("e2m1"),
    "ss_multi_e4m3_e2m3_e2m1": 1 + SCALE_B + BITS["e2m3"] / 8 + SCALE_B + BITS["e2m1"] / 8 + SCALE_B,
    "dequantize_e2m1_bf16": b_dequantize("e2m1", 2),
    "dequantize_int4_bf16": b_dequantize("int4", 2),
    "fake_quant_bf16_via_anchor": 4.0,
    "fake_quant_bwd_bf16": 4.0,
}
W2_STEP_BYTES_PER_ELEM = sum(W2_OPS.values())


def kernel_sources_digest() -> str:
    """sha256 over the CUDA sources of the library (file names and contents, sorted)."""
    import hashlib
    d = os.path.join(ROOT, "paper_2604_00529_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(d)):
        if name.startswith("mxq_") and name.endswith((".cu", ".cuh", ".h")):
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


def ncu_traffic(kernel: str, elements: int):
    """DRAM bytes (read + write) per launch of `kernel` from the ncu capture recorded under profiles/,
    scaled by the elements one launch processes (the capture ran a smaller case of the same kernel;
    the traffic of these streaming kernels grows in proportion).  None when the kernel sources have
    changed since the capture."""
    p = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        rec = json.load(open(p))
    except Exception:
        return None, None
    if rec.get("kernel_sources") != kernel_sources_digest():
        return None, None
    k = rec.get("kernels", {}).get(kernel)
    if not k:
        return None, None
    return int(round(k["dram_bytes_per_element"] * elements)), k.get("dram_pct_of_peak")


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------

class ClockSampler:
    """SM clock and throttle reasons of one GPU, sampled every 10 ms through NVML while the bench runs
    (nvidia-smi every 100 ms where the NVML module is missing).  Samples carry host timestamps, so
    that each timed section can report the clock seen during its own window."""

    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"),
               (0x4, "sw_power_cap"))

    def __init__(self, index: int, uuid: str = None):
        # `index` counts the devices this process sees; NVML counts all of the machine's, so the device
        # is looked up by UUID where torch gives one, else through CUDA_VISIBLE_DEVICES
        self.uuid = uuid
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [v.strip() for v in vis.split(",") if v.strip()]
        if uuid is None and index < len(ids):
            if ids[index].isdigit():
                index = int(ids[index])
            elif ids[index].startswith("GPU-"):
                self.uuid = ids[index]
        self.index = index
        self.samples = []                   # (t, sm_mhz, reasons bitmask)
        self.max_mhz = None
        self.stop_flag = threading.Event()
        self.thread = None
        self.how = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            if self.uuid:
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(self.uuid.encode())
                except TypeError:
                    h = pynvml.nvmlDeviceGetHandleByUUID(self.uuid)
            else:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(pynvml, "nvmlDeviceGetCurrentClocksThrottleReasons")

            def poll():
                while not self.stop_flag.is_set():
                    try:
                        self.samples.append((time.perf_counter(),
                                             float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)),
                                             int(reasons(h))))
                    except Exception:
                        pass
                    time.sleep(0.01)
            self.how = "nvml"
        except Exception:
            q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                 "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
            try:
                proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid or str(self.index), "--query-gpu=" + q,
                                         "--format=csv,noheader,nounits", "-lms", "100"],
                                        stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            except OSError:
                self.how = "unavailable"
                return
            self.proc = proc

            def poll():
                for line in proc.stdout:
                    f = [x.strip() for x in line.split(",")]
                    try:
                        mask = 0
                        for (bit, _), v in zip(self.REASONS, f[2:6]):
                            if v.lower().startswith("active"):
                                mask |= bit
                        self.samples.append((time.perf_counter(), float(f[0]), mask))
                        self.max_mhz = float(f[1])
                    except (ValueError, IndexError):
                        continue
                    if self.stop_flag.is_set():
                        break
            self.how = "nvidia-smi"
        self.thread = threading.Thread(target=poll, daemon=True)
        self.thread.start()

    def stop(self):
        self.stop_flag.set()
        if getattr(self, "proc", None) is not None:
            self.proc.terminate()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def window(self, t0: float, t1: float):
        """Median SM MHz over the samples taken in [t0, t1] (None when there were none)."""
        v = [m for t, m, _ in self.samples if t0 <= t <= t1]
        if v:
            return statistics.median(v)
        if not self.samples:
            return None
        mid = 0.5 * (t0 + t1)                 # a window shorter than the sampling period: the nearest sample
        return min(self.samples, key=lambda s: abs(s[0] - mid))[1]

    def summary(self, t0: float, t1: float):
        w = [(m, r) for t, m, r in self.samples if t0 <= t <= t1]
        if not w:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "samples": 0, "reasons": [self.how or "unavailable"]}
        mask = 0
        for _, r in w:
            mask |= r
        return {"sm_mhz": statistics.median(m for m, _ in w), "sm_min_mhz": min(m for m, _ in w),
                "sm_max_mhz": self.max_mhz, "samples": len(w), "how": self.how,
                "reasons": [name for bit, name in self.REASONS if mask & bit]}


# ----------------------------------------------------------------------------------------------
# timing
# ----------------------------------------------------------------------------------------------

class Bench:
    """CUDA-event timing on the current stream, with the clock seen during each measurement."""

    def __init__(self, torch, sampler, peak, peak_kind):
        self.torch, self.sampler, self.peak, self.peak_kind = torch, sampler, peak, peak_kind
        self.launches = 0

    def regions(self, launch, copies: int, reps: int, warm: int = 3, regions: int = REGIONS):
        """`regions` back-to-back timed regions of `reps` launches each (launch(j) uses buffer copy j);
        returns microseconds per launch: median, min and max over the regions, and the median SM clock."""
        torch = self.torch
        for j in range(warm):
            launch(j % copies)
        torch.cuda.synchronize()
        stream = torch.cuda.current_stream()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(regions + 1)]
        h0 = time.perf_counter()
        ev[0].record(stream)
        k = 0
        for r in range(regions):
            for _ in range(reps):
                launch(k % copies)
                k += 1
            ev[r + 1].record(stream)
        torch.cuda.synchronize()
        h1 = time.perf_counter()
        us = [ev[r].elapsed_time(ev[r + 1]) * 1e3 / reps for r in range(regions)]
        return {"us": statistics.median(us), "us_min": min(us), "us_max": max(us),
                "sm_mhz": self.sampler.window(h0, h1), "regions": regions, "launches_per_region": reps}

    def record(self, t: dict, nbytes: float, elements: int, launches_per_call: int = 1) -> dict:
        """A timing of `regions` turned into the figures the line reports."""
        us = t["us"]
        gbs = nbytes / us / 1e3
        out = {"us": round(us, 3), "us_min": round(t["us_min"], 3), "us_max": round(t["us_max"], 3),
               "gbs": round(gbs, 1), "gelem_s": round(elements / us / 1e3, 2),
               "frac_of_%s_peak" % self.peak_kind: round(gbs / self.peak, 4), "frac_of_8000": round(gbs / 8000.0, 4),
               "sm_mhz": t["sm_mhz"]}
        if t["sm_mhz"]:
            out["us_x_ghz"] = round(us * t["sm_mhz"] / 1e3, 3)      # compares boxes that settle at different clocks
        if launches_per_call != 1:
            out["launches"] = launches_per_call
        return out


def reps_for(us_estimate: float, target_us: float = 1500.0, lo: int = 2, hi: int = 50) -> int:
    """Launches per timed region: enough for about `target_us` of device time."""
    return int(max(lo, min(hi, round(target_us / max(us_estimate, 1e-3)))))


# ----------------------------------------------------------------------------------------------
# workload 2: BF16 8192 x 8192 Student-t matrix, the 12-launch step
# ----------------------------------------------------------------------------------------------

class HotPath:
    """Device buffers and the op list of one step on one tensor.  NSETS buffer sets (each with its own
    copy of the input tensor): set j is written by the producers of step j (mod NSETS) and read by the
    consumers of the following step, so a buffer is touched again only after about NSETS x 0.9 GB of
    other traffic has gone through the 126 MB L2."""

    def __init__(self, x_host_bits: np.ndarray, device, nsets: int = 4):
        import torch
        import paper_2604_00529_b200 as mxq
        self.NSETS = nsets
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
        self.op_names = list(W2_OPS)
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

    def step(self, i: int, only=None):
        """Runs the ops of step i (or just op `only`)."""
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
        for op in ops:
            op()
        return len(ops)


def workload2(bench: Bench, device, seed: int, nsets: int):
    """The 12-launch step on the 8192 x 8192 Student-t matrix: whole steps and every launch on its own."""
    torch = bench.torch
    x_bits = inputs.weight_bf16_student_t(8192, 8192, seed=seed)
    hp = HotPath(x_bits, device, nsets)
    n = hp.n
    for i in range(2 * nsets):
        hp.step(i)
    torch.cuda.synchronize()
    t = bench.regions(lambda j: hp.step(j), copies=4 * nsets, reps=10, warm=nsets)
    out = {"tensor": "bf16_8192x8192_student_t_outliers", "elements": n, "launches_per_step": len(hp.op_names),
           "bytes_per_step": int(W2_STEP_BYTES_PER_ELEM * n),
           "step": bench.record(t, W2_STEP_BYTES_PER_ELEM * n, n * len(hp.op_names)), "kernels": {}}
    bench.launches += len(hp.op_names) * (REGIONS * 10 + nsets)
    for k, name in enumerate(hp.op_names):
        t = bench.regions(lambda j, k=k: hp.step(j, only=k), copies=4 * nsets, reps=10)
        out["kernels"][name] = bench.record(t, W2_OPS[name] * n, n)
        bench.launches += REGIONS * 10 + 3
    del hp
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------------------------
# workload 1: FP32 4096 x 4096 N(0, 0.02): quantize -> MXINT8 -> MXINT4 -> reconstruct
# ----------------------------------------------------------------------------------------------

def workload1(bench: Bench, device):
    torch = bench.torch
    import paper_2604_00529_b200 as mxq
    x0 = torch.from_numpy(inputs.weight_f32_normal(4096, 4096, seed=0)).to(device)
    n = x0.numel()
    copies = 8                                   # 8 x 160 MB of buffers: nothing is found in L2 again
    u8 = dict(dtype=torch.uint8, device=device)
    xs = [x0] + [x0.clone() for _ in range(copies - 1)]
    a = [(torch.empty(n, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
    c4 = [(torch.empty(n // 2, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
    y = [torch.empty(n, dtype=torch.float32, device=device) for _ in range(copies)]
    q = [mxq.prepare_quantize(xs[j], "int8", BLOCK, *a[j]) for j in range(copies)]
    s = [mxq.prepare_slice_scale(*a[j], n, "int8", "int4", BLOCK, *c4[j]) for j in range(copies)]
    d = [mxq.prepare_dequantize(*c4[j], n, "int4", BLOCK, y[j]) for j in range(copies)]
    for j in range(copies):
        q[j](); s[j](); d[j]()
    ops = {"quantize_f32_int8": (q, b_quantize(4, "int8")), "ss_int8_int4": (s, b_slice_scale("int4")),
           "dequantize_int4_f32": (d, b_dequantize("int4", 4))}
    out = {"tensor": "f32_4096x4096_normal_0.02", "elements": n, "buffer_copies": copies, "ops": {}}
    for name, (calls, bpe) in ops.items():
        t = bench.regions(lambda j, calls=calls: calls[j](), copies, reps=50)
        out["ops"][name] = bench.record(t, bpe * n, n)
        bench.launches += REGIONS * 50 + 3
    # the chain as a user runs it: three dependent launches per tensor
    t = bench.regions(lambda j: (q[j](), s[j](), d[j]()), copies, reps=20)
    total = sum(bpe for _, bpe in ops.values())
    out["chain_quantize_ss_dequantize"] = bench.record(t, total * n, 3 * n, launches_per_call=3)
    bench.launches += 3 * (REGIONS * 20 + 3)
    return out


# ----------------------------------------------------------------------------------------------
# workload 4: fake-quant of BF16 activations [8, 4096, 4096], format sampled by seed, + backward
# ----------------------------------------------------------------------------------------------

def workload4(bench: Bench, device):
    torch = bench.torch
    import paper_2604_00529_b200 as mxq
    x0 = torch.from_numpy(inputs.activations_bf16(8, 4096, 4096, seed=4).view(np.int16)).to(device).view(torch.bfloat16)
    n = x0.numel()
    copies = 3                                   # 3 x (268 MB in + 268 MB out): every launch reads cold data
    xs = [x0] + [x0.clone() for _ in range(copies - 1)]
    ys = [torch.empty_like(x0) for _ in range(copies)]
    gs = [torch.empty_like(x0) for _ in range(copies)]
    out = {"tensor": "bf16_8x4096x4096_normal_hot_channels", "elements": n, "buffer_copies": copies, "ops": {}}
    modes = (("direct", mxq.FQ_DIRECT), ("via_anchor", mxq.FQ_VIA_ANCHOR))
    calls = {}
    for fmt in inputs.FQ_FORMATS:
        for tag, mode in modes:
            calls[(fmt, tag)] = [mxq.prepare_fake_quant(xs[j], fmt, BLOCK, mode, ys[j]) for j in range(copies)]
            t = bench.regions(lambda j, c=calls[(fmt, tag)]: c[j](), copies, reps=6)
            out["ops"]["fake_quant_bf16_%s_%s" % (fmt, tag)] = bench.record(t, 4.0 * n, n)
            bench.launches += REGIONS * 6 + 3
    bwd = [mxq.prepare_fake_quant_bwd(ys[j], gs[j]) for j in range(copies)]
    t = bench.regions(lambda j: bwd[j](), copies, reps=6)
    out["ops"]["fake_quant_bwd_bf16"] = bench.record(t, 4.0 * n, n)
    bench.launches += REGIONS * 6 + 3
    # a run of QAT calls: the format of call c is sampled by seed c; forward through the anchor, then backward
    seq = [inputs.fq_format_for_call(c) for c in range(12)]

    def run(j):
        for c, fmt in enumerate(seq):
            calls[(fmt, "via_anchor")][(j + c) % copies]()
            bwd[(j + c) % copies]()
    t = bench.regions(run, copies, reps=1, warm=1)
    rec = bench.record(t, 8.0 * n * len(seq), 2 * n * len(seq), launches_per_call=2 * len(seq))
    rec["formats_by_seed"] = seq
    out["sampled_sequence_fwd_bwd"] = rec
    bench.launches += 2 * len(seq) * (REGIONS + 1)
    return out


# ----------------------------------------------------------------------------------------------
# workload 5: size sweep 2^16 ... 2^31, every anchor-to-lower pair and direct quantization
# ----------------------------------------------------------------------------------------------

def workload5(bench: Bench, device, min_log2: int, max_log2: int):
    torch = bench.torch
    import paper_2604_00529_b200 as mxq
    base_n = 1 << 27
    base = torch.from_numpy(inputs.flat_bf16_normal(base_n, seed=5).view(np.int16)).to(device).view(torch.bfloat16)
    u8 = dict(dtype=torch.uint8, device=device)
    out = {"tensor": "bf16_flat_normal", "input": "2^27 elements drawn on the host (seed 5); larger sizes repeat them",
           "sizes": {}}
    for k in range(min_log2, max_log2 + 1):
        n = 1 << k
        # enough rotating copies that a buffer is not found in L2 again (2 to 512 of them)
        copies = int(min(512, max(2, -(-2 * L2_BYTES // (2 * n)))))
        xs = [base[:n].clone() if n <= base_n else base.repeat(n // base_n) for _ in range(copies)]
        est = max(3.0, 3.0 * n / 6.5e3 / 1e3)                  # microseconds per launch, roughly
        reps = reps_for(est)
        row = {}
        anchors = {}
        for fmt in ("int8", "e4m3", "int6", "int4", "e2m3", "e2m1"):
            cs = [(torch.empty(n * BITS[fmt] // 8, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
            calls = [mxq.prepare_quantize(xs[j], fmt, BLOCK, *cs[j]) for j in range(copies)]
            t = bench.regions(lambda j, c=calls: c[j](), copies, reps)
            row["quantize_bf16_" + fmt] = bench.record(t, b_quantize(2, fmt) * n, n)
            bench.launches += REGIONS * reps + 3
            if fmt in ("int8", "e4m3"):
                anchors[fmt] = cs
            del calls, cs
        for src, dsts in (("int8", ("int6", "int4")), ("e4m3", ("e2m3", "e3m2", "e2m1"))):
            for dst in dsts:
                os_ = [(torch.empty(n * BITS[dst] // 8, **u8), torch.empty(n // BLOCK, **u8)) for _ in range(copies)]
                calls = [mxq.prepare_slice_scale(*anchors[src][j], n, src, dst, BLOCK, *os_[j]) for j in range(copies)]
                t = bench.regions(lambda j, c=calls: c[j](), copies, reps)
                row["ss_%s_%s" % (src, dst)] = bench.record(t, b_slice_scale(dst) * n, n)
                bench.launches += REGIONS * reps + 3
                del calls, os_
        row["buffer_copies"] = copies
        out["sizes"]["2^%d" % k] = row
        del xs, anchors
        torch.cuda.empty_cache()
    del base
    torch.cuda.empty_cache()
    return out


def small_end_abi(device_index: int):
    """The small end of the sweep through the C ABI alone: `mxq_abi_timing` (built with the library)
    calls the entry points in a loop from C and reports, per operation and size, the host's time to
    enqueue a call and the device's time per launch.  Returns its records, or a note when it is missing."""
    exe = os.path.join(ROOT, "paper_2604_00529_b200", "mxq_abi_timing")
    if not os.path.exists(exe):
        return {"unavailable": "mxq_abi_timing is not built (python -m paper_2604_00529_b200.build)"}
    env = dict(os.environ)
    vis = env.get("CUDA_VISIBLE_DEVICES")
    env["CUDA_VISIBLE_DEVICES"] = vis.split(",")[device_index] if vis else str(device_index)
    try:
        out = subprocess.run([exe, "16", "24", "2"], capture_output=True, text=True, timeout=300, env=env)
    except subprocess.TimeoutExpired:
        return {"unavailable": "mxq_abi_timing did not finish in 300 s"}
    if out.returncode != 0:
        return {"unavailable": "mxq_abi_timing exited with %d: %s" % (out.returncode, out.stderr.strip()[-200:])}
    rows = {}
    for line in out.stdout.splitlines():
        if line.startswith("{"):
            r = json.loads(line)
            rows.setdefault("2^%d" % r["log2n"], {})[r["op"]] = {"host_enqueue_us": r["host_enqueue_us"],
                                                                 "device_us": r["device_us"], "gbs": r["gbs"]}
    return {"caller": "C program, no interpreter", "what": "per call: host time to enqueue / device time per launch, "
            "best of 5 runs of 100 - 400 back-to-back calls over rotating cold buffers", "sizes": rows}


# ----------------------------------------------------------------------------------------------
# workload 3 (the headline): the 224 linear weights of an 8B Llama-shaped decoder
# ----------------------------------------------------------------------------------------------

DRAWN_LAYERS = (0, 13, 31)     # drawn on the host (seed 1000 layer + idx); layer l holds the bits of DRAWN_LAYERS[l % 3]


class WholeModel:
    """One arena per stream of the hot path, every tensor a slice of it (so that the arena is also one
    flat tensor where an operation takes one): BF16 weights, the two 8-bit anchors, the four lower
    targets, one reconstruction buffer, the fake-quant output and the gradient.  About 89 GB."""

    def __init__(self, device, seed_offset: int = 0):
        import torch
        import paper_2604_00529_b200 as mxq
        self.torch, self.mxq, self.device = torch, mxq, device
        self.shapes = inputs.llama8b_shapes()
        self.sizes = [r * c for *_, r, c in self.shapes]
        self.total = total = sum(self.sizes)
        self.layer_elems = sum(r * c for _, r, c in inputs.LLAMA8B_LAYER)
        u8 = dict(dtype=torch.uint8, device=device)
        bf = dict(dtype=torch.bfloat16, device=device)
        self.w = torch.empty(total, **bf)
        self.host_layers = []                    # the drawn layers' bits, kept for the end-to-end leg and the oracle
        for li, layer in enumerate(DRAWN_LAYERS):
            bits = np.concatenate([inputs.llama8b_tensor(layer + seed_offset, idx) for idx in range(len(inputs.LLAMA8B_LAYER))])
            self.host_layers.append(bits)
            self.w[li * self.layer_elems:(li + 1) * self.layer_elems].copy_(
                torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16))
        for l in range(3, inputs.LLAMA8B_LAYERS):
            src = (l % 3) * self.layer_elems
            self.w[l * self.layer_elems:(l + 1) * self.layer_elems].copy_(self.w[src:src + self.layer_elems])
        self.anchor = {f: (torch.empty(total, **u8), torch.empty(total // BLOCK, **u8)) for f in ("int8", "e4m3")}
        self.target = {f: (torch.empty(total * BITS[f] // 8, **u8), torch.empty(total // BLOCK, **u8))
                       for f in ("int6", "int4", "e2m3", "e2m1")}
        self.deq = torch.empty(total, **bf)
        self.fq = torch.empty(total, **bf)
        self.grad = torch.empty(total, **bf)
        # per-tensor views and the prepared calls / item tables built from them
        offs = np.concatenate([[0], np.cumsum(self.sizes)]).astype(np.int64)
        self.offs = offs

        def view(buf, k, bits=8):
            return buf[int(offs[k]) * bits // 8:int(offs[k + 1]) * bits // 8]

        def sview(buf, k):
            return buf[int(offs[k]) // BLOCK:int(offs[k + 1]) // BLOCK]

        T = range(len(self.sizes))
        self.q_calls = {f: [mxq.prepare_quantize(self.w[int(offs[k]):int(offs[k + 1])], f, BLOCK,
                                                 view(self.anchor[f][0], k), sview(self.anchor[f][1], k)) for k in T]
                        for f in ("int8", "e4m3")}
        self.q_tables = {f: mxq.make_q_items([(self.w[int(offs[k]):int(offs[k + 1])], view(self.anchor[f][0], k),
                                               sview(self.anchor[f][1], k)) for k in T]) for f in ("int8", "e4m3")}
        self.ss_pairs = (("int8", "int6"), ("int8", "int4"), ("e4m3", "e2m3"), ("e4m3", "e2m1"))
        self.ss_items = {}
        self.ss_calls = {}
        for a, t in self.ss_pairs:
            items = [(view(self.anchor[a][0], k), sview(self.anchor[a][1], k), self.sizes[k],
                      view(self.target[t][0], k, BITS[t]), sview(self.target[t][1], k)) for k in T]
            self.ss_items[(a, t)] = mxq.make_items(items)
            self.ss_calls[(a, t)] = [mxq.prepare_slice_scale(c, s, n, a, t, BLOCK, oc, os_) for c, s, n, oc, os_ in items]
        self.dq_calls = {t: [mxq.prepare_dequantize(view(self.target[t][0], k, BITS[t]), sview(self.target[t][1], k),
                                                    self.sizes[k], t, BLOCK, self.deq[int(offs[k]):int(offs[k + 1])]) for k in T]
                         for t in ("int4", "e2m1")}
        self.dq_tables = {t: mxq.make_dq_items([(view(self.target[t][0], k, BITS[t]), sview(self.target[t][1], k),
                                                 self.sizes[k], self.deq[int(offs[k]):int(offs[k + 1])]) for k in T])
                          for t in ("int4", "e2m1")}
        self.fq_pairs = [(self.w[int(offs[k]):int(offs[k + 1])], self.fq[int(offs[k]):int(offs[k + 1])]) for k in T]
        self.fq_table = mxq.make_fq_items(self.fq_pairs)
        self.bwd = mxq.prepare_fake_quant_bwd(self.fq, self.grad)
        self.launches_per_step = len(STEP_OPS)               # every op group is one launch over the 224 tensors

    def step(self, mark=None):
        """One pass of the whole hot path over the weight set; `mark(k)` is called before op group k
        (the order of STEP_OPS) and after the last one."""
        mxq = self.mxq
        groups = [
            lambda: mxq.quantize_batched(self.q_tables["int8"], "int8", BLOCK),
            lambda: mxq.quantize_batched(self.q_tables["e4m3"], "e4m3", BLOCK),
            lambda: mxq.slice_scale_batched(self.ss_items[("int8", "int6")], "int8", "int6", BLOCK),
            lambda: mxq.slice_scale_batched(self.ss_items[("int8", "int4")], "int8", "int4", BLOCK),
            lambda: mxq.slice_scale_batched(self.ss_items[("e4m3", "e2m3")], "e4m3", "e2m3", BLOCK),
            lambda: mxq.slice_scale_batched(self.ss_items[("e4m3", "e2m1")], "e4m3", "e2m1", BLOCK),
            lambda: mxq.dequantize_batched(self.dq_tables["int4"], "int4", BLOCK),
            lambda: mxq.dequantize_batched(self.dq_tables["e2m1"], "e2m1", BLOCK),
            lambda: mxq.fake_quant_batched(self.fq_table, "e2m3", BLOCK, mxq.FQ_VIA_ANCHOR),
            lambda: self.bwd(),
        ]
        for k, g in enumerate(groups):
            if mark:
                mark(k)
            g()
        if mark:
            mark(len(groups))


def whole_model_conversions(bench: Bench, wm: WholeModel):
    """Wall time of the whole-model conversion per target: one batched launch against 224 launches;
    the fused fake-quant of all weights the same two ways."""
    mxq = wm.mxq
    out = {}
    for a, t in wm.ss_pairs:
        nbytes = b_slice_scale(t) * wm.total
        tb = bench.regions(lambda j: mxq.slice_scale_batched(wm.ss_items[(a, t)], a, t, BLOCK), 1, reps=1, warm=1)
        tp = bench.regions(lambda j: [c() for c in wm.ss_calls[(a, t)]], 1, reps=1, warm=1)
        out["%s_to_%s" % (a, t)] = {"batched_one_launch": bench.record(tb, nbytes, wm.total),
                                    "per_tensor_launches": bench.record(tp, nbytes, wm.total, launches_per_call=len(wm.sizes))}
        bench.launches += (REGIONS + 1) * (1 + len(wm.sizes))
    # both lower formats of a family from ONE read of the anchor, over the whole model in one launch
    for a, t1, t2 in (("int8", "int6", "int4"), ("e4m3", "e2m3", "e2m1")):
        table = mxq.make_pair_items([(c, s, n, oc1, os1, oc2, os2) for (c, s, n, oc1, os1), (_, _, _, oc2, os2)
                                     in zip(wm.ss_items[(a, t1)].tensors, wm.ss_items[(a, t2)].tensors)])
        nbytes = (1 + SCALE_B + BITS[t1] / 8 + SCALE_B + BITS[t2] / 8 + SCALE_B) * wm.total
        tb = bench.regions(lambda j: mxq.slice_scale_pair_batched(table, a, t1, t2, BLOCK), 1, reps=1, warm=1)
        out["%s_to_%s_and_%s_one_read" % (a, t1, t2)] = {"batched_one_launch": bench.record(tb, nbytes, wm.total)}
        bench.launches += REGIONS + 1
        del table
    for f in ("int8", "e4m3"):
        nbytes = b_quantize(2, f) * wm.total
        tb = bench.regions(lambda j: mxq.quantize_batched(wm.q_tables[f], f, BLOCK), 1, reps=1, warm=1)
        tp = bench.regions(lambda j: [c() for c in wm.q_calls[f]], 1, reps=1, warm=1)
        out["quantize_bf16_%s" % f] = {"batched_one_launch": bench.record(tb, nbytes, wm.total),
                                       "per_tensor_launches": bench.record(tp, nbytes, wm.total, launches_per_call=len(wm.sizes))}
        bench.launches += (REGIONS + 1) * (1 + len(wm.sizes))
    for t in ("int4", "e2m1"):
        nbytes = b_dequantize(t, 2) * wm.total
        tb = bench.regions(lambda j: mxq.dequantize_batched(wm.dq_tables[t], t, BLOCK), 1, reps=1, warm=1)
        tp = bench.regions(lambda j: [c() for c in wm.dq_calls[t]], 1, reps=1, warm=1)
        out["dequantize_%s_bf16" % t] = {"batched_one_launch": bench.record(tb, nbytes, wm.total),
                                         "per_tensor_launches": bench.record(tp, nbytes, wm.total, launches_per_call=len(wm.sizes))}
        bench.launches += (REGIONS + 1) * (1 + len(wm.sizes))
    for fmt in ("e2m3", "int4"):
        tb = bench.regions(lambda j: mxq.fake_quant_batched(wm.fq_table, fmt, BLOCK, mxq.FQ_VIA_ANCHOR), 1, reps=1, warm=1)
        out["fake_quant_%s_via_anchor" % fmt] = {"batched_one_launch": bench.record(tb, 4.0 * wm.total, wm.total)}
        bench.launches += REGIONS + 1
    return out


def end_to_end(wm: WholeModel, steps: int):
    """The headline step through the public API with HOST buffers: every step copies the 14 GB of BF16
    weights from pinned host memory (layer by layer, from the three drawn layers' pinned copies), runs
    the whole hot path, and copies the four converted sets (codes + scales, 18.3 GB) back to pinned host
    memory (layer by layer into one layer-sized pinned buffer).  Three streams: the copy-in of step k + 1
    overlaps the copy-out of step k; the kernels wait for both.  Returns (ms per step, h2d, d2h bytes)."""
    torch = wm.torch
    L, le = inputs.LLAMA8B_LAYERS, wm.layer_elems
    host_in = [torch.from_numpy(b.view(np.int16)).pin_memory() for b in wm.host_layers]
    host_out = {t: (torch.empty(le * BITS[t] // 8, dtype=torch.uint8).pin_memory(),
                    torch.empty(le // BLOCK, dtype=torch.uint8).pin_memory()) for t in wm.target}
    h2d = L * le * 2
    d2h = sum(L * (le * BITS[t] // 8 + le // BLOCK) for t in wm.target)
    s_in, s_cmp, s_out = torch.cuda.Stream(wm.device), torch.cuda.Stream(wm.device), torch.cuda.Stream(wm.device)
    w16 = wm.w.view(torch.int16)

    def run(count):
        ev_in = [torch.cuda.Event() for _ in range(count)]
        ev_cmp = [torch.cuda.Event() for _ in range(count)]
        ev_out = [torch.cuda.Event() for _ in range(count)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s_in)
        for k in range(count):
            with torch.cuda.stream(s_in):
                if k:
                    s_in.wait_event(ev_cmp[k - 1])            # the previous step has read the weights
                for l in range(L):
                    w16[l * le:(l + 1) * le].copy_(host_in[l % len(host_in)], non_blocking=True)
                ev_in[k].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in[k])
                if k:
                    s_cmp.wait_event(ev_out[k - 1])           # the previous results are on the host
                wm.step()
                ev_cmp[k].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[k])
                for l in range(L):
                    for t, (hc, hs) in host_out.items():
                        b = BITS[t]
                        hc.copy_(wm.target[t][0][l * le * b // 8:(l + 1) * le * b // 8], non_blocking=True)
                        hs.copy_(wm.target[t][1][l * le // BLOCK:(l + 1) * le // BLOCK], non_blocking=True)
                ev_out[k].record(s_out)
        e1.record(s_out)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / count

    run(1)                                                    # untimed: pages the pinned buffers in
    ms = run(steps)
    return ms, h2d, d2h


# ----------------------------------------------------------------------------------------------
# the CPU oracle arm (reported baseline; also `--impl reference`)
# ----------------------------------------------------------------------------------------------

def oracle_step(x_bits: np.ndarray):
    """The op groups of the headline step on the CPU oracle (as it stands), on one slice of the weights."""
    from oracle import mxq_oracle as orc
    ci, si = orc.quantize(x_bits, "int8", BLOCK)
    ca, sa = orc.quantize(x_bits, "e4m3", BLOCK)
    orc.slice_scale(ci, si, "int8", "int6", BLOCK)
    c4i, s4i = orc.slice_scale(ci, si, "int8", "int4", BLOCK)
    orc.slice_scale(ca, sa, "e4m3", "e2m3", BLOCK)
    c4, s4 = orc.slice_scale(ca, sa, "e4m3", "e2m1", BLOCK)
    orc.dequantize(c4i, s4i, "int4", BLOCK, orc.BF16)
    orc.dequantize(c4, s4, "e2m1", BLOCK, orc.BF16)
    g = orc.fake_quant(x_bits, "e2m3", BLOCK, orc.FQ_VIA_ANCHOR)
    orc.fake_quant_bwd(g)
    return x_bits.size


def _oracle_worker(args):
    path, lo, hi = args
    x = np.load(path, mmap_mode="r")[lo:hi]
    return oracle_step(np.ascontiguousarray(x))


def oracle_all_cores(sample: np.ndarray, pool, cores: int, path: str) -> float:
    """Seconds for the oracle step over `sample`, split over `cores` processes by contiguous runs of
    whole blocks (every MX block is converted on its own); the slices are read from a scratch file."""
    nblk = sample.size // BLOCK
    cuts = [(nblk * k // cores) * BLOCK for k in range(cores + 1)]
    jobs = [(path, cuts[k], cuts[k + 1]) for k in range(cores) if cuts[k + 1] > cuts[k]]
    t0 = time.perf_counter()
    done = sum(pool.map(_oracle_worker, jobs))
    dt = time.perf_counter() - t0
    assert done == sample.size
    return dt


def sample_weights(elements: int) -> np.ndarray:
    """The first `elements` elements of layer 0 of the headline weight set (q, k, v, o, then gate ...)."""
    parts, have = [], 0
    for idx in range(len(inputs.LLAMA8B_LAYER)):
        if have >= elements:
            break
        t = inputs.llama8b_tensor(0, idx)
        parts.append(t)
        have += t.size
    return np.ascontiguousarray(np.concatenate(parts)[:elements])


def cpu_baseline(sample_log2: int = 26):
    """Oracle throughput on the first 2^26 weights of the headline set: one thread, and the same code
    split over all host cores."""
    import multiprocessing as mp
    import tempfile
    from oracle import mxq_oracle as orc
    orc.lib()
    cores = len(os.sched_getaffinity(0))
    sample = sample_weights(1 << sample_log2)
    nbytes = STEP_BYTES_PER_ELEM * sample.size
    what = "first 2^%d elements of layer 0 of the weight set, the %d op groups of the step" % (sample_log2, len(STEP_OPS))
    with tempfile.TemporaryDirectory() as d:
        path = os.path.join(d, "sample.npy")
        np.save(path, sample)
        with mp.get_context("fork").Pool(cores) as pool:
            pool.map(_oracle_worker, [(path, 0, BLOCK)] * cores)          # start the workers, load the library
            dt_all = oracle_all_cores(sample, pool, cores, path)
    t0 = time.perf_counter()
    oracle_step(sample)
    dt_one = time.perf_counter() - t0
    return {"value": round(nbytes / dt_all / 1e9, 4), "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": "%s; %.1f s on %d cores" % (what, dt_all, cores),
            "melem_s": round(sample.size * len(STEP_OPS) / dt_all / 1e6, 2),
            "single_thread": {"value": round(nbytes / dt_one / 1e9, 4), "unit": "GB/s", "cores": 1,
                              "melem_s": round(sample.size * len(STEP_OPS) / dt_one / 1e6, 2),
                              "sample": "%s; %.1f s on one core" % (what, dt_one)}}


# ----------------------------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------------------------

def run_cuda(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    want = [w.strip() for w in args.workloads.split(",") if w.strip()]

    # the oracle is timed beside the one-GPU run only (at N > 1 every rank's GPU would be held meanwhile),
    # and before CUDA is initialised, so that its worker processes fork from a plain Python process
    cpu = cpu_baseline() if (world == 1 and not args.no_cpu_baseline) else None

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    import paper_2604_00529_b200 as mxq
    mxq.load_library()
    peak, peak_kind = peaks()
    uuid = getattr(torch.cuda.get_device_properties(local), "uuid", None)
    sampler = ClockSampler(local, "GPU-%s" % uuid if uuid is not None else None)
    sampler.start()
    bench = Bench(torch, sampler, peak, peak_kind)
    t_begin = time.perf_counter()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the headline: K steps of the whole hot path over the whole-model weight set ----
    wm = WholeModel(device, seed_offset=100 * rank)          # weak scaling: every rank its own replica
    nops = len(STEP_OPS)
    for _ in range(args.warmup):
        wm.step()
    barrier()
    stream = torch.cuda.current_stream()
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(nops + 1)] for _ in range(K)]
    barrier()
    h0 = time.perf_counter()
    for s in range(K):
        wm.step(mark=lambda k, e=ev[s]: e[k].record(stream))
    barrier()
    h1 = time.perf_counter()
    total_ms = ev[0][0].elapsed_time(ev[K - 1][nops])
    step_ms = [ev[s][0].elapsed_time(ev[s + 1][0] if s + 1 < K else ev[s][nops]) for s in range(K)]
    op_ms = [[ev[s][k].elapsed_time(ev[s][k + 1]) for s in range(K)] for k in range(nops)]
    if world > 1:
        t = torch.tensor([total_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    clocks = sampler.summary(h0, h1)
    ms_per_step = total_ms / K
    headline_launches = wm.launches_per_step * K

    workloads = {}
    if rank == 0 and "w3" in want:
        workloads["w3_whole_model"] = {"elements": wm.total, "tensors": len(wm.sizes),
                                       "conversions": whole_model_conversions(bench, wm)}

    # ---- end to end with host buffers ----
    barrier()
    e2e_steps = 3
    e2e_ms, h2d, d2h = end_to_end(wm, e2e_steps)
    barrier()
    if world > 1:
        t = torch.tensor([e2e_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    total_elems = wm.total
    n_tensors = len(wm.sizes)
    launches_per_step = wm.launches_per_step
    del wm
    torch.cuda.empty_cache()

    # ---- the other workloads (rank 0; the other ranks wait at the barrier) ----
    if rank == 0:
        if "w1" in want:
            workloads["w1_fp32_4096x4096"] = workload1(bench, device)
            torch.cuda.empty_cache()
        if "w2" in want:
            workloads["w2_bf16_8192x8192"] = workload2(bench, device, seed=1, nsets=args.buffer_sets)
        if "w4" in want:
            workloads["w4_fake_quant_activations"] = workload4(bench, device)
            torch.cuda.empty_cache()
        if "w5" in want:
            workloads["w5_size_sweep"] = workload5(bench, device, args.min_log2, args.max_log2)
            torch.cuda.synchronize()
            workloads["w5_size_sweep"]["c_abi_small_sizes"] = small_end_abi(local)
    barrier()
    sampler.stop()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    step_bytes = STEP_BYTES_PER_ELEM * total_elems
    value = step_bytes * world / (ms_per_step * 1e-3) / 1e9
    mhz = clocks["sm_mhz"]
    per_op = {}
    for (name, bpe), ms in zip(STEP_OPS, op_ms):
        med = statistics.median(ms)
        gbs = bpe * total_elems / (med * 1e-3) / 1e9
        per_op[name] = {"ms": round(med, 4), "ms_min": round(min(ms), 4), "ms_max": round(max(ms), 4),
                        "gbs": round(gbs, 1), "gelem_s": round(total_elems / (med * 1e-3) / 1e9, 2),
                        "frac_of_%s_peak" % peak_kind: round(gbs / peak, 4), "frac_of_8000": round(gbs / 8000.0, 4),
                        "launches": 1}
        if mhz:
            per_op[name]["ms_x_ghz"] = round(med * mhz / 1e3, 4)
    # the dominant kernel: the launch that takes the longest (the batched fake-quant or the copy)
    top = max(range(nops), key=lambda k: statistics.median(op_ms[k]))
    top_name, top_bpe = STEP_OPS[top]
    top_ms = sum(op_ms[top]) / K                              # average launch duration over the timed region
    top_gbs = top_bpe * total_elems / (top_ms * 1e-3) / 1e9
    traffic, dram_pct = ncu_traffic(top_name, total_elems)
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": "GB/s",
        "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4),
        "ms_per_step_spread": {"median": round(statistics.median(step_ms), 4), "min": round(min(step_ms), 4),
                               "max": round(max(step_ms), 4)},
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "impl": "mxq",
        "config": {"workload": HEADLINE, "elements_per_gpu": total_elems, "tensors": n_tensors, "block": BLOCK,
                   "ops_per_step": [name for name, _ in STEP_OPS], "bytes_per_step_per_gpu": int(step_bytes),
                   "gelem_per_s": round(total_elems * nops * world / (ms_per_step * 1e-3) / 1e9, 2),
                   "inputs": "BF16 N(0, 0.02) per tensor; layers %s are drawn on the host (seed 1000 layer + index), "
                             "the other 29 layers are device copies of them in turn" % (list(DRAWN_LAYERS),),
                   "l2": "inputs larger than L2: every buffer of the step is 3.7 - 14 GB",
                   "timing": "value: K steps between two CUDA events on the launching stream; an event between "
                             "steps and between op groups gives ms_per_step_spread and kernels; workloads: median / "
                             "min / max of %d back-to-back regions per figure" % REGIONS},
        "e2e": {"value": round(step_bytes * world / (e2e_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                "ms_per_step": round(e2e_ms, 2),
                "what": "weights from pinned host memory in, the four lower-format code + scale sets out"},
        "gpu_launches": headline_launches,
        "gpu_launches_all_workloads": headline_launches + bench.launches,
        "roofline": {"bound": "hbm", "kernel": top_name, "achieved": round(top_gbs, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(top_gbs / peak, 4), "faster_than_the_copy_peak": bool(top_gbs > peak),
                     "peak_kind": peak_kind, "traffic": traffic,
                     "bytes_per_launch": int(top_bpe * total_elems), "ms_per_launch": round(top_ms, 4),
                     "ncu_dram_pct_of_peak": dram_pct,
                     "note": "achieved counts algorithmic bytes over the CUDA-event duration inside the timed steps; "
                             "the copy peak it is divided by is itself a measured kernel, so a fraction a little "
                             "above 1 means faster than that copy, not faster than the memory"},
        "kernels": per_op,
        "workloads": workloads,
        "cpu_baseline": cpu,
        "clocks": clocks,
        "bench_seconds": round(time.perf_counter() - t_begin, 1),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_ncu_case(args):
    """A small case of the main kernels for profiler captures (a few GB on the device, a handful of
    launches, outputs several times the size of L2): every kernel named below runs three times."""
    import torch
    import paper_2604_00529_b200 as mxq
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    u8 = dict(dtype=torch.uint8, device=dev)
    n_ss, n = 1 << args.case_log2, 1 << (args.case_log2 - 1)
    x = torch.from_numpy(inputs.flat_bf16_normal(1 << 24, seed=5).view(np.int16)).to(dev).view(torch.bfloat16).repeat(n >> 24)
    codes, scales = torch.empty(n_ss, **u8), torch.empty(n_ss // BLOCK, **u8)
    out_c, out_s = torch.empty(n_ss * 6 // 8, **u8), torch.empty(n_ss // BLOCK, **u8)
    y = torch.empty(n, dtype=torch.bfloat16, device=dev)
    # anchors of the sweep input, repeated to 2^30 codes
    mxq.quantize(x, "int8", BLOCK, codes[:n], scales[:n // BLOCK])
    codes[n:].copy_(codes[:n]); scales[n // BLOCK:].copy_(scales[:n // BLOCK])
    torch.cuda.synchronize()
    for _ in range(3):
        mxq.slice_scale(codes, scales, n_ss, "int8", "int4", BLOCK, out_c[:n_ss // 2], out_s)
    for _ in range(3):
        mxq.slice_scale(codes, scales, n_ss, "int8", "int6", BLOCK, out_c, out_s)
    for _ in range(3):
        mxq.quantize(x, "e4m3", BLOCK, codes[:n], scales[:n // BLOCK])
    codes[n:].copy_(codes[:n]); scales[n // BLOCK:].copy_(scales[:n // BLOCK])
    for _ in range(3):
        mxq.slice_scale(codes, scales, n_ss, "e4m3", "e2m3", BLOCK, out_c, out_s)
    for _ in range(3):
        mxq.slice_scale(codes, scales, n_ss, "e4m3", "e2m1", BLOCK, out_c[:n_ss // 2], out_s)
    for _ in range(3):
        mxq.dequantize(out_c[:n // 2], out_s[:n // BLOCK], n, "e2m1", BLOCK, dst=y)
    for _ in range(3):
        mxq.fake_quant(x, "e2m3", BLOCK, mxq.FQ_VIA_ANCHOR, dst=y)
    # the two single launches that dominate the headline step, on two decoder layers' worth of weights
    sizes = [r * c for _, r, c in inputs.LLAMA8B_LAYER] * 2
    while sum(sizes) > n:
        sizes.pop()
    offs = np.concatenate([[0], np.cumsum(sizes)])
    pairs = [(x[int(offs[k]):int(offs[k + 1])], y[int(offs[k]):int(offs[k + 1])]) for k in range(len(sizes))]
    table = mxq.make_fq_items(pairs)
    for _ in range(3):
        mxq.fake_quant_batched(table, "e2m3", BLOCK, mxq.FQ_VIA_ANCHOR)
    for _ in range(3):
        mxq.fake_quant_bwd(x, y)
    torch.cuda.synchronize()
    print(json.dumps({"impl": "ncu-case", "elements": {"slice_scale": n_ss, "quantize": n, "dequantize": n, "fake_quant": n,
                                                        "fake_quant_batched": int(offs[-1]), "copy": n}}), flush=True)


def run_reference(args):
    """`--impl reference`: the CPU oracle on the machine's host cores, same metric and config; every step
    is the first 2^24 weights of the headline set through the op groups of the step, split over all
    cores.  Under torchrun rank 0 alone runs it."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import multiprocessing as mp
    import tempfile
    from oracle import mxq_oracle as orc
    orc.lib()
    cores = len(os.sched_getaffinity(0))
    sample = sample_weights(1 << 24)
    with tempfile.TemporaryDirectory() as d:
        path = os.path.join(d, "sample.npy")
        np.save(path, sample)
        with mp.get_context("fork").Pool(cores) as pool:
            for _ in range(max(1, min(args.warmup, 3))):
                oracle_all_cores(sample, pool, cores, path)
            t0 = time.perf_counter()
            for _ in range(args.steps):
                oracle_all_cores(sample, pool, cores, path)
            dt = (time.perf_counter() - t0) / args.steps
    gbs = STEP_BYTES_PER_ELEM * sample.size / dt / 1e9
    what = ("each step = the first 2^24 elements of layer 0 of the weight set through the %d op groups of the step, "
            "split over %d processes by block ranges" % (len(STEP_OPS), cores))
    line = {
        "metric": METRIC, "value": round(gbs, 4), "unit": "GB/s", "impl": "reference",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": HEADLINE, "block": BLOCK, "ops_per_step": [n for n, _ in STEP_OPS], "sample": what},
        "cpu_baseline": {"value": round(gbs, 4), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": round(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_selftest(args):
    """The rank plumbing alone, on CPU (gloo): rendezvous, barrier, max over ranks, one line from rank 0.
    Used by the tests to drive the `--gpus N` launcher without a GPU."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"impl": "selftest", "n_gpus": world, "max_over_ranks": float(t.item())}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def launch_ranks(n: int) -> int:
    """`--gpus N` outside torchrun: start N copies of this command, one rank per device, with the
    rendezvous variables torch.distributed reads; rank 0's line is the output.  Returns the exit code."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    rc = 0
    for p in procs:
        rc = max(rc, abs(p.wait()))
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="mxq", choices=["mxq", "reference", "selftest", "ncu-case"])
    ap.add_argument("--workloads", default="w1,w2,w3,w4,w5",
                    help="which entries of the `workloads` record to measure beside the headline")
    ap.add_argument("--min-log2", type=int, default=16)
    ap.add_argument("--max-log2", type=int, default=31)
    ap.add_argument("--buffer-sets", type=int, default=4, help="rotating buffer sets of workload 2 (>= 2)")
    ap.add_argument("--case-log2", type=int, default=30,
                    help="--impl ncu-case: 2^N codes for Slice-and-Scale, 2^(N-1) elements for the other kernels")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.steps = max(args.steps, 1)
    args.buffer_sets = max(args.buffer_sets, 2)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus))
    if args.impl == "reference":
        run_reference(args)
    elif args.impl == "selftest":
        run_selftest(args)
    elif args.impl == "ncu-case":
        run_ncu_case(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
