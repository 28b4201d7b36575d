"""mxq_slice_scale_batched_static -- the batched conversion for callers that may not allocate on the
device (their own pool owns all of HBM, or they cannot take the device-wide synchronisation of
cudaMalloc) -- must give exactly what mxq_slice_scale_batched gives, and what the CPU oracle gives.
Both entry points are called through the C ABI on the same inputs, twice in a row with different item
lists, so that the second call runs over whatever the first left in the library's fixed item table.
Outputs are codes and scale bytes: the tolerance is zero, as everywhere in these tests.  This file
sorts last on purpose: a run that stops at the first failure has then already been through every
other test."""
import numpy as np
import pytest
import torch

import paper_2604_00529_b200 as mxq
from oracle import mxq_oracle as orc

from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu


def _items(sizes, src_bits, dst, seed):
    rng = np.random.default_rng(seed)
    ins, outs_a, outs_b = [], [], []
    for n in sizes:
        codes = rng.integers(0, 1 << src_bits, n).astype(np.uint8)
        scales = rng.integers(0, 256, n // 32).astype(np.uint8)
        c, s = to_dev(codes), to_dev(scales)
        pair = []
        for _ in range(2):
            oc = torch.full((mxq.codes_bytes(n, dst) + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            os_ = torch.full((n // 32 + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            pair.append((c, s, n, oc, os_))
        outs_a.append(pair[0])
        outs_b.append(pair[1])
        ins.append((codes, scales))
    return outs_a, outs_b, ins


@pytest.mark.parametrize("src,dst", [("e4m3", "e2m1"), ("int8", "int6")])
def test_static_table_call_matches_allocating_call_twice(src, dst):
    first = [32 * 4097, 32, 32 * 65, 32 * 1000, 32 * 7, 32 * 64, 32 * 333]
    second = [32 * 129, 32 * 2048, 32 * 3]                 # fewer items: stale entries stay behind them
    for call, sizes in enumerate((first, second)):
        want_items, got_items, host_inputs = _items(sizes, 8, dst, seed=100 + call)
        mxq.slice_scale_batched(want_items, src, dst)
        mxq.slice_scale_batched_static(got_items, src, dst)
        torch.cuda.synchronize()
        for (_, _, n, wc, ws), (_, _, _, gc, gs), (codes, scales) in zip(want_items, got_items, host_inputs):
            assert np.array_equal(to_host(gc), to_host(wc)), (call, n)
            assert np.array_equal(to_host(gs), to_host(ws)), (call, n)
            nb = mxq.codes_bytes(n, dst)
            assert np.all(to_host(gc[nb:]) == 0xA5) and np.all(to_host(gs[n // 32:]) == 0xA5)
            oc, os_ = orc.slice_scale(codes, scales, src, dst)             # Eq. 4-5 on the CPU
            assert np.array_equal(to_host(gc[:nb]), orc.pack(oc, orc.bits(dst))), (call, n, "oracle")
            assert np.array_equal(to_host(gs[:n // 32]), os_), (call, n, "oracle")


def test_static_table_call_rejects_what_does_not_fit():
    n = 32
    c = torch.zeros(n, dtype=torch.uint8, device="cuda")
    s = torch.zeros(1, dtype=torch.uint8, device="cuda")
    oc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda")
    os_ = torch.zeros(1, dtype=torch.uint8, device="cuda")
    too_many = [(c, s, n, oc, os_)] * (mxq.STATIC_BATCH_MAX + 1)
    with pytest.raises(mxq.MxqError) as e:
        mxq.slice_scale_batched_static(too_many, "int8", "int4")
    assert e.value.status == -4                            # MXQ_ERR_SIZE, nothing launched
    mxq.slice_scale_batched_static([(c, s, n, oc, os_)] * mxq.STATIC_BATCH_MAX, "int8", "int4")
    torch.cuda.synchronize()


def test_static_table_call_refuses_a_capturing_stream():
    """The call copies its item table from a buffer that dies with the call, so it must not be
    recorded: on a stream under capture it returns MXQ_ERR_CUDA and enqueues nothing (the captured
    graph stays empty and is never replayed)."""
    n = 32 * 64
    c = torch.zeros(n, dtype=torch.uint8, device="cuda")
    s = torch.full((n // 32,), 127, dtype=torch.uint8, device="cuda")
    oc = torch.full((n // 2,), 0xA5, dtype=torch.uint8, device="cuda")
    os_ = torch.full((n // 32,), 0xA5, dtype=torch.uint8, device="cuda")
    items = [(c, s, n, oc, os_)]
    mxq.slice_scale_batched_static(items, "int8", "int4")      # first call on the device: outside any capture
    torch.cuda.synchronize()
    oc.fill_(0xA5)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    import warnings
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")                        # torch remarks on the empty graph
        with pytest.raises(mxq.MxqError) as e:
            with torch.cuda.graph(graph, stream=side):
                mxq.slice_scale_batched_static(items, "int8", "int4")
    assert e.value.status == -7                                # MXQ_ERR_CUDA
    torch.cuda.synchronize()
    assert np.all(to_host(oc) == 0xA5)                         # nothing ran
    mxq.slice_scale_batched_static(items, "int8", "int4")      # and the entry point still works afterwards
    torch.cuda.synchronize()
    assert np.all(to_host(oc) == 0)
