"""The N > 1 path on CPU: two gloo ranks shard a tensor by whole blocks (no data-path collective),
each converts its shard, and the stitched result equals the unsharded conversion.  The conversion
itself is done by the CPU oracle here (no GPU in this test); what is under test is the host logic:
the shard ranges, the output byte ranges, and the max-over-ranks timing reduction of the bench."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n, tmp):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import mxq_oracle as orc
        from paper_2604_00529_b200 import inputs
        from paper_2604_00529_b200.shard import block_range, output_ranges
        x = inputs.weight_bf16_normal(n // 256, 256, seed=11)
        lo, hi = block_range(n, 32, rank, world)
        codes, scales = orc.quantize(x[lo:hi], "e4m3")
        lc, ls = orc.slice_scale(codes, scales, "e4m3", "e2m1")
        packed = orc.pack(lc, 4)
        (c_lo, c_hi), (s_lo, s_hi) = output_ranges(lo, hi, 4, 32)
        assert packed.size == c_hi - c_lo and ls.size == s_hi - s_lo
        # every rank writes its own byte range of the full outputs: files stand in for the buffers
        full_c = np.lib.format.open_memmap(os.path.join(tmp, "codes.npy"), mode="r+")
        full_s = np.lib.format.open_memmap(os.path.join(tmp, "scales.npy"), mode="r+")
        full_c[c_lo:c_hi] = packed
        full_s[s_lo:s_hi] = ls
        full_c.flush()
        full_s.flush()
        # the bench's timing rule: the slowest rank defines the step time
        t = torch.tensor([1.0 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == float(world)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("nblk", [4096, 4096 + 37])
def test_two_ranks_shard_by_blocks(tmp_path, nblk):
    sys.path.insert(0, ROOT)
    from oracle import mxq_oracle as orc
    from paper_2604_00529_b200 import inputs
    n = nblk * 32
    n = (n // 256) * 256
    np.save(tmp_path / "codes.npy", np.zeros(n // 2, np.uint8))
    np.save(tmp_path / "scales.npy", np.zeros(n // 32, np.uint8))
    orc.lib()                                       # compile once before the ranks start
    mp.spawn(_worker, args=(2, _free_port(), n, str(tmp_path)), nprocs=2, join=True)
    x = inputs.weight_bf16_normal(n // 256, 256, seed=11)
    codes, scales = orc.quantize(x, "e4m3")
    lc, ls = orc.slice_scale(codes, scales, "e4m3", "e2m1")
    assert np.array_equal(np.load(tmp_path / "codes.npy"), orc.pack(lc, 4))
    assert np.array_equal(np.load(tmp_path / "scales.npy"), ls)


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("nblk", [1, 31, 32, 33, 1000, 218103808 // 7])
def test_block_ranges_cover_and_align(world, nblk):
    sys.path.insert(0, ROOT)
    from paper_2604_00529_b200.shard import block_range
    n = nblk * 32
    prev = 0
    for r in range(world):
        lo, hi = block_range(n, 32, r, world)
        assert lo == prev and hi >= lo
        assert hi == lo or lo % (32 * 32) == 0      # a rank with work starts on an aligned chunk
        prev = hi
    assert prev == n


def test_bench_gpus_flag_starts_the_ranks():
    """`bench.py --gpus 2` outside torchrun starts two ranks itself (here the CPU self-test worker over
    gloo) and rank 0 prints one line with n_gpus = 2 and the max over the ranks."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "selftest"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["max_over_ranks"] == 2.0


def test_bench_under_a_launcher_reads_the_rank_environment():
    """Started by a launcher (WORLD_SIZE set), bench.py is one rank and starts nothing itself: a
    one-rank environment prints n_gpus = 1 even with --gpus 1."""
    import json
    import subprocess
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1", "--impl", "selftest"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr
    assert json.loads(out.stdout.strip().splitlines()[-1])["n_gpus"] == 1
