"""Two pieces of index arithmetic that the kernels share with the host, checked on the CPU by a small
host-only program compiled from the library's own header: the coarse tile index of the batched kernels
(owner of every tile against a linear scan) and the tiled scale offset with its multiply-and-shift
division (against the plain formula with exact division)."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2604_00529_b200", "csrc")

PROGRAM = r"""
#include <cstdio>
#include <random>
#include <vector>
#include "mxq_kernels.cuh"
using namespace mxq;

static int check_index(std::mt19937_64& g, int count, size_t max_tiles_per_item)
{
    std::vector<SsDeviceItem> items(count);
    size_t tiles = 0;
    for (int i = 0; i < count; ++i) {
        items[i] = SsDeviceItem{};
        items[i].tile_begin = tiles;
        tiles += 1 + g() % max_tiles_per_item;
    }
    TileIndex ix;
    build_tile_index(ix, items.data(), count, tiles);
    size_t step = tiles > 200000 ? tiles / 100003 : 1;
    int owner = 0;
    for (size_t t = 0; t < tiles; ++t) {
        while (owner + 1 < count && items[owner + 1].tile_begin <= t) ++owner;
        if (t % step && t + 1 != tiles && t != items[owner].tile_begin) continue;     // sample, but keep every boundary
        if (find_item(items.data(), ix, t) != owner) {
            std::printf("index: count %d tiles %zu tile %zu: got %d want %d\n", count, tiles, t,
                        find_item(items.data(), ix, t), owner);
            return 1;
        }
    }
    return 0;
}

static int check_offsets(uint32_t rows, uint32_t kblocks)
{
    const TiledScales t = make_tiled_scales(nullptr, kblocks);
    const size_t col_tiles = (kblocks + 3) / 4;
    for (uint32_t r = 0; r < rows; ++r)
        for (uint32_t c = 0; c < kblocks; ++c) {
            const size_t want = ((size_t)(r / 128) * col_tiles + c / 4) * 512 + (r % 32) * 16 + (r / 32 % 4) * 4 + c % 4;
            const size_t got = tiled_scale_offset(t, (size_t)r * kblocks + c);
            if (got != want) {
                std::printf("offset: rows %u kblocks %u r %u c %u: got %zu want %zu\n", rows, kblocks, r, c, got, want);
                return 1;
            }
        }
    return 0;
}

int main()
{
    std::mt19937_64 g(7);
    int bad = 0;
    for (int count : {1, 2, 3, 7, 64, 65, 224, 255, 256, 257, 511, 512})
        for (size_t m : {(size_t)1, (size_t)3, (size_t)40, (size_t)5000, (size_t)300000}) bad += check_index(g, count, m);
    // very uneven sizes: one huge tensor among tiny ones
    {
        std::vector<SsDeviceItem> items(300);
        size_t tiles = 0;
        for (int i = 0; i < 300; ++i) { items[i] = SsDeviceItem{}; items[i].tile_begin = tiles; tiles += i == 150 ? 5000000 : 1; }
        TileIndex ix;
        build_tile_index(ix, items.data(), 300, tiles);
        for (size_t t : {(size_t)0, (size_t)149, (size_t)150, (size_t)151, (size_t)5000149, (size_t)5000150, tiles - 1}) {
            int owner = 0;
            while (owner + 1 < 300 && items[owner + 1].tile_begin <= t) ++owner;
            if (find_item(items.data(), ix, t) != owner) { std::printf("uneven: tile %zu\n", t); ++bad; }
        }
    }
    for (uint32_t kb : {1u, 2u, 3u, 4u, 5u, 7u, 8u, 33u, 100u, 127u, 128u, 129u, 448u, 1000u}) bad += check_offsets(300, kb);
    bad += check_offsets(3, 70001);
    // the largest legal block indices: rows * kblocks just below 2^32
    {
        const uint32_t kb = 65521, rows = 65549;                  // 4294920029 blocks
        const TiledScales t = make_tiled_scales(nullptr, kb);
        for (uint32_t r : {0u, 1u, rows / 2, rows - 2, rows - 1})
            for (uint32_t c : {0u, 1u, kb - 1}) {
                const size_t want = ((size_t)(r / 128) * ((kb + 3) / 4) + c / 4) * 512 + (r % 32) * 16 + (r / 32 % 4) * 4 + c % 4;
                if (tiled_scale_offset(t, (size_t)r * kb + c) != want) { std::printf("large: r %u c %u\n", r, c); ++bad; }
            }
    }
    std::printf("%s\n", bad ? "FAILED" : "index arithmetic ok");
    return bad != 0;
}
"""


def test_coarse_tile_index_and_tiled_offsets_on_the_host(tmp_path):
    src = tmp_path / "index_check.cu"
    src.write_text(PROGRAM)
    exe = tmp_path / "index_check"
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not found")
    subprocess.check_call([nvcc, "-std=c++20", "-O1", "-gencode", "arch=compute_100a,code=sm_100a", "-I", CSRC, str(src), "-o", str(exe)])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout[-2000:]
    assert "index arithmetic ok" in out.stdout
