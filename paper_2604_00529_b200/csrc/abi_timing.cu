// mxq_abi_timing: calls the C ABI of libmxq directly, in a loop, and splits the cost of a call into
// the host's time to enqueue it and the device's time to run it -- without an interpreter between
// the caller and the library.  For every operation and tensor size it prints one JSON line:
//   {"op": ..., "log2n": k, "copies": c, "reps": r, "host_enqueue_us": h, "device_us": d, "gbs": g}
// host_enqueue_us = wall time of the r calls (no synchronisation inside) / r; device_us = CUDA-event
// time of the same r launches / r (the launches rotate over `copies` buffer sets whose total size
// exceeds L2 several times over, so the figures are cold).  Small tensors are bound by whichever of
// the two is larger.
//
//   mxq_abi_timing [min_log2 [max_log2 [step]]]      (defaults 16, 24 and 1)
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/mxq.h"

#define CK(x)                                                                                   \
    do {                                                                                        \
        cudaError_t e_ = (x);                                                                   \
        if (e_ != cudaSuccess) {                                                                \
            fprintf(stderr, "%s failed: %s\n", #x, cudaGetErrorString(e_));                     \
            return 2;                                                                           \
        }                                                                                       \
    } while (0)

namespace {

struct Set {
    void *x, *y, *codes, *out;
    uint8_t *scales, *out_scales;
};

double now_us()
{
    using namespace std::chrono;
    return duration<double, std::micro>(steady_clock::now().time_since_epoch()).count();
}

}  // namespace

int main(int argc, char** argv)
{
    const int lo = argc > 1 ? atoi(argv[1]) : 16, hi = argc > 2 ? atoi(argv[2]) : 24, step = argc > 3 ? atoi(argv[3]) : 1;
    if (lo < 10 || hi > 28 || lo > hi || step < 1) {
        fprintf(stderr, "sizes 2^10 ... 2^28\n");
        return 1;
    }
    cudaStream_t stream;
    CK(cudaStreamCreate(&stream));
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    const size_t l2 = 126u << 20;

    for (int k = lo; k <= hi; k += step) {
        const size_t n = (size_t)1 << k;
        size_t copies = (4 * l2) / (2 * n) + 1;
        if (copies < 2) copies = 2;
        if (copies > 2048) copies = 2048;
        // seeded contents: BF16 values of moderate magnitude, codes without E4M3 NaN patterns
        std::vector<uint16_t> hx(n);
        std::vector<uint8_t> hc(n), hs(n / 32);
        uint32_t r = 12345u + (uint32_t)k;
        for (size_t i = 0; i < n; ++i) {
            r = r * 1664525u + 1013904223u;
            hx[i] = (uint16_t)(0x3C00u + ((r >> 16) & 0x03FFu)) | (uint16_t)((r >> 3) & 0x8000u);
            hc[i] = (uint8_t)((r >> 8) & 0xF7u);
        }
        for (size_t i = 0; i < n / 32; ++i) hs[i] = (uint8_t)(100 + i % 40);
        std::vector<Set> sets(copies);
        for (auto& s : sets) {
            CK(cudaMalloc(&s.x, n * 2));
            CK(cudaMalloc(&s.y, n * 2));
            CK(cudaMalloc(&s.codes, n));
            CK(cudaMalloc(&s.out, n));
            CK(cudaMalloc((void**)&s.scales, n / 32 + 32));
            CK(cudaMalloc((void**)&s.out_scales, n / 32 + 32));
            CK(cudaMemcpy(s.x, hx.data(), n * 2, cudaMemcpyHostToDevice));
            CK(cudaMemcpy(s.codes, hc.data(), n, cudaMemcpyHostToDevice));
            CK(cudaMemcpy(s.scales, hs.data(), n / 32, cudaMemcpyHostToDevice));
        }
        struct Op {
            const char* name;
            double bytes_per_elem;
            int (*call)(const Set&, size_t, cudaStream_t);
        };
        const Op ops[] = {
            {"quantize_bf16_e4m3", 2 + 1 + 1.0 / 32,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_quantize(s.x, MXQ_BF16, n, MXQ_FP8_E4M3, 32, s.out, s.out_scales, st); }},
            {"quantize_bf16_int8", 2 + 1 + 1.0 / 32,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_quantize(s.x, MXQ_BF16, n, MXQ_INT8, 32, s.out, s.out_scales, st); }},
            {"ss_e4m3_e2m1", 1 + 0.5 + 2.0 / 32,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_slice_scale(s.codes, s.scales, n, 32, MXQ_FP8_E4M3, MXQ_FP4_E2M1, s.out, s.out_scales, st); }},
            {"ss_e4m3_e2m3", 1 + 0.75 + 2.0 / 32,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_slice_scale(s.codes, s.scales, n, 32, MXQ_FP8_E4M3, MXQ_FP6_E2M3, s.out, s.out_scales, st); }},
            {"ss_int8_int4", 1 + 0.5 + 2.0 / 32,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_slice_scale(s.codes, s.scales, n, 32, MXQ_INT8, MXQ_INT4, s.out, s.out_scales, st); }},
            {"ss_int8_int6", 1 + 0.75 + 2.0 / 32,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_slice_scale(s.codes, s.scales, n, 32, MXQ_INT8, MXQ_INT6, s.out, s.out_scales, st); }},
            {"dequantize_e2m1_bf16", 0.5 + 1.0 / 32 + 2,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_dequantize(s.codes, s.scales, n, MXQ_FP4_E2M1, 32, s.y, MXQ_BF16, st); }},
            {"fake_quant_bf16_e2m3_via_anchor", 4.0,
             [](const Set& s, size_t n, cudaStream_t st) { return mxq_fake_quant(s.x, MXQ_BF16, n, MXQ_FP6_E2M3, 32, MXQ_FQ_VIA_ANCHOR, s.y, st); }},
        };
        const int reps = k <= 22 ? 400 : 100;
        for (const Op& op : ops) {
            for (size_t j = 0; j < 8; ++j)
                if (op.call(sets[j % copies], n, stream) != MXQ_OK) {
                    fprintf(stderr, "%s failed\n", op.name);
                    return 3;
                }
            CK(cudaStreamSynchronize(stream));
            double best_host = 1e30, best_dev = 1e30;
            for (int round = 0; round < 5; ++round) {
                CK(cudaEventRecord(e0, stream));
                const double t0 = now_us();
                for (int i = 0; i < reps; ++i) op.call(sets[(size_t)i % copies], n, stream);
                const double t1 = now_us();
                CK(cudaEventRecord(e1, stream));
                CK(cudaEventSynchronize(e1));
                float ms = 0;
                CK(cudaEventElapsedTime(&ms, e0, e1));
                const double host = (t1 - t0) / reps, dev = ms * 1e3 / reps;
                if (host < best_host) best_host = host;
                if (dev < best_dev) best_dev = dev;
            }
            printf("{\"op\": \"%s\", \"log2n\": %d, \"copies\": %zu, \"reps\": %d, \"host_enqueue_us\": %.3f, "
                   "\"device_us\": %.3f, \"gbs\": %.1f}\n",
                   op.name, k, copies, reps, best_host, best_dev, op.bytes_per_elem * (double)n / best_dev / 1e3);
            fflush(stdout);
        }
        for (auto& s : sets) {
            cudaFree(s.x); cudaFree(s.y); cudaFree(s.codes); cudaFree(s.out); cudaFree(s.scales); cudaFree(s.out_scales);
        }
    }
    return 0;
}
