// Register-only microbenchmarks of the integer pipes: the denominators of the search kernel's
// roofline.  Three instruction mixes, each with enough independent chains per thread to hide the
// pipe latency, no memory traffic inside the timed loops:
//   [0] 32-bit three-input logic ops           (ALU pipe only)
//   [1] 32-bit add + logic pairs               (the compiler may spread adds over ALU and FMA pipes)
//   [2] the search kernel's own candidate mix: 64-bit add followed by 64-bit signed compare,
//       counted as 4 32-bit instructions per candidate
//   [3] SM clock in MHz seen during the runs (clock64 ticks per microsecond of globaltimer)
#include <cuda_runtime.h>
#include <stdint.h>

#include "mmee_search.h"

namespace mmee {

namespace {

constexpr int kChains = 12;
constexpr int kIters = 2048;

__global__ void __launch_bounds__(256) logic_kernel(const uint32_t* __restrict__ seed, uint32_t* __restrict__ sink) {
    uint32_t a[kChains];
    const uint32_t m = seed[0], n = seed[1];
#pragma unroll
    for (int c = 0; c < kChains; ++c) a[c] = seed[2 + c] + threadIdx.x;
#pragma unroll 1
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int c = 0; c < kChains; ++c) a[c] = (a[c] & m) ^ (a[c] | n);     // one LOP3 each
    }
    uint32_t x = 0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) x ^= a[c];
    if (x == 0x12345u) sink[0] = x;
}

__global__ void __launch_bounds__(256) add_kernel(const uint32_t* __restrict__ seed, uint32_t* __restrict__ sink) {
    uint32_t a[kChains], b[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) { a[c] = seed[2 + c] + threadIdx.x; b[c] = seed[c] | 1u; }
#pragma unroll 1
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int c = 0; c < kChains; ++c) { a[c] += b[c]; b[c] ^= a[c]; }     // one add, one logic op
    }
    uint32_t x = 0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) x ^= a[c] + b[c];
    if (x == 0x12345u) sink[0] = x;
}

__global__ void __launch_bounds__(256) key_mix_kernel(const int64_t* __restrict__ seed, uint32_t* __restrict__ sink,
                                                      unsigned long long* __restrict__ clocks) {
    int64_t w[9];
#pragma unroll
    for (int s = 0; s < 9; ++s) w[s] = seed[s];
    const int64_t thr = seed[9], dx = seed[10];
    int64_t x0 = seed[11] + threadIdx.x, x1 = seed[12] + threadIdx.x;
    bool any = false;
    unsigned long long t0 = 0, c0 = 0;
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        c0 = clock64();
    }
#pragma unroll 1
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            x0 += dx;
            x1 -= dx;
#pragma unroll
            for (int s = 0; s < 9; ++s) {
                any |= (x0 + w[s]) < thr;
                any |= (x1 + w[s]) < thr;
            }
        }
    }
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        unsigned long long t1, c1 = clock64();
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        clocks[0] = c1 - c0;
        clocks[1] = t1 - t0;
    }
    if (any) sink[1] = 1;
}

}  // namespace

cudaError_t measure_alu_peak(double* giops) {
    int dev = 0;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaGetDeviceProperties(&prop, dev)) != cudaSuccess) return e;
    const int grid = prop.multiProcessorCount * 8;
    void* buf = nullptr;
    if ((e = cudaMalloc(&buf, 4096)) != cudaSuccess) return e;
    int64_t host[64];
    for (int i = 0; i < 64; ++i) host[i] = 0x0101010101010101ll * (i + 1);
    // keys never fall below the threshold, as in the steady state of a search
    host[9] = INT64_MIN + 16;
    host[10] = 3;
    if ((e = cudaMemcpy(buf, host, sizeof(host), cudaMemcpyHostToDevice)) != cudaSuccess) { cudaFree(buf); return e; }
    uint32_t* sink = reinterpret_cast<uint32_t*>(static_cast<char*>(buf) + 1024);
    unsigned long long* clocks = reinterpret_cast<unsigned long long*>(static_cast<char*>(buf) + 2048);
    cudaEvent_t ev0, ev1;
    cudaEventCreate(&ev0);
    cudaEventCreate(&ev1);
    const double threads = (double)grid * 256.0;
    double best[3] = {0, 0, 0};
    for (int rep = 0; rep < 4 && e == cudaSuccess; ++rep) {
        for (int which = 0; which < 3; ++which) {
            cudaEventRecord(ev0);
            if (which == 0) logic_kernel<<<grid, 256>>>(static_cast<uint32_t*>(buf), sink);
            else if (which == 1) add_kernel<<<grid, 256>>>(static_cast<uint32_t*>(buf), sink);
            else key_mix_kernel<<<grid, 256>>>(static_cast<int64_t*>(buf), sink, clocks);
            cudaEventRecord(ev1);
            if ((e = cudaEventSynchronize(ev1)) != cudaSuccess) break;
            float ms = 0;
            cudaEventElapsedTime(&ms, ev0, ev1);
            double inst;
            if (which == 0) inst = threads * kIters * 8.0 * kChains;
            else if (which == 1) inst = threads * kIters * 8.0 * kChains * 2.0;
            else inst = threads * kIters * 4.0 * 18.0 * 4.0;
            const double rate = inst / (ms * 1e-3) / 1e9;
            if (rep > 0 && rate > best[which]) best[which] = rate;
        }
    }
    unsigned long long hc[2] = {0, 1};
    if (e == cudaSuccess) e = cudaMemcpy(hc, clocks, sizeof(hc), cudaMemcpyDeviceToHost);
    giops[0] = best[0];
    giops[1] = best[1];
    giops[2] = best[2];
    giops[3] = hc[1] ? (double)hc[0] / (double)hc[1] * 1e3 : 0.0;
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    cudaFree(buf);
    return e;
}

}  // namespace mmee
