// Issue rates of the pipes the decision path leans on, measured on the device at hand:
// fp32 min / max (ALU pipe), warp shuffles and fp32 fused multiply-adds, each as warp-instructions
// per clock per SM.  One CTA of 32 warps per SM runs eight independent dependency chains per thread,
// so the pipe, not latency, limits the rate; the CTA times itself with the SM's cycle counter.
// These are the measured denominators the benchmark sets the sort and the chain against.
#pragma once
#include <cstdint>

namespace cutoff {

constexpr int kRateThreads = 1024;
constexpr int kRateChains = 8;
constexpr int kRateIters = 2048;

// kind 0: min / max, 1: shuffle, 2: fused multiply-add
template <int KIND>
__global__ void __launch_bounds__(kRateThreads) k_pipe_rate(float seed, long long* __restrict__ cycles,
                                                             float* __restrict__ sink) {
    float v[kRateChains];
#pragma unroll
    for (int i = 0; i < kRateChains; ++i) v[i] = seed * static_cast<float>(threadIdx.x * kRateChains + i + 1);
    const float a = seed * 1.0001f, b = seed * 0.5f;
    __syncthreads();
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < kRateIters; ++it) {
#pragma unroll
        for (int i = 0; i < kRateChains; ++i) {
            if (KIND == 0) v[i] = (i & 1) ? fminf(v[i], v[(i + 3) % kRateChains]) : fmaxf(v[i], v[(i + 5) % kRateChains]);
            if (KIND == 1) v[i] = __shfl_xor_sync(0xffffffffu, v[i], 1 + ((i + it) & 15));
            if (KIND == 2) v[i] = fmaf(v[i], a, b);
        }
    }
    const long long t1 = clock64();
    __syncthreads();
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < kRateChains; ++i) s += v[i];
    if (s == 123.456f) sink[0] = s;                   // keeps the chains alive; never true in practice
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}  // namespace cutoff
