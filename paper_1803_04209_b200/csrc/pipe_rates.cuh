// Issue rates of the pipes the decision path leans on, measured on the device at hand:
// fp32 min / max (ALU pipe), warp shuffles and fp32 fused multiply-adds, each as warp-instructions
// per clock per SM.  One CTA of 32 warps per SM runs eight independent dependency chains per thread,
// so the pipe, not latency, limits the rate; the CTA times itself with the SM's cycle counter.
// These are the measured denominators the benchmark sets the sort and the chain against.
#pragma once
#include <cstdint>
#include <cuda.h>

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

// ---------------------------------------------------------------------------------------------
// Rate of the operand stream L2 -> shared memory: what the emission output layer is set against.
// Every SM runs one CTA in which one thread keeps a ring of four stages filled with the copies that kernel
// issues per K block (three tensor-map boxes of 128 rows x 128 bytes, 128-byte swizzle: 48 KB), re-arming a
// stage as soon as its copies have landed; nothing consumes the data.  The boxes walk over a matrix of 256
// columns that the caller sizes: a few MB that every SM re-reads (the weights' case) or tens of MB that
// are read a few times each (the hidden vectors' case).  Waits are bounded by an iteration count.
// ---------------------------------------------------------------------------------------------
constexpr int kStreamStages = 4;
constexpr int kStreamBoxes = 3;
constexpr int kStreamBoxRows = 128;
constexpr int kStreamBoxBytes = kStreamBoxRows * 128;
constexpr int kStreamStageBytes = kStreamBoxes * kStreamBoxBytes;
constexpr size_t kStreamSmemBytes = kStreamStages * kStreamStageBytes + 1024 + 8 * kStreamStages;

__global__ void __launch_bounds__(32, 1) k_operand_stream(const __grid_constant__ CUtensorMap map, int n_rows, int n_kb,
                                                          int iters, int* __restrict__ error) {
    extern __shared__ uint8_t stream_smem[];
    const uint32_t raw = static_cast<uint32_t>(__cvta_generic_to_shared(stream_smem));
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t bars = base + kStreamStages * kStreamStageBytes;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStreamStages; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8 * s), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x != 0) return;
    const int row_blocks = n_rows / kStreamBoxRows;
    int rb = static_cast<int>((blockIdx.x * 977u) % static_cast<unsigned>(row_blocks)), kb = 0;
    for (int it = 0; it < iters + kStreamStages; ++it) {
        const int s = it % kStreamStages;
        const uint32_t bar = bars + 8 * s;
        if (it >= kStreamStages) {                       // the copies this stage was armed with have to land first
            const uint32_t parity = ((it / kStreamStages) - 1) & 1;
            uint32_t done = 0;
            for (long long spins = 0; !done; ++spins) {
                asm volatile(
                    "{\n\t.reg .pred p;\n\t"
                    "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                    "selp.u32 %0, 1, 0, p;\n\t}"
                    : "=r"(done) : "r"(bar), "r"(parity) : "memory");
                if (!done && spins > (1ll << 24)) { *error = 1; return; }
            }
        }
        if (it < iters) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kStreamStageBytes) : "memory");
            for (int l = 0; l < kStreamBoxes; ++l) {
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                    ::"r"(base + s * kStreamStageBytes + l * kStreamBoxBytes), "l"(&map), "r"(kb * 32),
                      "r"(rb * kStreamBoxRows), "r"(bar) : "memory");
                rb += 13;
                if (rb >= row_blocks) rb -= row_blocks;
            }
            if (++kb == n_kb) kb = 0;
        }
    }
}

}  // namespace cutoff
