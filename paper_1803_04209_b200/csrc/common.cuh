// Shared device-side declarations of the cutoff library.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace cutoff {

// Observation and decision state that lives on the device, so that a captured CUDA graph can
// replay push + predict without any host-side argument changing between replays.
struct DevState {
    double norm_sum;        // sum of every entry of the first lag+1 pushed vectors
    float scale;            // s = 2 * mean of those entries; valid once push_count >= window
    float inv_scale;
    uint32_t push_count;    // vectors pushed since reset
    uint32_t step;          // decisions made since reset (addresses the noise)
    int32_t error_flags;    // bit 0: a pushed value was not finite or not > 0; bit 1: device wait timed out; bit 2: all workers censored
    int32_t c_star;         // last decision
    int32_t code;           // 0 ok, 2 degenerate
    uint32_t ticket;        // CTAs that have finished their column sums (self-resetting)
};

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may begin while its
// predecessor in the stream is still running, once every CTA of the predecessor has called launch_dependents (or
// exited).  Whatever it does before dependency_wait() must not touch anything an earlier kernel writes; after it
// the predecessor has completed and its writes are visible.  Both are no-ops in a kernel launched the plain way.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

constexpr int kErrBadValue = 1;
constexpr int kErrTimeout = 2;
constexpr int kErrNoFinisher = 4;   // a censored push in which every worker was censored

// Model dimensions and device pointers handed to the kernels by value.
struct ModelDev {
    int N, D, H, W;          // workers, latent size, hidden width, window = lag + 1
    // encoder RNNs
    const float *Wxf, *Whf, *bf, *a0, *Wxb, *Whb, *bb, *b0;
    // guide (WzT is the transposed copy [D x H]; Wmu as loaded [D x H])
    const float *WzT, *bz, *Wmu, *bmu, *Wsig, *bsig, *z0;
    // transition (W1T transposed copy [D x H]; W2 as loaded [2D x H])
    const float *W1T, *b1, *W2, *b2;
    // emission (W3T transposed copy [D x H]; W4 as loaded [2N x H])
    const float *W3T, *b3, *W4, *b4;
};

struct NoiseKey {
    uint32_t seed_lo, seed_hi;
};

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
__host__ __device__ inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

}  // namespace cutoff
