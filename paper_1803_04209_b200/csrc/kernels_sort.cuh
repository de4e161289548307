// Per-sample sort into order statistics, the sum over samples, and the decision
// (Section 3.1.1, last paragraph: "sample, sort, record, repeat"; Section 3: Omega(c) = c / x~_(c)).
#pragma once
#include <cfloat>
#include <cmath>
#include "common.cuh"

namespace cutoff {

// Key types of the sorting network: float for the decision path; a 64-bit composite
// (order-preserving key bits, original position) for the permutation test hook.
template <typename T> struct KeyOps;
template <> struct KeyOps<float> {
    static __device__ __forceinline__ float lo(float a, float b) { return fminf(a, b); }
    static __device__ __forceinline__ float hi(float a, float b) { return fmaxf(a, b); }
    static __device__ __forceinline__ float pad() { return INFINITY; }
    static __device__ __forceinline__ float shfl_xor(float v, int mask) { return __shfl_xor_sync(0xffffffffu, v, mask); }
};
template <> struct KeyOps<unsigned long long> {
    using T = unsigned long long;
    static __device__ __forceinline__ T lo(T a, T b) { return a < b ? a : b; }
    static __device__ __forceinline__ T hi(T a, T b) { return a < b ? b : a; }
    static __device__ __forceinline__ T pad() { return ~0ull; }
    static __device__ __forceinline__ T shfl_xor(T v, int mask) { return __shfl_xor_sync(0xffffffffu, v, mask); }
};

// Bitonic sorting network over 32*E keys held by one warp, E keys per lane, key index
// idx = lane*E + r ("blocked").  Exchange distances below E stay inside a lane's registers;
// distances of E and more are lane exchanges by shuffle.  Ascending on exit.
template <typename T, int E>
__device__ __forceinline__ void warp_bitonic_sort(T (&v)[E], int lane) {
    using Ops = KeyOps<T>;
#pragma unroll
    for (int k = 2; k <= 32 * E; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j < E) {
#pragma unroll
                for (int r = 0; r < E; ++r) {
                    if ((r & j) == 0) {
                        const bool up = (k < E) ? ((r & k) == 0) : (((lane * E) & k) == 0);
                        const T a = v[r], b = v[r | j];
                        const T lo = Ops::lo(a, b), hi = Ops::hi(a, b);
                        v[r] = up ? lo : hi;
                        v[r | j] = up ? hi : lo;
                    }
                }
            } else {
                const int lane_mask = j / E;
                const bool lower = (lane & lane_mask) == 0;
                const bool up = ((lane * E) & k) == 0;
                const bool keep_lo = (lower == up);
#pragma unroll
                for (int r = 0; r < E; ++r) {
                    const T other = Ops::shfl_xor(v[r], lane_mask);
                    v[r] = keep_lo ? Ops::lo(v[r], other) : Ops::hi(v[r], other);
                }
            }
        }
    }
}

// Bitonic sorting network over P keys (a power of two) in shared memory, all threads of the CTA.
template <typename T>
__device__ __forceinline__ void cta_bitonic_sort(T* s, int P) {
    using Ops = KeyOps<T>;
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int p = threadIdx.x; p < P / 2; p += blockDim.x) {
                const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));      // index with bit j clear
                const bool up = (i & k) == 0;
                const T a = s[i], b = s[i | j];
                const T lo = Ops::lo(a, b), hi = Ops::hi(a, b);
                s[i] = up ? lo : hi;
                s[i | j] = up ? hi : lo;
            }
            __syncthreads();
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Sort + accumulate, one warp per sample row, N <= 32*E.  Each warp keeps the running sum of its
// sorted rows in registers; a CTA adds its warps in a fixed order and writes one partial row.
// The network sorts any arrangement, so rows are loaded coalesced (element r*32 + lane).
// ---------------------------------------------------------------------------------------------
constexpr int kSortWarps = 8;

template <int E>
__global__ void __launch_bounds__(kSortWarps * 32) k_sort_sum_warp(const float* __restrict__ x, int ldx, int N,
                                                                    int count, float* __restrict__ partial) {
    __shared__ float stage[kSortWarps][32 * E];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float acc[E];
#pragma unroll
    for (int r = 0; r < E; ++r) acc[r] = 0.0f;
    for (int row = blockIdx.x * kSortWarps + warp; row < count; row += gridDim.x * kSortWarps) {
        const float* src = x + static_cast<size_t>(row) * ldx;
        float v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * 32 + lane;
            v[r] = e < N ? src[e] : INFINITY;
        }
        warp_bitonic_sort<float, E>(v, lane);
#pragma unroll
        for (int r = 0; r < E; ++r) acc[r] += v[r];
    }
#pragma unroll
    for (int r = 0; r < E; ++r) stage[warp][lane * E + r] = acc[r];
    __syncthreads();
    for (int j = threadIdx.x; j < N; j += kSortWarps * 32) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < kSortWarps; ++w) s += stage[w][j];
        partial[static_cast<size_t>(blockIdx.x) * N + j] = s;
    }
}

// ---------------------------------------------------------------------------------------------
// Sort + accumulate for wide rows (N > 1024): one CTA per row, the row in shared memory.
// ---------------------------------------------------------------------------------------------
constexpr int kSortCtaThreads = 512;

__global__ void __launch_bounds__(kSortCtaThreads) k_sort_sum_cta(const float* __restrict__ x, int ldx, int N, int P,
                                                                   int count, float* __restrict__ partial) {
    extern __shared__ float srow[];
    float acc[8];           // P <= 4096 -> at most 8 positions per thread
#pragma unroll
    for (int a = 0; a < 8; ++a) acc[a] = 0.0f;
    for (int row = blockIdx.x; row < count; row += gridDim.x) {
        const float* src = x + static_cast<size_t>(row) * ldx;
        for (int e = threadIdx.x; e < P; e += kSortCtaThreads) srow[e] = e < N ? src[e] : INFINITY;
        __syncthreads();
        cta_bitonic_sort<float>(srow, P);
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            const int e = a * kSortCtaThreads + threadIdx.x;
            if (e < N) acc[a] += srow[e];
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        const int e = a * kSortCtaThreads + threadIdx.x;
        if (e < N) partial[static_cast<size_t>(blockIdx.x) * N + e] = acc[a];
    }
}

// ---------------------------------------------------------------------------------------------
// Column sums of the partial rows, in a fixed order, in double.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_colsum(const float* __restrict__ partial, int n_part, int N,
                                                double* __restrict__ sums) {
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= N) return;
    double s = 0.0;
    for (int p = 0; p < n_part; ++p) s += static_cast<double>(partial[static_cast<size_t>(p) * N + j]);
    sums[j] = s;
}

// ---------------------------------------------------------------------------------------------
// Decision: E_j = s * sums_j / S (seconds), Omega(c) = c / E_c (minus infinity where E_c <= 0),
// c* = the largest c attaining the maximum; c* = N and code 2 if no c is admissible.
// One CTA.  Advances the decision counter when asked to.
// ---------------------------------------------------------------------------------------------
constexpr int kDecideThreads = 1024;

__global__ void __launch_bounds__(kDecideThreads) k_decide(const double* __restrict__ sums, int N, double inv_samples,
                                                            DevState* st, int advance, float* __restrict__ e_out,
                                                            float* __restrict__ omega_out) {
    __shared__ double best_val[kDecideThreads / 32];
    __shared__ int best_idx[kDecideThreads / 32];
    const double scale = static_cast<double>(st->scale);
    double bv = -INFINITY;
    int bi = 0;                                   // 0 = nothing admissible yet
    for (int j = threadIdx.x; j < N; j += kDecideThreads) {
        const double e = scale * sums[j] * inv_samples;
        const double om = e > 0.0 ? static_cast<double>(j + 1) / e : -INFINITY;
        e_out[j] = static_cast<float>(e);
        omega_out[j] = static_cast<float>(om);
        if (om > -INFINITY && om >= bv) { bv = om; bi = j + 1; }   // j ascends per thread: ties -> larger c
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        if (oi != 0 && (bi == 0 || ov > bv || (ov == bv && oi > bi))) { bv = ov; bi = oi; }
    }
    if (lane == 0) { best_val[warp] = bv; best_idx[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kDecideThreads / 32; ++w) {
            const double ov = best_val[w];
            const int oi = best_idx[w];
            if (oi != 0 && (bi == 0 || ov > bv || (ov == bv && oi > bi))) { bv = ov; bi = oi; }
        }
        st->c_star = bi == 0 ? N : bi;
        st->code = bi == 0 ? 2 : 0;
        if (advance) st->step += 1;
    }
}

// ---------------------------------------------------------------------------------------------
// Test hook: sort caller rows as (key, original position) pairs with the same networks.
// A float maps to an order-preserving unsigned integer (flip all bits of negatives, the sign bit
// of the others); the composite key << 32 | position orders equal keys by position.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long make_composite(float key, int pos) {
    uint32_t b = __float_as_uint(key);
    b = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    return (static_cast<unsigned long long>(b) << 32) | static_cast<uint32_t>(pos);
}
__device__ __forceinline__ float composite_key(unsigned long long c) {
    uint32_t b = static_cast<uint32_t>(c >> 32);
    b = (b & 0x80000000u) ? (b & 0x7fffffffu) : ~b;
    return __uint_as_float(b);
}

template <int E>
__global__ void __launch_bounds__(kSortWarps * 32) k_debug_sort_warp(const float* __restrict__ rows, int n, int n_rows,
                                                                      float* __restrict__ keys, int* __restrict__ perm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int row = blockIdx.x * kSortWarps + warp; row < n_rows; row += gridDim.x * kSortWarps) {
        unsigned long long v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * 32 + lane;
            v[r] = e < n ? make_composite(rows[static_cast<size_t>(row) * n + e], e) : ~0ull;
        }
        warp_bitonic_sort<unsigned long long, E>(v, lane);
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int idx = lane * E + r;
            if (idx < n) {
                keys[static_cast<size_t>(row) * n + idx] = composite_key(v[r]);
                perm[static_cast<size_t>(row) * n + idx] = static_cast<int>(v[r] & 0xffffffffu);
            }
        }
    }
}

__global__ void __launch_bounds__(kSortCtaThreads) k_debug_sort_cta(const float* __restrict__ rows, int n, int P,
                                                                     int n_rows, float* __restrict__ keys,
                                                                     int* __restrict__ perm) {
    extern __shared__ unsigned long long scomp[];
    for (int row = blockIdx.x; row < n_rows; row += gridDim.x) {
        for (int e = threadIdx.x; e < P; e += kSortCtaThreads)
            scomp[e] = e < n ? make_composite(rows[static_cast<size_t>(row) * n + e], e) : ~0ull;
        __syncthreads();
        cta_bitonic_sort<unsigned long long>(scomp, P);
        for (int e = threadIdx.x; e < n; e += kSortCtaThreads) {
            keys[static_cast<size_t>(row) * n + e] = composite_key(scomp[e]);
            perm[static_cast<size_t>(row) * n + e] = static_cast<int>(scomp[e] & 0xffffffffu);
        }
        __syncthreads();
    }
}

}  // namespace cutoff
