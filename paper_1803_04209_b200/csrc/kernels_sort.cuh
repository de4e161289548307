// Per-sample sort into order statistics, the sum over samples, and the decision
// (Section 3.1.1, last paragraph: "sample, sort, record, repeat"; Section 3: Omega(c) = c / x~_(c)).
#pragma once
#include <cfloat>
#include <cmath>
#include "async.cuh"
#include "common.cuh"

namespace cutoff {

// Key types of the sorting network: float for the decision path; a 64-bit composite
// (order-preserving key bits, original position) for the permutation test hook.
// Besides min and max each type has an order-reversing involution ("reverse": negation for
// floats, bitwise complement for unsigned integers).  A lane that has to keep the LARGER key of
// an exchange holds its keys reversed, so that every lane executes the same min(own, reverse(other)).
template <typename T> struct KeyOps;
template <> struct KeyOps<float> {
    using Flip = float;                                   // +1: as is, -1: reversed
    static __device__ __forceinline__ float lo(float a, float b) { return fminf(a, b); }
    static __device__ __forceinline__ float hi(float a, float b) { return fmaxf(a, b); }
    static __device__ __forceinline__ float pad() { return INFINITY; }
    static __device__ __forceinline__ float shfl_xor(float v, int mask) { return __shfl_xor_sync(0xffffffffu, v, mask); }
    static __device__ __forceinline__ Flip identity() { return 1.0f; }
    static __device__ __forceinline__ Flip flip_if(bool reversed) { return reversed ? -1.0f : 1.0f; }
    static __device__ __forceinline__ Flip combine(Flip a, Flip b) { return a * b; }
    static __device__ __forceinline__ float apply(float v, Flip f) { return v * f; }
    static __device__ __forceinline__ float reverse(float v) { return -v; }
};
template <> struct KeyOps<unsigned long long> {
    using T = unsigned long long;
    using Flip = unsigned long long;                      // 0: as is, ~0: reversed
    static __device__ __forceinline__ T lo(T a, T b) { return a < b ? a : b; }
    static __device__ __forceinline__ T hi(T a, T b) { return a < b ? b : a; }
    static __device__ __forceinline__ T pad() { return ~0ull; }
    static __device__ __forceinline__ T shfl_xor(T v, int mask) { return __shfl_xor_sync(0xffffffffu, v, mask); }
    static __device__ __forceinline__ Flip identity() { return 0ull; }
    static __device__ __forceinline__ Flip flip_if(bool reversed) { return reversed ? ~0ull : 0ull; }
    static __device__ __forceinline__ Flip combine(Flip a, Flip b) { return a ^ b; }
    static __device__ __forceinline__ T apply(T v, Flip f) { return v ^ f; }
    static __device__ __forceinline__ T reverse(T v) { return ~v; }
};

// Sorting network over 32*E keys held by one warp, E keys per lane, key index idx = lane*E + r
// ("blocked"): every lane first sorts its own keys (lane_sort), then bitonic merges of width
// k = 2E .. 32E combine them.  Every merge of width k starts with the mirror exchange
// idx <-> idx ^ (k-1) and continues with half-cleaners idx <-> idx ^ j, j = k/4 .. 1; the lower
// index always keeps the smaller key, so no exchange depends on a direction flag.  Distances
// below E stay inside a lane's registers (one min and one max per pair); distances of E and more
// are lane exchanges by shuffle in the reversed-key form described above (one min per key; the
// reversals are multiplications by +-1, which run on the otherwise idle FMA pipe).
// The register stages are always unrolled (their register indices must be static); the merges across
// lanes are unrolled too, or (LOOPED) a run-time loop over the merge width.
// Ascending on exit.

// Half-cleaners idx <-> idx ^ j for j = E/2 .. 1: inside a lane's registers.
template <typename T, int E>
__device__ __forceinline__ void lane_half_cleaners(T (&v)[E]) {
    using Ops = KeyOps<T>;
#pragma unroll
    for (int j = E / 2; j > 0; j >>= 1) {
#pragma unroll
        for (int r = 0; r < E; ++r) {
            if ((r & j) == 0) {
                const T a = v[r], b = v[r | j];
                v[r] = Ops::lo(a, b);
                v[r | j] = Ops::hi(a, b);
            }
        }
    }
}

// A lane's own E keys, ascending: Batcher's odd-even merge sort (Batcher, "Sorting networks and their
// applications", 1968), which needs fewer compare-exchanges than the bitonic network (191 against 240 for
// 32 keys) at the same depth.  All indices are compile-time constants, so the keys stay in registers.
template <typename T, int E, int LO, int N, int R>
__device__ __forceinline__ void lane_odd_even_merge(T (&v)[E]) {
    using Ops = KeyOps<T>;
    constexpr int M = 2 * R;
    if constexpr (M < N) {
        lane_odd_even_merge<T, E, LO, N, M>(v);          // even subsequence
        lane_odd_even_merge<T, E, LO + R, N, M>(v);      // odd subsequence
#pragma unroll
        for (int i = LO + R; i + R < LO + N; i += M) {
            const T a = v[i], b = v[i + R];
            v[i] = Ops::lo(a, b);
            v[i + R] = Ops::hi(a, b);
        }
    } else {
        const T a = v[LO], b = v[LO + R];
        v[LO] = Ops::lo(a, b);
        v[LO + R] = Ops::hi(a, b);
    }
}
template <typename T, int E, int LO, int N>
__device__ __forceinline__ void lane_sort(T (&v)[E]) {
    if constexpr (N > 1) {
        lane_sort<T, E, LO, N / 2>(v);
        lane_sort<T, E, LO + N / 2, N / 2>(v);
        lane_odd_even_merge<T, E, LO, N, 1>(v);
    }
}

// Half-cleaners between lanes, lane distances first_mask, first_mask/2, .. 1, in the reversed-key form.
// `cur` is the form the lane's keys are held in on entry; plain keys on exit.
template <typename T, int E>
__device__ __forceinline__ void shuffle_half_cleaners(T (&v)[E], int lane, int first_mask, typename KeyOps<T>::Flip cur) {
    using Ops = KeyOps<T>;
#pragma unroll 1
    for (int lane_mask = first_mask; lane_mask > 0; lane_mask >>= 1) {
        const typename Ops::Flip want = Ops::flip_if((lane & lane_mask) != 0);
        const typename Ops::Flip f = Ops::combine(want, cur);
        cur = want;
#pragma unroll
        for (int r = 0; r < E; ++r) v[r] = Ops::apply(v[r], f);
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const T other = Ops::shfl_xor(v[r], lane_mask);
            v[r] = Ops::lo(v[r], Ops::reverse(other));
        }
    }
#pragma unroll
    for (int r = 0; r < E; ++r) v[r] = Ops::apply(v[r], cur);
}

template <typename T, int E, bool LOOPED = false>
__device__ __forceinline__ void warp_bitonic_sort(T (&v)[E], int lane) {
    using Ops = KeyOps<T>;
    lane_sort<T, E, 0, E>(v);                // each lane sorts its own keys
    if constexpr (!LOOPED) {
        // merges of width 2E .. 32E, m = lanes per merge, fully unrolled: the fastest form when one warp sorts a row
#pragma unroll
        for (int m = 2; m <= 32; m <<= 1) {
            typename Ops::Flip cur = Ops::flip_if((lane & (m >> 1)) != 0);
#pragma unroll
            for (int r = 0; r < E; ++r) v[r] = Ops::apply(v[r], cur);
            T other[E];
#pragma unroll
            for (int r = 0; r < E; ++r) other[r] = Ops::shfl_xor(v[E - 1 - r], m - 1);
#pragma unroll
            for (int r = 0; r < E; ++r) v[r] = Ops::lo(v[r], Ops::reverse(other[r]));
#pragma unroll
            for (int lane_mask = m >> 2; lane_mask > 0; lane_mask >>= 1) {
                const typename Ops::Flip want = Ops::flip_if((lane & lane_mask) != 0);
                const typename Ops::Flip f = Ops::combine(want, cur);
                cur = want;
#pragma unroll
                for (int r = 0; r < E; ++r) v[r] = Ops::apply(v[r], f);
#pragma unroll
                for (int r = 0; r < E; ++r) {
                    const T o = Ops::shfl_xor(v[r], lane_mask);
                    v[r] = Ops::lo(v[r], Ops::reverse(o));
                }
            }
#pragma unroll
            for (int r = 0; r < E; ++r) v[r] = Ops::apply(v[r], cur);
            lane_half_cleaners<T, E>(v);
        }
    } else {
    // the same merges as a run-time loop whose body serves all five widths: a fraction of the code, for the
    // kernels in which several warps share a row (unrolled, their code overflows the instruction cache)
#pragma unroll 1
    for (int m = 2; m <= 32; m <<= 1) {
        // mirror exchange idx <-> idx ^ (mE - 1): lane ^ (m-1), register E-1-r
        const typename Ops::Flip cur = Ops::flip_if((lane & (m >> 1)) != 0);
#pragma unroll
        for (int r = 0; r < E; ++r) v[r] = Ops::apply(v[r], cur);
        T other[E];
#pragma unroll
        for (int r = 0; r < E; ++r) other[r] = Ops::shfl_xor(v[E - 1 - r], m - 1);
#pragma unroll
        for (int r = 0; r < E; ++r) v[r] = Ops::lo(v[r], Ops::reverse(other[r]));
        shuffle_half_cleaners<T, E>(v, lane, m >> 2, cur);
        lane_half_cleaners<T, E>(v);
    }
    }
}

// The half-cleaners idx <-> idx ^ j for j = 16E .. 1 of one merge, inside a warp: what remains of a
// merge wider than the warp once its cross-warp exchanges are done.  Plain keys in, plain keys out.
template <typename T, int E>
__device__ __forceinline__ void warp_half_cleaners(T (&v)[E], int lane) {
    shuffle_half_cleaners<T, E>(v, lane, 16, KeyOps<T>::identity());
    lane_half_cleaners<T, E>(v);
}

// Bitonic sorting network over WPR * 1024 keys held by the WPR warps of a CTA, 32 keys per lane,
// key index idx = (warp * 32 + lane) * 32 + r.  Each warp first sorts its 1024 keys in registers
// and by shuffles; the merges of width 2048 and 4096 then start with exchanges between warps (one
// for 2048, two for 4096), which go through shared memory (`xch`, WPR * 1024 keys, stored as
// [register][thread] so that both the writes and the partner reads are conflict-free), and finish
// inside the warps.  All threads of the CTA must call it.  Ascending on exit.
template <typename T, int WPR>
__device__ __forceinline__ void cta_bitonic_sort(T (&v)[32], T* xch) {
    using Ops = KeyOps<T>;
    constexpr int E = 32, T_ = WPR * 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    warp_bitonic_sort<T, E, true>(v, lane);
#pragma unroll 1
    for (int k = 2; k <= WPR; k <<= 1) {                 // merge width in warps
        // mirror exchange: idx <-> idx ^ (k*1024 - 1)
        {
#pragma unroll
            for (int r = 0; r < E; ++r) xch[r * T_ + threadIdx.x] = v[r];
            __syncthreads();
            const int partner = ((warp ^ (k - 1)) << 5) | (lane ^ 31);
            if ((warp & (k >> 1)) == 0) {
#pragma unroll
                for (int r = 0; r < E; ++r) v[r] = Ops::lo(v[r], xch[(E - 1 - r) * T_ + partner]);
            } else {
#pragma unroll
                for (int r = 0; r < E; ++r) v[r] = Ops::hi(v[r], xch[(E - 1 - r) * T_ + partner]);
            }
            __syncthreads();
        }
        // half-cleaners between warps: idx <-> idx ^ (j*1024), j = k/4 .. 1
#pragma unroll 1
        for (int j = k >> 2; j > 0; j >>= 1) {
#pragma unroll
            for (int r = 0; r < E; ++r) xch[r * T_ + threadIdx.x] = v[r];
            __syncthreads();
            const int partner = ((warp ^ j) << 5) | lane;
            if ((warp & j) == 0) {
#pragma unroll
                for (int r = 0; r < E; ++r) v[r] = Ops::lo(v[r], xch[r * T_ + partner]);
            } else {
#pragma unroll
                for (int r = 0; r < E; ++r) v[r] = Ops::hi(v[r], xch[r * T_ + partner]);
            }
            __syncthreads();
        }
        warp_half_cleaners<T, E>(v, lane);
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
// The same, with the rows brought into shared memory by the bulk-copy engine one row ahead of the
// sort: each warp owns two row buffers and two mbarriers; while it sorts row i, row i+1 is in
// flight, so the sort never waits on global memory.  Needs ldx*4 and the matrix base to be
// multiples of 16 bytes.  Dynamic shared memory: kSortWarps * 2 * ldx floats (reused for the CTA
// reduction at the end), then 2 * kSortWarps mbarriers and the abort flag.
// ---------------------------------------------------------------------------------------------
template <int E>
inline size_t sort_tma_smem_bytes(int ldx) {
    const size_t rows = static_cast<size_t>(kSortWarps) * 2 * ldx * sizeof(float);
    const size_t stage = static_cast<size_t>(kSortWarps) * 32 * E * sizeof(float);
    return (rows > stage ? rows : stage) + 16 * kSortWarps + 16;
}

template <int E, bool SQ>
__global__ void __launch_bounds__(kSortWarps * 32) k_sort_sum_tma(const float* __restrict__ x, int ldx, int N, int count,
                                                                   float* __restrict__ partial,
                                                                   float* __restrict__ partial_sq, DevState* st) {
    using namespace cutoff::async;
    extern __shared__ __align__(16) float sm_sort[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t row_floats = static_cast<size_t>(kSortWarps) * 2 * ldx;
    const size_t stage_floats = static_cast<size_t>(kSortWarps) * 32 * E;
    const size_t data_floats = row_floats > stage_floats ? row_floats : stage_floats;
    const uint32_t bars = smem_u32(sm_sort + data_floats);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm_sort + data_floats + 4 * kSortWarps);
    float* const buf0 = sm_sort + static_cast<size_t>(warp) * 2 * ldx;      // buffer b = buf0 + b*ldx
    const uint32_t bar0 = bars + 16u * warp;                                // barrier b = bar0 + 8*b
    const uint32_t row_bytes = static_cast<uint32_t>(ldx) * 4u;
    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8u, 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    __syncthreads();
    dependency_wait();            // the sample matrix is an earlier kernel's
    launch_dependents();

    float acc[E], acc_sq[SQ ? E : 1];
#pragma unroll
    for (int r = 0; r < E; ++r) acc[r] = 0.0f;
#pragma unroll
    for (int r = 0; r < (SQ ? E : 1); ++r) acc_sq[r] = 0.0f;
    const int stride = gridDim.x * kSortWarps;
    int row = blockIdx.x * kSortWarps + warp;
    if (row < count && lane == 0) {
        mbar_arrive_expect_tx(bar0, row_bytes);
        bulk_load_1d(smem_u32(buf0), x + static_cast<size_t>(row) * ldx, row_bytes, bar0);
    }
    bool aborted = false;
    // iteration `it` uses buffer it & 1 for the (it >> 1)-th time: its barrier completes phase (it >> 1) & 1
    for (uint32_t it = 0; row < count; row += stride, ++it) {
        const uint32_t b = it & 1u, par = (it >> 1) & 1u;
        const int next = row + stride;
        if (next < count) {
            // the other buffer was read in the previous iteration: order those reads before the engine's write
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                const uint32_t nb = b ^ 1u;
                mbar_arrive_expect_tx(bar0 + 8u * nb, row_bytes);
                bulk_load_1d(smem_u32(buf0 + nb * ldx), x + static_cast<size_t>(next) * ldx, row_bytes, bar0 + 8u * nb);
            }
        }
        if (!mbar_wait(bar0 + 8u * b, par, abort_flag, st)) {
            // wind down: give both copies that may still be in flight time to land (bounded)
            mbar_wait_quiet(bar0 + 8u * b, par);
            if (next < count) mbar_wait_quiet(bar0 + 8u * (b ^ 1u), ((it + 1u) >> 1) & 1u);
            aborted = true;
            break;
        }
        const float* src = buf0 + b * ldx;
        float v[E];
        if (N == 32 * E) {                             // a full row: no padding keys to put in
#pragma unroll
            for (int r = 0; r < E; ++r) v[r] = src[r * 32 + lane];
        } else {
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const int e = r * 32 + lane;
                v[r] = e < N ? src[e] : INFINITY;
            }
        }
        __syncwarp();
        warp_bitonic_sort<float, E>(v, lane);
#pragma unroll
        for (int r = 0; r < E; ++r) acc[r] += v[r];
        if (SQ) {
#pragma unroll
            for (int r = 0; r < E; ++r) acc_sq[SQ ? r : 0] = fmaf(v[r], v[r], acc_sq[SQ ? r : 0]);
        }
    }
    (void)aborted;
    __syncthreads();                                   // all row buffers are dead: reuse them as the stage
    float* stage = sm_sort;
#pragma unroll
    for (int r = 0; r < E; ++r) stage[warp * 32 * E + lane * E + r] = acc[r];
    __syncthreads();
    for (int j = threadIdx.x; j < N; j += kSortWarps * 32) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < kSortWarps; ++w) s += stage[w * 32 * E + j];
        partial[static_cast<size_t>(blockIdx.x) * N + j] = s;
    }
    if (SQ) {                                          // the same reduction for the sums of squares
        __syncthreads();
#pragma unroll
        for (int r = 0; r < E; ++r) stage[warp * 32 * E + lane * E + r] = acc_sq[SQ ? r : 0];
        __syncthreads();
        for (int j = threadIdx.x; j < N; j += kSortWarps * 32) {
            float s = 0.0f;
#pragma unroll
            for (int w = 0; w < kSortWarps; ++w) s += stage[w * 32 * E + j];
            partial_sq[static_cast<size_t>(blockIdx.x) * N + j] = s;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Sort + accumulate for wide rows (1024 < N <= 4096): a CTA of WPR = P/1024 warps per row, keys in
// registers, running sums in registers, one partial row per CTA.
// ---------------------------------------------------------------------------------------------
template <int WPR, bool SQ>
__global__ void __launch_bounds__(WPR * 32, SQ ? 3 : 4) k_sort_sum_cta(const float* __restrict__ x, int ldx, int N, int count,
                                                            float* __restrict__ partial, float* __restrict__ partial_sq) {
    __shared__ float xch[WPR * 1024];
    constexpr int E = 32, T_ = WPR * 32;
    float acc[E], acc_sq[SQ ? E : 1];
#pragma unroll
    for (int r = 0; r < E; ++r) acc[r] = 0.0f;
#pragma unroll
    for (int r = 0; r < (SQ ? E : 1); ++r) acc_sq[r] = 0.0f;
    for (int row = blockIdx.x; row < count; row += gridDim.x) {
        const float* src = x + static_cast<size_t>(row) * ldx;
        float v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * T_ + threadIdx.x;            // any arrangement sorts; this one loads coalesced
            v[r] = e < N ? src[e] : INFINITY;
        }
        cta_bitonic_sort<float, WPR>(v, xch);
#pragma unroll
        for (int r = 0; r < E; ++r) acc[r] += v[r];
        if (SQ) {
#pragma unroll
            for (int r = 0; r < E; ++r) acc_sq[SQ ? r : 0] = fmaf(v[r], v[r], acc_sq[SQ ? r : 0]);
        }
    }
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const int idx = threadIdx.x * E + r;
        if (idx < N) {
            partial[static_cast<size_t>(blockIdx.x) * N + idx] = acc[r];
            if (SQ) partial_sq[static_cast<size_t>(blockIdx.x) * N + idx] = acc_sq[SQ ? r : 0];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Decision: E_j = s * sums_j / S (seconds), Omega(c) = c / E_c (minus infinity where E_c <= 0),
// c* = the largest c attaining the maximum; c* = N and code 2 if no c is admissible.
// Executed by one whole CTA of THREADS threads.  Advances the decision counter when asked to.
// ---------------------------------------------------------------------------------------------
template <int THREADS>
__device__ __forceinline__ void decide_block(const double* sums, int N, double inv_samples, DevState* st, int advance,
                                             float* __restrict__ e_out, float* __restrict__ omega_out) {
    __shared__ double best_val[THREADS / 32];
    __shared__ int best_idx[THREADS / 32];
    const double scale = static_cast<double>(st->scale);
    double bv = -INFINITY;
    int bi = 0;                                   // 0 = nothing admissible yet
    for (int j = threadIdx.x; j < N; j += THREADS) {
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
        for (int w = 1; w < THREADS / 32; ++w) {
            const double ov = best_val[w];
            const int oi = best_idx[w];
            if (oi != 0 && (bi == 0 || ov > bv || (ov == bv && oi > bi))) { bv = ov; bi = oi; }
        }
        st->c_star = bi == 0 ? N : bi;
        st->code = bi == 0 ? 2 : 0;
        if (advance) st->step += 1;
    }
}

constexpr int kDecideThreads = 1024;

__global__ void __launch_bounds__(kDecideThreads) k_decide(const double* __restrict__ sums, int N, double inv_samples,
                                                            DevState* st, int advance, float* __restrict__ e_out,
                                                            float* __restrict__ omega_out) {
    decide_block<kDecideThreads>(sums, N, inv_samples, st, advance, e_out, omega_out);
}

// ---------------------------------------------------------------------------------------------
// Column sums of the partial rows, in a fixed order, in double, followed by the decision in the
// CTA that finishes last (a ticket counter in the device state; nobody waits on anybody); decide = 0
// stops after the sums.
// A CTA covers 32 columns with 32 row slices; slice s adds rows s, s+32, ...; the slices are then
// added in order.
// ---------------------------------------------------------------------------------------------
constexpr int kColsumSlices = 32;
constexpr int kColsumThreads = 32 * kColsumSlices;

__global__ void __launch_bounds__(kColsumThreads) k_colsum_decide(const float* __restrict__ partial, int n_part, int N,
                                                                   double* sums, double inv_samples, DevState* st,
                                                                   float* __restrict__ e_out, float* __restrict__ omega_out,
                                                                   const float* __restrict__ partial_sq,
                                                                   float* __restrict__ std_out, int decide) {
    __shared__ double red[kColsumSlices][32];
    __shared__ bool is_last;
    dependency_wait();            // the partial rows are an earlier kernel's
    const int col = blockIdx.x * 32 + (threadIdx.x & 31), slice = threadIdx.x >> 5;
    if (partial_sq) {
        // spread of each order statistic over the samples: sqrt(E[x^2] - E[x]^2), in seconds
        double s1 = 0.0, s2 = 0.0;
        if (col < N)
            for (int p = slice; p < n_part; p += kColsumSlices) {
                s1 += static_cast<double>(partial[static_cast<size_t>(p) * N + col]);
                s2 += static_cast<double>(partial_sq[static_cast<size_t>(p) * N + col]);
            }
        red[slice][threadIdx.x & 31] = s1;
        __syncthreads();
        double t1 = 0.0;
        if (slice == 0)
            for (int k = 0; k < kColsumSlices; ++k) t1 += red[k][threadIdx.x];
        __syncthreads();
        red[slice][threadIdx.x & 31] = s2;
        __syncthreads();
        if (slice == 0 && col < N) {
            double t2 = 0.0;
            for (int k = 0; k < kColsumSlices; ++k) t2 += red[k][threadIdx.x];
            const double mean = t1 * inv_samples, var = t2 * inv_samples - mean * mean;
            std_out[col] = static_cast<float>(static_cast<double>(st->scale) * sqrt(var > 0.0 ? var : 0.0));
        }
        __syncthreads();
    }
    double s = 0.0;
    if (col < N) {
        int p = slice;
        for (; p + 3 * kColsumSlices < n_part; p += 4 * kColsumSlices) {        // four loads in flight
            const float a = partial[static_cast<size_t>(p) * N + col];
            const float b = partial[static_cast<size_t>(p + kColsumSlices) * N + col];
            const float c = partial[static_cast<size_t>(p + 2 * kColsumSlices) * N + col];
            const float d = partial[static_cast<size_t>(p + 3 * kColsumSlices) * N + col];
            s += static_cast<double>(a);
            s += static_cast<double>(b);
            s += static_cast<double>(c);
            s += static_cast<double>(d);
        }
        for (; p < n_part; p += kColsumSlices) s += static_cast<double>(partial[static_cast<size_t>(p) * N + col]);
    }
    red[slice][threadIdx.x & 31] = s;
    __syncthreads();
    if (slice == 0 && col < N) {
        double total = 0.0;
#pragma unroll
        for (int k = 0; k < kColsumSlices; ++k) total += red[k][threadIdx.x];
        sums[col] = total;
    }
    if (!decide) return;                                // only the sums were asked for
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t ticket = atomicAdd(&st->ticket, 1u);
        is_last = ticket == gridDim.x - 1;
        if (is_last) st->ticket = 0;
    }
    __syncthreads();
    if (is_last) {
        __threadfence();
        decide_block<kColsumThreads>(sums, N, inv_samples, st, 1, e_out, omega_out);
    }
}

// Plain column sums of partial rows (fixed order, double): one thread per column.  With `accumulate` the
// result is added to what sums already holds.
__global__ void __launch_bounds__(256) k_colsum(const float* __restrict__ partial, int n_part, int N,
                                                double* __restrict__ sums, int accumulate) {
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= N) return;
    double s = accumulate ? sums[j] : 0.0;
    for (int p = 0; p < n_part; ++p) s += static_cast<double>(partial[static_cast<size_t>(p) * N + j]);
    sums[j] = s;
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

template <int WPR>
__global__ void __launch_bounds__(WPR * 32) k_debug_sort_cta(const float* __restrict__ rows, int n, int n_rows,
                                                              float* __restrict__ keys, int* __restrict__ perm) {
    __shared__ unsigned long long xch[WPR * 1024];
    constexpr int E = 32, T_ = WPR * 32;
    for (int row = blockIdx.x; row < n_rows; row += gridDim.x) {
        unsigned long long v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * T_ + threadIdx.x;
            v[r] = e < n ? make_composite(rows[static_cast<size_t>(row) * n + e], e) : ~0ull;
        }
        cta_bitonic_sort<unsigned long long, WPR>(v, xch);
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int idx = threadIdx.x * E + r;
            if (idx < n) {
                keys[static_cast<size_t>(row) * n + idx] = composite_key(v[r]);
                perm[static_cast<size_t>(row) * n + idx] = static_cast<int>(v[r] & 0xffffffffu);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Test hook: the float instantiation of the networks -- the one the decision path runs -- applied to
// caller rows, the sorted rows written out instead of summed.  Rows are loaded, padded and sorted
// exactly as k_sort_sum_* do it.
// ---------------------------------------------------------------------------------------------
template <int E>
__global__ void __launch_bounds__(kSortWarps * 32) k_debug_sort_values_warp(const float* __restrict__ rows, int n, int n_rows,
                                                                             float* __restrict__ keys) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int row = blockIdx.x * kSortWarps + warp; row < n_rows; row += gridDim.x * kSortWarps) {
        float v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * 32 + lane;
            v[r] = e < n ? rows[static_cast<size_t>(row) * n + e] : INFINITY;
        }
        warp_bitonic_sort<float, E>(v, lane);
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int idx = lane * E + r;
            if (idx < n) keys[static_cast<size_t>(row) * n + idx] = v[r];
        }
    }
}

template <int WPR>
__global__ void __launch_bounds__(WPR * 32) k_debug_sort_values_cta(const float* __restrict__ rows, int n, int n_rows,
                                                                     float* __restrict__ keys) {
    __shared__ float xch[WPR * 1024];
    constexpr int E = 32, T_ = WPR * 32;
    for (int row = blockIdx.x; row < n_rows; row += gridDim.x) {
        float v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * T_ + threadIdx.x;
            v[r] = e < n ? rows[static_cast<size_t>(row) * n + e] : INFINITY;
        }
        cta_bitonic_sort<float, WPR>(v, xch);
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int idx = threadIdx.x * E + r;
            if (idx < n) keys[static_cast<size_t>(row) * n + idx] = v[r];
        }
    }
}

}  // namespace cutoff
