// Evaluation of cutoff rules on recorded run-times (Sections 3, 3.1.1 and 4.1; Fig. 2 and Fig. 4):
// per SGD step the observed run-times are sorted, then
//   Omega(c) = c / x~_(c) for every c, its maximum and the cutoff that attains it (known in hindsight only),
//   the throughput of waiting for all workers, N / x~_(N),
//   the throughput and the duration x~_(c) of the step under each of M given cutoffs;
// over a whole trace: the best static cutoff (one c for all steps), and the "order" baseline -- the cutoff
// that maximises c / E[x~_(c)] with Elfving's normal-theory expectations from the running mean and
// deviation of everything observed before the step.
#pragma once
#include <cmath>

#include "common.cuh"
#include "kernels_sort.cuh"

namespace cutoff {

// One sorted row in shared memory -> the step's scores.  Executed by `threads` consecutive threads
// (a warp or a whole CTA) whose first thread is `tid == 0`; `sync` separates its phases.
template <typename Sync>
__device__ __forceinline__ void eval_sorted_row(const float* __restrict__ sorted, int N, int tid, int threads, Sync sync,
                                                double* red_val, int* red_idx, int64_t t, int64_t T,
                                                const int32_t* __restrict__ cutoffs, int M,
                                                int32_t* __restrict__ best_c, float* __restrict__ best,
                                                float* __restrict__ all, float* __restrict__ achieved,
                                                float* __restrict__ time_at) {
    // hindsight maximum of Omega(c) = c / x~_(c); ties go to the larger c
    double bv = -INFINITY;
    int bi = 0;
    for (int j = tid; j < N; j += threads) {
        const double om = static_cast<double>(j + 1) / static_cast<double>(sorted[j]);
        if (om >= bv) { bv = om; bi = j + 1; }
    }
    red_val[tid] = bv;
    red_idx[tid] = bi;
    sync();
    if (tid == 0) {
        for (int k = 1; k < threads; ++k) {
            const double ov = red_val[k];
            const int oi = red_idx[k];
            if (oi != 0 && (ov > bv || (ov == bv && oi > bi))) { bv = ov; bi = oi; }
        }
        best_c[t] = bi;
        best[t] = static_cast<float>(bv);
        all[t] = static_cast<float>(static_cast<double>(N) / static_cast<double>(sorted[N - 1]));
    }
    for (int m = tid; m < M; m += threads) {
        int c = cutoffs[static_cast<int64_t>(m) * T + t];
        c = c < 1 ? 1 : (c > N ? N : c);
        const float x_c = sorted[c - 1];
        achieved[static_cast<int64_t>(m) * T + t] = static_cast<float>(static_cast<double>(c) / static_cast<double>(x_c));
        time_at[static_cast<int64_t>(m) * T + t] = x_c;
    }
    sync();
}

// N <= 1024: one warp per step, E = P / 32 keys per lane.
template <int E>
__global__ void __launch_bounds__(kSortWarps * 32) k_eval_trace_warp(const float* __restrict__ trace, int64_t T, int N, int ld,
                                                                      const int32_t* __restrict__ cutoffs, int M,
                                                                      int32_t* __restrict__ best_c, float* __restrict__ best,
                                                                      float* __restrict__ all, float* __restrict__ achieved,
                                                                      float* __restrict__ time_at,
                                                                      float* __restrict__ sorted_out) {
    __shared__ float rows[kSortWarps][32 * E];
    __shared__ double red_val[kSortWarps][32];
    __shared__ int red_idx[kSortWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t t = static_cast<int64_t>(blockIdx.x) * kSortWarps + warp; t < T; t += static_cast<int64_t>(gridDim.x) * kSortWarps) {
        const float* src = trace + t * ld;
        float v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * 32 + lane;
            v[r] = e < N ? src[e] : INFINITY;
        }
        warp_bitonic_sort<float, E>(v, lane);
#pragma unroll
        for (int r = 0; r < E; ++r) {
            rows[warp][lane * E + r] = v[r];
            if (sorted_out && lane * E + r < N) sorted_out[t * N + lane * E + r] = v[r];
        }
        __syncwarp();
        eval_sorted_row(rows[warp], N, lane, 32, [] { __syncwarp(); }, red_val[warp], red_idx[warp], t, T, cutoffs, M,
                        best_c, best, all, achieved, time_at);
    }
}

// 1024 < N <= 4096: a CTA of WPR warps per step.
template <int WPR>
__global__ void __launch_bounds__(WPR * 32) k_eval_trace_cta(const float* __restrict__ trace, int64_t T, int N, int ld,
                                                              const int32_t* __restrict__ cutoffs, int M,
                                                              int32_t* __restrict__ best_c, float* __restrict__ best,
                                                              float* __restrict__ all, float* __restrict__ achieved,
                                                              float* __restrict__ time_at, float* __restrict__ sorted_out) {
    __shared__ float xch[WPR * 1024];
    __shared__ double red_val[WPR * 32];
    __shared__ int red_idx[WPR * 32];
    constexpr int E = 32, T_ = WPR * 32;
    for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
        const float* src = trace + t * ld;
        float v[E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int e = r * T_ + threadIdx.x;
            v[r] = e < N ? src[e] : INFINITY;
        }
        cta_bitonic_sort<float, WPR>(v, xch);
        __syncthreads();                                   // the exchange buffer is free: it now holds the sorted row
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int idx = threadIdx.x * E + r;
            xch[idx] = v[r];
            if (sorted_out && idx < N) sorted_out[t * N + idx] = v[r];
        }
        __syncthreads();
        eval_sorted_row(xch, N, static_cast<int>(threadIdx.x), T_, [] { __syncthreads(); }, red_val, red_idx, t, T, cutoffs, M,
                        best_c, best, all, achieved, time_at);
    }
}

// Best static cutoff: argmax_c sum_t c / x~_(c)(t) over the sorted rows of a trace (ties -> larger c).
// One CTA; thread j adds column j over the steps in a fixed order.
constexpr int kStaticThreads = 1024;

__global__ void __launch_bounds__(kStaticThreads) k_best_static(const float* __restrict__ sorted, int64_t T, int N,
                                                                 int32_t* __restrict__ static_c, double* __restrict__ static_total) {
    __shared__ double val[kStaticThreads];
    __shared__ int idx[kStaticThreads];
    double bv = -INFINITY;
    int bi = 0;
    for (int j = threadIdx.x; j < N; j += kStaticThreads) {
        double s = 0.0;
        for (int64_t t = 0; t < T; ++t) s += static_cast<double>(j + 1) / static_cast<double>(sorted[t * N + j]);
        if (s >= bv) { bv = s; bi = j + 1; }
    }
    val[threadIdx.x] = bv;
    idx[threadIdx.x] = bi;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int k = 1; k < kStaticThreads; ++k)
            if (idx[k] != 0 && (val[k] > bv || (val[k] == bv && idx[k] > bi))) { bv = val[k]; bi = idx[k]; }
        *static_c = bi;
        *static_total = bv;
    }
}

// ---- the "order" baseline (Fig. 4; Elfving's formula, Section 3.1.1) ----------------------------------------
// Per-step sums of x and x^2 in double, fixed order (one CTA per step).
constexpr int kMomentThreads = 256;

__global__ void __launch_bounds__(kMomentThreads) k_step_moments(const float* __restrict__ trace, int64_t T, int N, int ld,
                                                                  double* __restrict__ sum1, double* __restrict__ sum2) {
    __shared__ double r1[kMomentThreads], r2[kMomentThreads];
    const int64_t t = blockIdx.x;
    double a = 0.0, b = 0.0;
    for (int j = threadIdx.x; j < N; j += kMomentThreads) {
        const double v = static_cast<double>(trace[t * ld + j]);
        a += v;
        b += v * v;
    }
    r1[threadIdx.x] = a;
    r2[threadIdx.x] = b;
    __syncthreads();
    for (int half = kMomentThreads / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) { r1[threadIdx.x] += r1[threadIdx.x + half]; r2[threadIdx.x] += r2[threadIdx.x + half]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { sum1[t] = r1[0]; sum2[t] = r2[0]; }
}

// Normal quantiles q_j = Phi^-1((j - pi/8) / (n - pi/4 + 1)), j = 1..n (the standard form of the fraction).
__global__ void k_elfving_quantiles(int N, double* __restrict__ q) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= N) return;
    const double pi = 3.14159265358979323846;
    q[j] = normcdfinv((static_cast<double>(j + 1) - pi / 8.0) / (static_cast<double>(N) - pi / 4.0 + 1.0));
}

// In place: sums of step t -> mean and deviation of everything observed in steps 0 .. t-1 (exclusive running sums).
__global__ void k_running_moments(int64_t T, int N, double* __restrict__ sum1, double* __restrict__ sum2) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    double a = 0.0, b = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        const double s1 = sum1[t], s2 = sum2[t];
        const double count = static_cast<double>(t) * static_cast<double>(N);
        const double mu = t > 0 ? a / count : 0.0;
        const double var = t > 0 ? b / count - mu * mu : 0.0;
        sum1[t] = mu;
        sum2[t] = sqrt(var > 0.0 ? var : 0.0);
        a += s1;
        b += s2;
    }
}

// Cutoff of step t: argmax_c c / (mu_t + sigma_t q_c) over the c with a positive expectation; ties -> larger c;
// c = N for step 0 (nothing observed yet) and when no c is admissible.  One warp per step.
__global__ void __launch_bounds__(256) k_order_cutoffs(int64_t T, int N, const double* __restrict__ mu,
                                                        const double* __restrict__ sigma, const double* __restrict__ q,
                                                        int32_t* __restrict__ cutoffs) {
    const int lane = threadIdx.x & 31;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    double bv = -INFINITY;
    int bi = 0;
    if (t > 0) {
        const double m = mu[t], s = sigma[t];
        for (int j = lane; j < N; j += 32) {
            const double e = m + s * q[j];
            if (e > 0.0) {
                const double om = static_cast<double>(j + 1) / e;
                if (om >= bv) { bv = om; bi = j + 1; }
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        if (oi != 0 && (bi == 0 || ov > bv || (ov == bv && oi > bi))) { bv = ov; bi = oi; }
    }
    if (lane == 0) cutoffs[t] = bi == 0 ? N : bi;
}

}  // namespace cutoff
