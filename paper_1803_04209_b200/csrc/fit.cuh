// Learning the model on the GPU: the one-sample, reparameterised ELBO of Section 3.1.3 for a batch of windows,
// its gradient with respect to every weight tensor (reverse mode, layer by layer), and Adam with clipping by the
// global norm (Section 4.1), for the compact networks, in fp32.
//
//   ELBO_b = sum_t  log p(x_t | z_t) + log p(z_t | z_{t-1}) - log q(z_t | z_{t-1}, x),     z_t = mu_t + sigma_t eps_t,
//   log N(y; m, exp(lv)) = -1/2 [log 2 pi + lv + (y - m)^2 exp(-lv)],   log q = sum_d -1/2 log 2 pi - log sigma_d - eps_d^2 / 2.
//
// Every product is one launch of a plain tiled fp32 GEMM with strided operands (the three orientations a dense
// layer needs: X W^T forward, dY W for the input gradient, dY^T X for the weight gradient); every reduction runs
// in a fixed order (no floating-point atomics), so a step is reproducible bit for bit.  A training step of these
// sizes is a chain of small dependent layers -- the batch is tens of windows -- so this is a correct and
// deterministic first version, not a tuned one.
#pragma once
#include <cmath>

#include "common.cuh"

namespace cutoff {
namespace fit {

constexpr float kLog2Pi = 1.8378770664093453f;

// ---- C[m][n] = (accumulate ? C[m][n] : 0) + sum_k A(m, k) B(k, n) (+ bias[n]) ------------------------------------
struct Gemm {
    const float* A; long long a_m, a_k;      // A(m, k) = A[m * a_m + k * a_k]
    const float* B; long long b_k, b_n;      // B(k, n) = B[k * b_k + n * b_n]
    float* C; long long c_m;                 // C(m, n) = C[m * c_m + n]
    const float* bias;                       // [N] or null
    int M, N, K, accumulate;
};

constexpr int kGemmTile = 32;

__global__ void __launch_bounds__(256) k_gemm(Gemm g) {
    __shared__ float As[kGemmTile][kGemmTile + 1];
    __shared__ float Bs[kGemmTile][kGemmTile + 1];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;             // 32 x 8 threads, 4 rows each
    const int m0 = blockIdx.y * kGemmTile, n0 = blockIdx.x * kGemmTile;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k0 = 0; k0 < g.K; k0 += kGemmTile) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = ty + 8 * i;
            const int m = m0 + r, k = k0 + tx;
            As[r][tx] = (m < g.M && k < g.K) ? g.A[m * g.a_m + k * g.a_k] : 0.f;
            const int kk = k0 + r, n = n0 + tx;
            Bs[r][tx] = (kk < g.K && n < g.N) ? g.B[kk * g.b_k + n * g.b_n] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kGemmTile; ++kk) {
            const float b = Bs[kk][tx];
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] = fmaf(As[ty + 8 * i][kk], b, acc[i]);
        }
        __syncthreads();
    }
    const int n = n0 + tx;
    if (n >= g.N) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i;
        if (m >= g.M) continue;
        float v = acc[i] + (g.bias ? g.bias[n] : 0.f);
        if (g.accumulate) v += g.C[m * g.c_m + n];
        g.C[m * g.c_m + n] = v;
    }
}

// ---- element-wise pieces ---------------------------------------------------------------------------------------
__device__ __forceinline__ float softplus_f(float v) { return v > 20.f ? v : log1pf(expf(v)); }
__device__ __forceinline__ float sigmoid_f(float v) { return 1.f / (1.f + expf(-v)); }

__global__ void k_relu(float* __restrict__ v, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) v[i] = fmaxf(v[i], 0.f);
}
// dst[b][j] = src[j]
__global__ void k_broadcast_rows(float* __restrict__ dst, const float* __restrict__ src, int rows, int cols) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < static_cast<long long>(rows) * cols) dst[i] = src[i % cols];
}
// d[i] *= (act[i] > 0)
__global__ void k_relu_back(float* __restrict__ d, const float* __restrict__ act, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) d[i] = act[i] > 0.f ? d[i] : 0.f;
}
// d[i] = (ga[i] + carry[i]) * (act[i] > 0)
__global__ void k_rnn_back(float* __restrict__ d, const float* __restrict__ ga, const float* __restrict__ carry,
                           const float* __restrict__ act, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) d[i] = act[i] > 0.f ? ga[i] + carry[i] : 0.f;
}
// comb = tanh(pre); h = (comb + a + b) / 3
__global__ void k_combine(const float* __restrict__ pre, const float* __restrict__ a, const float* __restrict__ b,
                          float* __restrict__ comb, float* __restrict__ h, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float c = tanhf(pre[i]);
    comb[i] = c;
    h[i] = (c + a[i] + b[i]) * (1.f / 3.f);
}
// d_h = d_h_raw / 3; g_a = g_b = d_h (h_left(t) and h_right(t) enter the ELBO only through step t); d_pre_c = d_h (1 - comb^2)
__global__ void k_combine_back(const float* __restrict__ d_h_raw, const float* __restrict__ comb, float* __restrict__ g_a,
                               float* __restrict__ g_b, float* __restrict__ d_pre_c, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float d = d_h_raw[i] * (1.f / 3.f);
    g_a[i] = d;
    g_b[i] = d;
    const float c = comb[i];
    d_pre_c[i] = d * (1.f - c * c);
}
// guide sample: sigma = softplus(pre); z = mu + sigma eps; elbo[b] += sum_d (1/2 log 2 pi + log sigma + eps^2 / 2)  (= - log q)
// one thread per window; eps is [B][W][D] and this is step t
__global__ void k_guide_sample(const float* __restrict__ mu, const float* __restrict__ pre, const float* __restrict__ eps,
                               int eps_stride, float* __restrict__ sigma, float* __restrict__ z, float* __restrict__ elbo,
                               int B, int D) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    float s = 0.f;
    for (int d = 0; d < D; ++d) {
        const float sg = softplus_f(pre[b * D + d]);
        const float e = eps[static_cast<long long>(b) * eps_stride + d];
        sigma[b * D + d] = sg;
        z[b * D + d] = fmaf(sg, e, mu[b * D + d]);
        s += 0.5f * kLog2Pi + logf(sg) + 0.5f * e * e;
    }
    elbo[b] += s;
}
// d_mu = g_z;  d_pre_sig = (g_z eps + 1 / sigma) sigmoid(pre_sig)
__global__ void k_guide_back(const float* __restrict__ g_z, const float* __restrict__ eps, int eps_stride,
                             const float* __restrict__ sigma, const float* __restrict__ pre, float* __restrict__ d_mu,
                             float* __restrict__ d_pre, int B, int D) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * D) return;
    const int b = i / D, d = i % D;
    const float g = g_z[i];
    d_mu[i] = g;
    d_pre[i] = (g * eps[static_cast<long long>(b) * eps_stride + d] + 1.f / sigma[i]) * sigmoid_f(pre[i]);
}
// Gaussian head: head = [mean | logvar] ([B][2K]), target y ([B] rows of K with stride y_stride).
//   elbo[b] += sum_k -1/2 (log 2 pi + lv + r^2 exp(-lv)),  r = y - mean
//   d_head = [r inv | -1/2 + r^2 inv / 2],   d_y (optional) += -r inv
// One CTA per window, fixed-order tree reduction.
constexpr int kDensityThreads = 256;
// d_head may be the head array itself (each thread reads its mean and log-variance before it overwrites them).
__global__ void __launch_bounds__(kDensityThreads) k_gauss_density(const float* head, const float* __restrict__ y,
                                                                    long long y_stride, int K, float* __restrict__ elbo,
                                                                    float* d_head, float* __restrict__ d_y) {
    __shared__ float red[kDensityThreads];
    const int b = blockIdx.x;
    const float* h = head + static_cast<long long>(b) * 2 * K;
    float s = 0.f;
    for (int k = threadIdx.x; k < K; k += kDensityThreads) {
        const float m = h[k], lv = h[K + k];
        const float r = y[b * y_stride + k] - m;
        const float inv = expf(-lv);
        s += -0.5f * (kLog2Pi + lv + r * r * inv);
        if (d_head) {
            d_head[static_cast<long long>(b) * 2 * K + k] = r * inv;
            d_head[static_cast<long long>(b) * 2 * K + K + k] = -0.5f + 0.5f * r * r * inv;
        }
        if (d_y) d_y[static_cast<long long>(b) * K + k] += -r * inv;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int half = kDensityThreads / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) red[threadIdx.x] += red[threadIdx.x + half];
        __syncthreads();
    }
    if (threadIdx.x == 0) elbo[b] += red[0];
}
// out[j] (+)= sum_b in[b][j]   (bias gradients), fixed order
__global__ void k_colsum_rows(const float* __restrict__ in, int rows, int cols, float* __restrict__ out, int accumulate) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    float s = accumulate ? out[j] : 0.f;
    for (int r = 0; r < rows; ++r) s += in[static_cast<long long>(r) * cols + j];
    out[j] = s;
}
__global__ void k_add(float* __restrict__ dst, const float* __restrict__ src, long long n) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) dst[i] += src[i];
}

// ---- Adam with clipping by the global norm (Kingma & Ba 2015; Section 4.1) ---------------------------------------
// pass 1: partial sums of squares of scale * g, one per CTA (fixed order); pass 2: one CTA adds them and stores the norm
constexpr int kNormThreads = 256;
__global__ void __launch_bounds__(kNormThreads) k_sumsq_partial(const float* __restrict__ g, long long n, float scale,
                                                                 double* __restrict__ partial) {
    __shared__ double red[kNormThreads];
    double s = 0.0;
    for (long long i = static_cast<long long>(blockIdx.x) * kNormThreads + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * kNormThreads) {
        const double v = static_cast<double>(g[i]) * scale;
        s += v * v;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int half = kNormThreads / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) red[threadIdx.x] += red[threadIdx.x + half];
        __syncthreads();
    }
    if (threadIdx.x == 0) partial[blockIdx.x] = red[0];
}
__global__ void k_norm_finish(const double* __restrict__ partial, int n_part, float* __restrict__ norm_out) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    double s = 0.0;
    for (int i = 0; i < n_part; ++i) s += partial[i];
    *norm_out = static_cast<float>(sqrt(s));
}
// g' = scale * g, clipped: g' *= clip / norm if norm > clip; then the Adam update of step t (t >= 1)
__global__ void k_adam(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
                       long long n, float scale, const float* __restrict__ norm, float clip, float lr, float beta1,
                       float beta2, float eps, float corr1, float corr2) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float nm = *norm;
    const float gs = g[i] * scale * (nm > clip ? clip / nm : 1.f);
    const float mi = beta1 * m[i] + (1.f - beta1) * gs;
    const float vi = beta2 * v[i] + (1.f - beta2) * gs * gs;
    m[i] = mi;
    v[i] = vi;
    p[i] -= lr * (mi / corr1) / (sqrtf(vi / corr2) + eps);
}

}  // namespace fit
}  // namespace cutoff
