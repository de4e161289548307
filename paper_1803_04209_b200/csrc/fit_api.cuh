// Host side of the learning entry points (see include/cutoff.h): lays the forward and backward pass of fit.cuh out
// as launches on one stream.  The parameter vector is the weight blob's tensors, in its order, without the header.
#pragma once
#include "fit.cuh"

namespace cutoff {
namespace fit {

enum { iWxf, iWhf, ibf, ia0, iWxb, iWhb, ibb, ib0, iWz, ibz, iWmu, ibmu, iWsig, ibsig, iz0, iW1, ib1, iW2, ib2, iW3, ib3, iW4, ib4, kTensors };

struct Layout {
    long long off[kTensors + 1];
};

inline Layout layout(long long N, long long D, long long H) {
    const long long size[kTensors] = {H * N, H * H, H, H, H * N, H * H, H, H, H * D, H, D * H, D, D * D, D, D,
                                      H * D, H, 2 * D * H, 2 * D, H * D, H, 2 * N * H, 2 * N};
    Layout l;
    l.off[0] = 0;
    for (int i = 0; i < kTensors; ++i) l.off[i + 1] = l.off[i] + size[i];
    return l;
}

// floats of workspace for a batch of B windows of W vectors
inline long long workspace_floats(long long N, long long D, long long H, long long W, long long B) {
    const long long bh = B * H, bd = B * D;
    return 2 * bh                     // a0, b0 broadcast
         + 2 * W * bh                 // a, b
         + (W + 1) * bd               // z (index 0: z0 broadcast)
         + W * (2 * bh + 4 * bd)      // comb, h_out | mu, pre_sig, sigma, dz of the transition density
         + W * (2 * bh)               // u, v
         + W * (B * 2 * D)            // transition head, then its gradient
         + W * (B * 2 * N)            // emission head, then its gradient
         + 2 * W * bh                 // g_a, g_b
         + 3 * bd                     // g_z, g_z_next, g_z_prev
         + 2 * bd                     // d_mu, d_pre_sig
         + 4 * bh;                    // pre_c / d_h, d_v / d_u / d_pre_c, d_pre, carry
}

struct Launcher {
    cudaStream_t s;
    void gemm(const float* A, long long a_m, long long a_k, const float* Bm, long long b_k, long long b_n, float* C, long long c_m,
              const float* bias, int M, int N, int K, int acc) const {
        Gemm g{A, a_m, a_k, Bm, b_k, b_n, C, c_m, bias, M, N, K, acc};
        dim3 grid((N + kGemmTile - 1) / kGemmTile, (M + kGemmTile - 1) / kGemmTile);
        k_gemm<<<grid, 256, 0, s>>>(g);
    }
    // Y[M x O] (+)= X[M x K] W[O x K]^T + bias
    void linear(const float* X, long long ldx, const float* Wt, const float* bias, float* Y, int M, int O, int K, int acc = 0) const {
        gemm(X, ldx, 1, Wt, 1, K, Y, O, bias, M, O, K, acc);
    }
    // dX[M x K] (+)= dY[M x O] W[O x K]
    void input_grad(const float* dY, const float* Wt, float* dX, int M, int O, int K, int acc) const {
        gemm(dY, O, 1, Wt, K, 1, dX, K, nullptr, M, K, O, acc);
    }
    // dW[O x K] += dY[M x O]^T X[M x K];  db[O] += column sums of dY
    void weight_grad(const float* dY, const float* X, long long ldx, float* dW, float* db, int M, int O, int K) const {
        gemm(dY, 1, O, X, ldx, 1, dW, K, nullptr, O, K, M, 1);
        if (db) k_colsum_rows<<<(O + 255) / 256, 256, 0, s>>>(dY, M, O, db, 1);
    }
    static unsigned blocks(long long n) { return static_cast<unsigned>((n + 255) / 256); }
};

// Enqueue forward (+ backward if grads) on `stream`.  All pointers are device pointers.
inline void elbo_grad(int N, int D, int H, int W, int B, const float* p, const float* xhat, const float* eps, float* elbo,
                      float* grads, float* ws, cudaStream_t stream) {
    const Layout L = layout(N, D, H);
    auto w = [&](int i) { return p + L.off[i]; };
    auto g = [&](int i) { return grads + L.off[i]; };
    const Launcher run{stream};
    const long long bh = static_cast<long long>(B) * H, bd = static_cast<long long>(B) * D;
    float* cur = ws;
    auto take = [&](long long n) { float* r = cur; cur += n; return r; };
    float* a0b = take(bh); float* b0b = take(bh);
    float* a = take(W * bh); float* b = take(W * bh);
    float* z = take((W + 1) * bd);
    float* comb = take(W * bh); float* hout = take(W * bh);
    float* mu = take(W * bd); float* presig = take(W * bd); float* sigma = take(W * bd); float* dzt = take(W * bd);
    float* u = take(W * bh); float* v = take(W * bh);
    float* headz = take(static_cast<long long>(W) * B * 2 * D);
    float* headx = take(static_cast<long long>(W) * B * 2 * N);
    float* g_a = take(W * bh); float* g_b = take(W * bh);
    float* g_z = take(bd); float* g_zn = take(bd); float* g_zp = take(bd);
    float* d_mu = take(bd); float* d_ps = take(bd);
    float* t1 = take(bh); float* t2 = take(bh); float* d_pre = take(bh); float* carry = take(bh);
    const bool back = grads != nullptr;
    const long long xs = static_cast<long long>(W) * N;           // stride between windows in xhat
    const int es = W * D;                                         // stride between windows in eps

    cudaMemsetAsync(elbo, 0, sizeof(float) * B, stream);
    if (back) cudaMemsetAsync(dzt, 0, sizeof(float) * W * bd, stream);
    k_broadcast_rows<<<Launcher::blocks(bh), 256, 0, stream>>>(a0b, w(ia0), B, H);
    k_broadcast_rows<<<Launcher::blocks(bh), 256, 0, stream>>>(b0b, w(ib0), B, H);
    k_broadcast_rows<<<Launcher::blocks(bd), 256, 0, stream>>>(z, w(iz0), B, D);
    // ---- encoder RNNs ------------------------------------------------------------------------------------------
    for (int t = 0; t < W; ++t) {
        float* at = a + t * bh;
        run.linear(xhat + static_cast<long long>(t) * N, xs, w(iWxf), w(ibf), at, B, H, N);
        run.linear(t > 0 ? a + (t - 1) * bh : a0b, H, w(iWhf), nullptr, at, B, H, H, 1);
        k_relu<<<Launcher::blocks(bh), 256, 0, stream>>>(at, bh);
    }
    for (int t = W - 1; t >= 0; --t) {
        float* bt = b + t * bh;
        run.linear(xhat + static_cast<long long>(t) * N, xs, w(iWxb), w(ibb), bt, B, H, N);
        run.linear(t + 1 < W ? b + (t + 1) * bh : b0b, H, w(iWhb), nullptr, bt, B, H, H, 1);
        k_relu<<<Launcher::blocks(bh), 256, 0, stream>>>(bt, bh);
    }
    // ---- guide chain and the two densities along the sampled path --------------------------------------------------
    for (int t = 0; t < W; ++t) {
        const float* zp = z + t * bd;
        float* zt = z + (t + 1) * bd;
        run.linear(zp, D, w(iWz), w(ibz), t1, B, H, D);
        k_combine<<<Launcher::blocks(bh), 256, 0, stream>>>(t1, a + t * bh, b + t * bh, comb + t * bh, hout + t * bh, bh);
        run.linear(hout + t * bh, H, w(iWmu), w(ibmu), mu + t * bd, B, D, H);
        run.linear(mu + t * bd, D, w(iWsig), w(ibsig), presig + t * bd, B, D, D);
        k_guide_sample<<<(B + 127) / 128, 128, 0, stream>>>(mu + t * bd, presig + t * bd, eps + t * D, es, sigma + t * bd, zt, elbo, B, D);
        float* ut = u + t * bh;
        run.linear(zp, D, w(iW1), w(ib1), ut, B, H, D);
        k_relu<<<Launcher::blocks(bh), 256, 0, stream>>>(ut, bh);
        float* hz = headz + static_cast<long long>(t) * B * 2 * D;
        run.linear(ut, H, w(iW2), w(ib2), hz, B, 2 * D, H);
        k_gauss_density<<<B, kDensityThreads, 0, stream>>>(hz, zt, D, D, elbo, back ? hz : nullptr, back ? dzt + t * bd : nullptr);
        float* vt = v + t * bh;
        run.linear(zt, D, w(iW3), w(ib3), vt, B, H, D);
        k_relu<<<Launcher::blocks(bh), 256, 0, stream>>>(vt, bh);
        float* hx = headx + static_cast<long long>(t) * B * 2 * N;
        run.linear(vt, H, w(iW4), w(ib4), hx, B, 2 * N, H);
        k_gauss_density<<<B, kDensityThreads, 0, stream>>>(hx, xhat + static_cast<long long>(t) * N, xs, N, elbo, back ? hx : nullptr, nullptr);
    }
    if (!back) return;
    // ---- backward ---------------------------------------------------------------------------------------------------
    cudaMemsetAsync(grads, 0, sizeof(float) * L.off[kTensors], stream);
    cudaMemsetAsync(g_zn, 0, sizeof(float) * bd, stream);
    for (int t = W - 1; t >= 0; --t) {
        const float* zp = z + t * bd;
        const float* zt = z + (t + 1) * bd;
        const float* dhx = headx + static_cast<long long>(t) * B * 2 * N;
        const float* dhz = headz + static_cast<long long>(t) * B * 2 * D;
        // d ELBO / d z_t so far: from step t+1, and from z_t as the target of the transition density
        cudaMemcpyAsync(g_z, g_zn, sizeof(float) * bd, cudaMemcpyDeviceToDevice, stream);
        k_add<<<Launcher::blocks(bd), 256, 0, stream>>>(g_z, dzt + t * bd, bd);
        // emission density
        run.weight_grad(dhx, v + t * bh, H, g(iW4), g(ib4), B, 2 * N, H);
        run.input_grad(dhx, w(iW4), t2, B, 2 * N, H, 0);
        k_relu_back<<<Launcher::blocks(bh), 256, 0, stream>>>(t2, v + t * bh, bh);
        run.weight_grad(t2, zt, D, g(iW3), g(ib3), B, H, D);
        run.input_grad(t2, w(iW3), g_z, B, H, D, 1);
        // transition density
        run.weight_grad(dhz, u + t * bh, H, g(iW2), g(ib2), B, 2 * D, H);
        run.input_grad(dhz, w(iW2), t2, B, 2 * D, H, 0);
        k_relu_back<<<Launcher::blocks(bh), 256, 0, stream>>>(t2, u + t * bh, bh);
        run.weight_grad(t2, zp, D, g(iW1), g(ib1), B, H, D);
        run.input_grad(t2, w(iW1), g_zp, B, H, D, 0);
        // guide
        k_guide_back<<<Launcher::blocks(bd), 256, 0, stream>>>(g_z, eps + t * D, es, sigma + t * bd, presig + t * bd, d_mu, d_ps, B, D);
        run.weight_grad(d_ps, mu + t * bd, D, g(iWsig), g(ibsig), B, D, D);
        run.input_grad(d_ps, w(iWsig), d_mu, B, D, D, 1);
        run.weight_grad(d_mu, hout + t * bh, H, g(iWmu), g(ibmu), B, D, H);
        run.input_grad(d_mu, w(iWmu), t1, B, D, H, 0);
        k_combine_back<<<Launcher::blocks(bh), 256, 0, stream>>>(t1, comb + t * bh, g_a + t * bh, g_b + t * bh, t2, bh);
        run.weight_grad(t2, zp, D, g(iWz), g(ibz), B, H, D);
        run.input_grad(t2, w(iWz), g_zp, B, H, D, 1);
        float* swap = g_zn; g_zn = g_zp; g_zp = swap;
    }
    k_colsum_rows<<<(D + 255) / 256, 256, 0, stream>>>(g_zn, B, D, g(iz0), 1);
    // encoder RNNs
    cudaMemsetAsync(carry, 0, sizeof(float) * bh, stream);
    for (int t = W - 1; t >= 0; --t) {
        k_rnn_back<<<Launcher::blocks(bh), 256, 0, stream>>>(d_pre, g_a + t * bh, carry, a + t * bh, bh);
        run.weight_grad(d_pre, xhat + static_cast<long long>(t) * N, xs, g(iWxf), g(ibf), B, H, N);
        run.weight_grad(d_pre, t > 0 ? a + (t - 1) * bh : a0b, H, g(iWhf), nullptr, B, H, H);
        run.input_grad(d_pre, w(iWhf), carry, B, H, H, 0);
    }
    k_colsum_rows<<<(H + 255) / 256, 256, 0, stream>>>(carry, B, H, g(ia0), 1);
    cudaMemsetAsync(carry, 0, sizeof(float) * bh, stream);
    for (int t = 0; t < W; ++t) {
        k_rnn_back<<<Launcher::blocks(bh), 256, 0, stream>>>(d_pre, g_b + t * bh, carry, b + t * bh, bh);
        run.weight_grad(d_pre, xhat + static_cast<long long>(t) * N, xs, g(iWxb), g(ibb), B, H, N);
        run.weight_grad(d_pre, t + 1 < W ? b + (t + 1) * bh : b0b, H, g(iWhb), nullptr, B, H, H);
        run.input_grad(d_pre, w(iWhb), carry, B, H, H, 0);
    }
    k_colsum_rows<<<(H + 255) / 256, 256, 0, stream>>>(carry, B, H, g(ib0), 1);
}

}  // namespace fit
}  // namespace cutoff
