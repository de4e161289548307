// The generative model as Section 3.1.3 prints it ("literal" variant), in fp32 FMA:
//   gated transition   g = MLP_2(z, ReLU, Sigmoid),  h = MLP_2(z, ReLU, Identity),
//                      G = (1 - g) * MLP_1(z, Identity) + g * h,  H = MLP_1(ReLU(G), Softplus),
//                      z' = G + H * eps
//   emission           I = MLP_2(z', Identity, Identity),  J = MLP_2(I, ReLU, Softplus),  x = I + J * eps
// H and J are standard deviations.  The guide is the one of kernels_model.cuh.
//
// The chain kernel ends with the first (affine) layer of I; the rest of the emission is three
// matrix products over all samples (k_gemm_fma here; tc::k_gemm_relu_tc and tc::k_emit_dual_tc on the tensor cores):
//   I = u Wi2^T + bi2        r = relu(I Wj1^T + bj1)        x = I + softplus(r Wj2^T + bj2) * eps
#pragma once
#include "common.cuh"
#include "kernels_model.cuh"
#include "rng.cuh"

namespace cutoff {

// Device pointers of the literal variant's generative model.
struct LiteralDev {
    const float *Wg1T, *bg1, *Wg2, *bg2;    // gate:      Wg1T [D][H] (transposed copy), Wg2 [D][H]
    const float *Wh1T, *bh1, *Wh2, *bh2;    // proposal:  Wh1T [D][H] (transposed copy), Wh2 [D][H]
    const float *Wl, *bl, *Ws, *bs;         // linear map and scale, each [D][D]
    const float *Wi1T, *bi1;                // emission mean, first layer: Wi1T [D][H] (transposed copy)
    const float *Wi2, *bi2;                 // emission mean, second layer [N][H]
    const float *Wj1, *bj1;                 // emission scale, first layer [H][ldn] (rows padded with zeros to ldn)
    const float *Wj2, *bj2;                 // emission scale, second layer [N][H]
    int ldn;
};

__device__ __forceinline__ float sigmoidf(float x) { return 1.0f / (1.0f + expf(-x)); }

// out_own[c] = bias[4g + c] + sum_e M[4g + c][e] * in[e]      (M staged in shared memory as [D][D])
template <int D>
__device__ __forceinline__ void small_linear_own(const float* sM, const float* __restrict__ bias, int g,
                                                 const float (&in)[D], float (&out_own)[4]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float acc = bias[4 * g + c];
        const float* wrow = sM + (4 * g + c) * D;
#pragma unroll
        for (int e4 = 0; e4 < D / 4; ++e4) {
            const float4 w = lds4(wrow + 4 * e4);
            acc = fmaf(w.x, in[4 * e4 + 0], acc);
            acc = fmaf(w.y, in[4 * e4 + 1], acc);
            acc = fmaf(w.z, in[4 * e4 + 2], acc);
            acc = fmaf(w.w, in[4 * e4 + 3], acc);
        }
        out_own[c] = acc;
    }
}

// out[s][:] += B relu(A z[s] + a), the two-layer pattern of the gate and of the proposal (before the last bias).
template <int D>
__device__ __forceinline__ void relu_mlp2_partial(const float* sAT, const float* sbias, const float* sB, int H, int g,
                                                  const float (&z)[ChainShape<D>::SPL][D],
                                                  float (&out)[ChainShape<D>::SPL][D]) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    for (int i0 = 4 * g; i0 < H; i0 += 4 * G) {
        float hid[SPL][4];
        hidden_block<D, SPL>(sAT, sbias, H, i0, z, hid);
#pragma unroll
        for (int s = 0; s < SPL; ++s)
#pragma unroll
            for (int c = 0; c < 4; ++c) hid[s][c] = fmaxf(hid[s][c], 0.0f);
        output_block<D, SPL>(sB, H, i0, hid, out);
    }
}

// First layer of the emission mean, u = Wi1 z + bi1 (no activation), written for the samples that exist.
template <int D>
__device__ __forceinline__ void literal_emission_first(const float* sWi1T, const float* sbi1, int H, int g,
                                                       const float (&z)[ChainShape<D>::SPL][D], int k0, int count,
                                                       int round_u, float* __restrict__ u_out) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    for (int i0 = 4 * g; i0 < H; i0 += 4 * G) {
        float hid[SPL][4];
        hidden_block<D, SPL>(sWi1T, sbi1, H, i0, z, hid);
#pragma unroll
        for (int s = 0; s < SPL; ++s) {
            float4 o = make_float4(hid[s][0], hid[s][1], hid[s][2], hid[s][3]);
            if (round_u) { o.x = round_tf32(o.x); o.y = round_tf32(o.y); o.z = round_tf32(o.z); o.w = round_tf32(o.w); }
            if (k0 + s < count) *reinterpret_cast<float4*>(u_out + static_cast<size_t>(k0 + s) * H + i0) = o;
        }
    }
}

// Per-sample chain of the literal variant: guide steps over the window, gated transition, first emission layer.
// Same work split as k_chain (G = D/4 lanes per group of SPL samples); the weights of each phase are staged in
// shared memory one phase after the other: guide | gate | proposal | linear map, scale and first emission layer.
template <int D>
__global__ void __launch_bounds__(ChainShape<D>::kThreads) k_chain_literal(ModelDev m, LiteralDev lit,
                                                                           const float* __restrict__ hlr,
                                                                           const DevState* __restrict__ st, NoiseKey key,
                                                                           uint32_t sample_base, int count, int round_u,
                                                                           float* __restrict__ u_out /*[count][H]*/) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    extern __shared__ __align__(16) float sm[];
    const int H = m.H, W = m.W;
    const int g = threadIdx.x % G;
    const int k0 = (blockIdx.x * (ChainShape<D>::kThreads / G) + threadIdx.x / G) * SPL;
    const ChainNoise nz{key, st->step, sample_base + static_cast<uint32_t>(k0)};

    {   // guide
        float* sWzT = sm;
        float* sWmu = sWzT + H * D;
        float* sWsig = sWmu + H * D;
        float* sbz = sWsig + D * D;
        float* shl = sbz + H;
        stage_vector4(sWzT, m.WzT, H * D);
        stage_vector4(sWmu, m.Wmu, H * D);
        stage_vector4(sWsig, m.Wsig, D * D);
        stage_vector4(sbz, m.bz, H);
        for (int i = threadIdx.x; i < W * H; i += blockDim.x) shl[i] = hlr[i] + hlr[W * H + i];
    }
    __syncthreads();
    float z[SPL][D];
#pragma unroll
    for (int s = 0; s < SPL; ++s)
#pragma unroll
        for (int d = 0; d < D; ++d) z[s][d] = m.z0[d];
    chain_guide<D>(m, sm, sm + H * D, sm + 2 * H * D, sm + 2 * H * D + D * D, sm + 2 * H * D + D * D + H, g, nz, z);
    __syncthreads();

    float* sAT = sm;                    // [D][H]  first layer, transposed
    float* sB = sAT + H * D;            // [D][H]  second layer
    float* sb = sB + H * D;             // [H]
    float pre_gate[SPL][D], pre_prop[SPL][D];
#pragma unroll
    for (int s = 0; s < SPL; ++s)
#pragma unroll
        for (int d = 0; d < D; ++d) pre_gate[s][d] = pre_prop[s][d] = 0.0f;
    stage_vector4(sAT, lit.Wg1T, H * D);
    stage_vector4(sB, lit.Wg2, H * D);
    stage_vector4(sb, lit.bg1, H);
    __syncthreads();
    relu_mlp2_partial<D>(sAT, sb, sB, H, g, z, pre_gate);
    __syncthreads();
    stage_vector4(sAT, lit.Wh1T, H * D);
    stage_vector4(sB, lit.Wh2, H * D);
    stage_vector4(sb, lit.bh1, H);
    __syncthreads();
    relu_mlp2_partial<D>(sAT, sb, sB, H, g, z, pre_prop);
    __syncthreads();

    float* sWi1T = sm;                  // [D][H]
    float* sbi1 = sWi1T + H * D;        // [H]
    float* sWl = sbi1 + H;              // [D][D]
    float* sWs = sWl + D * D;           // [D][D]
    stage_vector4(sWi1T, lit.Wi1T, H * D);
    stage_vector4(sbi1, lit.bi1, H);
    stage_vector4(sWl, lit.Wl, D * D);
    stage_vector4(sWs, lit.Ws, D * D);
    __syncthreads();
#pragma unroll
    for (int s = 0; s < SPL; ++s) {
        group_allreduce<G, D>(pre_gate[s]);
        group_allreduce<G, D>(pre_prop[s]);
        float gate_own[4], prop_own[4], lin_own[4], G_own[4], scale_own[4], eps[4], z_own[4];
        select_own<G, D>(pre_gate[s], 0, g, gate_own);
        select_own<G, D>(pre_prop[s], 0, g, prop_own);
        small_linear_own<D>(sWl, lit.bl, g, z[s], lin_own);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float gate = sigmoidf(gate_own[c] + lit.bg2[4 * g + c]);
            const float prop = prop_own[c] + lit.bh2[4 * g + c];
            G_own[c] = (1.0f - gate) * lin_own[c] + gate * prop;
        }
        float G_all[D];
        group_allgather<G, D>(G_own, G_all);
#pragma unroll
        for (int d = 0; d < D; ++d) G_all[d] = fmaxf(G_all[d], 0.0f);
        small_linear_own<D>(sWs, lit.bs, g, G_all, scale_own);
        normal4(static_cast<uint32_t>(g), nz.sample0 + s, kStreamTransition, nz.step, key.seed_lo, key.seed_hi, eps);
#pragma unroll
        for (int c = 0; c < 4; ++c) z_own[c] = fmaf(softplusf(scale_own[c]), eps[c], G_own[c]);
        group_allgather<G, D>(z_own, z[s]);
    }
    literal_emission_first<D>(sWi1T, sbi1, H, g, z, k0, count, round_u, u_out);
}

// ---------------------------------------------------------------------------------------------
// C = A B^T with an epilogue, fp32 FMA: A [M][lda] (K columns used), B [Nout][ldb], 64 x 64 outputs per
// CTA, 4 x 4 per thread.  K, lda and ldb are multiples of 4; entries of A and B beyond the logical K
// must be zero (padded rows).
//   kEpiAffine      out = acc + bias
//   kEpiRelu        out = relu(acc + bias)                      (rounded to tf32 if round_out)
//   kEpiScaleNoise  out = add + softplus(acc + bias) * eps      (add: [M][ld_out]; eps: emission stream)
// ---------------------------------------------------------------------------------------------
enum { kEpiAffine = 0, kEpiRelu = 1, kEpiScaleNoise = 2 };

struct GemmFmaArgs {
    const float* A; int lda;
    const float* B; int ldb;
    const float* bias;
    const float* add;
    float* out; int ld_out;
    int M, Nout, K;
    int round_out;
    const DevState* st;
    NoiseKey key;
    uint32_t sample_base;
};

template <int EPI>
__global__ void __launch_bounds__(kEmitThreads) k_gemm_fma(GemmFmaArgs a) {
    __shared__ __align__(16) float As[kEmitTK][kEmitTM + 4];
    __shared__ __align__(16) float Bs[kEmitTK][kEmitTN + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int row0 = blockIdx.y * kEmitTM, j0 = blockIdx.x * kEmitTN;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    const int lr = tid >> 2, lc = (tid & 3) * 4;
    for (int kk = 0; kk < a.K; kk += kEmitTK) {
        float4 av = make_float4(0.f, 0.f, 0.f, 0.f), bv = av;
        if (kk + lc < a.K) {
            if (row0 + lr < a.M) av = *reinterpret_cast<const float4*>(a.A + static_cast<size_t>(row0 + lr) * a.lda + kk + lc);
            if (j0 + lr < a.Nout) bv = *reinterpret_cast<const float4*>(a.B + static_cast<size_t>(j0 + lr) * a.ldb + kk + lc);
        }
        As[lc + 0][lr] = av.x; As[lc + 1][lr] = av.y; As[lc + 2][lr] = av.z; As[lc + 3][lr] = av.w;
        Bs[lc + 0][lr] = bv.x; Bs[lc + 1][lr] = bv.y; Bs[lc + 2][lr] = bv.z; Bs[lc + 3][lr] = bv.w;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kEmitTK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float ar[4] = {a4.x, a4.y, a4.z, a4.w};
            const float br[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
        __syncthreads();
    }
    const int jbase = j0 + tx * 4;
    if (jbase >= a.Nout) return;
    const uint32_t step = EPI == kEpiScaleNoise ? a.st->step : 0u;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int k = row0 + ty * 4 + s;
        if (k >= a.M) continue;
        float eps[4] = {0.f, 0.f, 0.f, 0.f};
        if (EPI == kEpiScaleNoise)
            normal4(static_cast<uint32_t>(jbase >> 2), a.sample_base + static_cast<uint32_t>(k), kStreamEmission, step,
                    a.key.seed_lo, a.key.seed_hi, eps);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = jbase + c;
            if (j >= a.Nout) continue;
            const size_t o = static_cast<size_t>(k) * a.ld_out + j;
            float v = acc[s][c] + a.bias[j];
            if (EPI == kEpiRelu) {
                v = fmaxf(v, 0.0f);
                if (a.round_out) v = round_tf32(v);
            }
            if (EPI == kEpiScaleNoise) v = fmaf(softplusf(v), eps[c], a.add[o]);
            a.out[o] = v;
        }
    }
}

}  // namespace cutoff
