// Observation handling, the guide q_phi, the transition and the first emission layer, and the
// fp32 FMA version of the emission output layer.
#pragma once
#include "common.cuh"
#include "rng.cuh"

namespace cutoff {

// ---------------------------------------------------------------------------------------------
// push: obs <- obs U r_w for one whole step (Algorithm 1), plus the normaliser of Section 3.1.3
// (twice the mean of the first fixed-lag window).  One CTA; the sum is a fixed-order tree.
// ---------------------------------------------------------------------------------------------
constexpr int kPushThreads = 256;

__global__ void __launch_bounds__(kPushThreads) k_push(const float* __restrict__ src, float* __restrict__ ring,
                                                       DevState* st, int N, int W) {
    __shared__ double red[kPushThreads];
    const int tid = threadIdx.x;
    const uint32_t pushes = st->push_count;
    double s = 0.0;
    int bad = 0;
    for (int j = tid; j < N; j += kPushThreads) {
        const float v = src[j];
        if (!(v > 0.0f) || !isfinite(v)) bad = 1;
        s += static_cast<double>(v);
    }
    bad = __syncthreads_or(bad);
    if (bad) {
        if (tid == 0) st->error_flags |= kErrBadValue;
        return;
    }
    red[tid] = s;
    __syncthreads();
    for (int half = kPushThreads / 2; half > 0; half >>= 1) {
        if (tid < half) red[tid] += red[tid + half];
        __syncthreads();
    }
    float* dst = ring + static_cast<size_t>(pushes % W) * N;
    for (int j = tid; j < N; j += kPushThreads) dst[j] = src[j];
    if (tid == 0) {
        if (pushes < static_cast<uint32_t>(W)) {
            const double total = st->norm_sum + red[0];
            st->norm_sum = total;
            if (pushes + 1 == static_cast<uint32_t>(W)) {
                const double scale = 2.0 * total / (static_cast<double>(N) * W);
                st->scale = static_cast<float>(scale);
                st->inv_scale = static_cast<float>(1.0 / scale);
            }
        }
        st->push_count = pushes + 1;
    }
}

// ---------------------------------------------------------------------------------------------
// Encoder, part 1: input projections of both RNNs for every window position,
//   P[dir][t][i] = sum_j Wx_dir[i][j] * xhat_t[j] + b_dir[i],   xhat_t = x_t / s.
// One warp per hidden unit i; the weight row is read once for all window positions.
// Window position t (0 = oldest) lives in ring slot (push_count + t) mod W.
// ---------------------------------------------------------------------------------------------
constexpr int kProjWarps = 8;
constexpr int kProjChunk = 8;

__global__ void __launch_bounds__(kProjWarps * 32) k_enc_proj(ModelDev m, const float* __restrict__ ring,
                                                               const DevState* __restrict__ st,
                                                               float* __restrict__ proj /*[2][W][H]*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i = blockIdx.x * kProjWarps + warp;
    const int dir = blockIdx.y;
    if (i >= m.H) return;
    const float* Wx = (dir ? m.Wxb : m.Wxf) + static_cast<size_t>(i) * m.N;
    const float bias = (dir ? m.bb : m.bf)[i];
    const uint32_t pushes = st->push_count;
    const float inv_scale = st->inv_scale;
    for (int t0 = 0; t0 < m.W; t0 += kProjChunk) {
        float acc[kProjChunk];
        const float* row[kProjChunk];
#pragma unroll
        for (int tt = 0; tt < kProjChunk; ++tt) {
            acc[tt] = 0.0f;
            const int t = min(t0 + tt, m.W - 1);
            row[tt] = ring + static_cast<size_t>((pushes + t) % m.W) * m.N;
        }
        for (int j = lane; j < m.N; j += 32) {
            const float w = Wx[j];
#pragma unroll
            for (int tt = 0; tt < kProjChunk; ++tt) acc[tt] = fmaf(w, row[tt][j] * inv_scale, acc[tt]);
        }
#pragma unroll
        for (int tt = 0; tt < kProjChunk; ++tt) {
            float v = acc[tt];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lane == 0 && t0 + tt < m.W) proj[(static_cast<size_t>(dir) * m.W + t0 + tt) * m.H + i] = v + bias;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Encoder, part 2: the two recurrences (h_left forward, h_right backward; Section 3.1.3).
//   a_t = relu(P[0][t] + Whf a_{t-1}),  b_t = relu(P[1][t] + Whb b_{t+1}).
// One CTA per direction; the state lives in shared memory.  hlr[dir][t][i] is written.
// ---------------------------------------------------------------------------------------------
constexpr int kRnnThreads = 1024;

__global__ void __launch_bounds__(kRnnThreads) k_enc_rnn(ModelDev m, const float* __restrict__ proj,
                                                          float* __restrict__ hlr /*[2][W][H]*/) {
    extern __shared__ float sm_rnn[];
    float* state = sm_rnn;
    float* next = sm_rnn + m.H;
    const int dir = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* Wh = dir ? m.Whb : m.Whf;
    const float* init = dir ? m.b0 : m.a0;
    for (int i = threadIdx.x; i < m.H; i += kRnnThreads) state[i] = init[i];
    __syncthreads();
    for (int s = 0; s < m.W; ++s) {
        const int t = dir ? (m.W - 1 - s) : s;
        const float* p = proj + (static_cast<size_t>(dir) * m.W + t) * m.H;
        for (int i = warp; i < m.H; i += kRnnThreads / 32) {
            const float* wrow = Wh + static_cast<size_t>(i) * m.H;
            float acc = 0.0f;
            for (int j = lane; j < m.H; j += 32) acc = fmaf(wrow[j], state[j], acc);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) next[i] = fmaxf(acc + p[i], 0.0f);
        }
        __syncthreads();
        float* out = hlr + (static_cast<size_t>(dir) * m.W + t) * m.H;
        for (int i = threadIdx.x; i < m.H; i += kRnnThreads) {
            const float v = next[i];
            state[i] = v;
            out[i] = v;
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// Per-sample chain: guide steps over the window, transition, first emission layer.
//
// A sample is worked on by a group of G = D/4 adjacent lanes.  Lane g of the group owns the hidden
// units i = g, g+G, g+2G, ... of every layer and the four latent dimensions 4g..4g+3 (exactly one
// Philox call per noise stream).  Every lane keeps the whole latent vector in registers; partial
// layer outputs are summed over the group with xor-shuffles.  Weights are staged in shared memory
// phase by phase, rows padded by four floats so that the G rows a warp reads at once fall into
// different banks.
// ---------------------------------------------------------------------------------------------
constexpr int kChainThreads = 256;

__device__ __forceinline__ float softplusf(float x) { return x > 20.0f ? x : log1pf(expf(x)); }

__device__ __forceinline__ float round_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// Copy a row-major [rows][cols] matrix into shared memory with row stride ld.
__device__ __forceinline__ void stage_matrix(float* dst, const float* __restrict__ src, int rows, int cols, int ld) {
    for (int idx = threadIdx.x; idx < rows * cols; idx += blockDim.x) {
        const int r = idx / cols, c = idx - r * cols;
        dst[r * ld + c] = src[idx];
    }
}

template <int D>
__device__ __forceinline__ float dot_smem(const float* w, const float (&z)[D], float acc) {
    const float4* w4 = reinterpret_cast<const float4*>(w);
#pragma unroll
    for (int d4 = 0; d4 < D / 4; ++d4) {
        const float4 q = w4[d4];
        acc = fmaf(q.x, z[4 * d4 + 0], acc);
        acc = fmaf(q.y, z[4 * d4 + 1], acc);
        acc = fmaf(q.z, z[4 * d4 + 2], acc);
        acc = fmaf(q.w, z[4 * d4 + 3], acc);
    }
    return acc;
}

template <int D2>
__device__ __forceinline__ void axpy_smem(const float* w, float a, float (&y)[D2]) {
    const float4* w4 = reinterpret_cast<const float4*>(w);
#pragma unroll
    for (int d4 = 0; d4 < D2 / 4; ++d4) {
        const float4 q = w4[d4];
        y[4 * d4 + 0] = fmaf(q.x, a, y[4 * d4 + 0]);
        y[4 * d4 + 1] = fmaf(q.y, a, y[4 * d4 + 1]);
        y[4 * d4 + 2] = fmaf(q.z, a, y[4 * d4 + 2]);
        y[4 * d4 + 3] = fmaf(q.w, a, y[4 * d4 + 3]);
    }
}

// Sum y over the G lanes of a group; every lane ends with the total.
template <int G, int M>
__device__ __forceinline__ void group_allreduce(float (&y)[M]) {
#pragma unroll
    for (int off = G / 2; off > 0; off >>= 1)
#pragma unroll
        for (int d = 0; d < M; ++d) y[d] += __shfl_xor_sync(0xffffffffu, y[d], off);
}

// own[c] = y[base + 4g + c] without dynamic register indexing.
template <int G, int M>
__device__ __forceinline__ void select_own(const float (&y)[M], int base, int g, float (&own)[4]) {
#pragma unroll
    for (int gg = 0; gg < G; ++gg)
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (gg == g) own[c] = y[base + 4 * gg + c];
}

// z[4gg + c] = own[c] of lane gg of the group.
template <int G, int D>
__device__ __forceinline__ void group_allgather(const float (&own)[4], float (&z)[D]) {
#pragma unroll
    for (int gg = 0; gg < G; ++gg)
#pragma unroll
        for (int c = 0; c < 4; ++c) z[4 * gg + c] = __shfl_sync(0xffffffffu, own[c], gg, G);
}

// Shared memory needed by k_chain, in floats.
inline size_t chain_smem_floats(int D, int H, int W) {
    const size_t ld = D + 4, ld2 = 2 * D + 4;
    const size_t guide = 2 * H * ld + H + static_cast<size_t>(W) * H + D * ld;
    const size_t trans = H * ld + H * ld2 + H;
    return guide > trans ? guide : trans;
}

template <int D>
__global__ void __launch_bounds__(kChainThreads) k_chain(ModelDev m, const float* __restrict__ hlr,
                                                          const DevState* __restrict__ st, NoiseKey key,
                                                          uint32_t sample_base, int count, int round_v,
                                                          float* __restrict__ v_out /*[count][H]*/) {
    constexpr int G = D / 4, LD = D + 4, LD2 = 2 * D + 4;
    extern __shared__ __align__(16) float sm[];
    const int H = m.H, W = m.W;
    const int g = threadIdx.x % G;
    const int k = blockIdx.x * (kChainThreads / G) + threadIdx.x / G;
    const uint32_t sample = sample_base + static_cast<uint32_t>(k);
    const uint32_t step = st->step;

    // ---- guide: z_t = mu + sigma * eps over the window --------------------------------------
    float* sWz = sm;                    // [H][LD]
    float* sWmuT = sWz + H * LD;        // [H][LD]
    float* sWsig = sWmuT + H * LD;      // [D][LD]
    float* sbz = sWsig + D * LD;        // [H]
    float* shl = sbz + H;               // [W][H]  h_left + h_right
    stage_matrix(sWz, m.Wz, H, D, LD);
    stage_matrix(sWmuT, m.WmuT, H, D, LD);
    stage_matrix(sWsig, m.Wsig, D, D, LD);
    for (int i = threadIdx.x; i < H; i += kChainThreads) sbz[i] = m.bz[i];
    for (int i = threadIdx.x; i < W * H; i += kChainThreads) shl[i] = hlr[i] + hlr[W * H + i];
    __syncthreads();

    float z[D];
#pragma unroll
    for (int d = 0; d < D; ++d) z[d] = m.z0[d];
    for (int t = 0; t < W; ++t) {
        float mu[D];
#pragma unroll
        for (int d = 0; d < D; ++d) mu[d] = 0.0f;
        const float* hl = shl + t * H;
#pragma unroll 2
        for (int i = g; i < H; i += G) {
            const float pre = dot_smem<D>(sWz + i * LD, z, sbz[i]);
            const float h_out = (tanhf(pre) + hl[i]) * (1.0f / 3.0f);
            axpy_smem<D>(sWmuT + i * LD, h_out, mu);
        }
        group_allreduce<G, D>(mu);
#pragma unroll
        for (int d = 0; d < D; ++d) mu[d] += m.bmu[d];
        float eps[4], mu_own[4], z_own[4];
        normal4(static_cast<uint32_t>(g), sample, static_cast<uint32_t>(t), step, key.seed_lo, key.seed_hi, eps);
        select_own<G, D>(mu, 0, g, mu_own);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int d = 4 * g + c;
            const float pre = dot_smem<D>(sWsig + d * LD, mu, m.bsig[d]);
            z_own[c] = fmaf(softplusf(pre), eps[c], mu_own[c]);
        }
        group_allgather<G, D>(z_own, z);
    }
    __syncthreads();

    // ---- transition: z_{T+1} = mean + exp(logvar / 2) * eps ---------------------------------
    float* sW1 = sm;                    // [H][LD]
    float* sW2T = sW1 + H * LD;         // [H][LD2]
    float* sb1 = sW2T + H * LD2;        // [H]
    stage_matrix(sW1, m.W1, H, D, LD);
    stage_matrix(sW2T, m.W2T, H, 2 * D, LD2);
    for (int i = threadIdx.x; i < H; i += kChainThreads) sb1[i] = m.b1[i];
    __syncthreads();
    {
        float head[2 * D];
#pragma unroll
        for (int o = 0; o < 2 * D; ++o) head[o] = 0.0f;
#pragma unroll 2
        for (int i = g; i < H; i += G) {
            const float u = fmaxf(dot_smem<D>(sW1 + i * LD, z, sb1[i]), 0.0f);
            axpy_smem<2 * D>(sW2T + i * LD2, u, head);
        }
        group_allreduce<G, 2 * D>(head);
        float eps[4], mean_own[4], logvar_own[4], z_own[4];
        normal4(static_cast<uint32_t>(g), sample, kStreamTransition, step, key.seed_lo, key.seed_hi, eps);
        select_own<G, 2 * D>(head, 0, g, mean_own);
        select_own<G, 2 * D>(head, D, g, logvar_own);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float mean = mean_own[c] + m.b2[4 * g + c];
            const float logvar = logvar_own[c] + m.b2[D + 4 * g + c];
            z_own[c] = fmaf(expf(0.5f * logvar), eps[c], mean);
        }
        group_allgather<G, D>(z_own, z);
    }
    __syncthreads();

    // ---- emission, hidden layer: v = relu(W3 z + b3) ----------------------------------------
    float* sW3 = sm;                    // [H][LD]
    float* sb3 = sW3 + H * LD;          // [H]
    stage_matrix(sW3, m.W3, H, D, LD);
    for (int i = threadIdx.x; i < H; i += kChainThreads) sb3[i] = m.b3[i];
    __syncthreads();
    if (k < count) {
        float* dst = v_out + static_cast<size_t>(k) * H;
#pragma unroll 4
        for (int i = g; i < H; i += G) {
            float o = fmaxf(dot_smem<D>(sW3 + i * LD, z, sb3[i]), 0.0f);
            if (round_v) o = round_tf32(o);
            dst[i] = o;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Emission output layer in fp32 FMA, with the noise drawn in the epilogue:
//   [mean | logvar] = W4 v + b4,   x_j = mean_j + exp(logvar_j / 2) * eps_j.
// 64 samples x 64 workers per CTA, 4 x 4 (x 2 heads) per thread.
// ---------------------------------------------------------------------------------------------
constexpr int kEmitTM = 64, kEmitTN = 64, kEmitTK = 16, kEmitThreads = 256;

__global__ void __launch_bounds__(kEmitThreads) k_emit_fma(ModelDev m, const float* __restrict__ v,
                                                            const DevState* __restrict__ st, NoiseKey key,
                                                            uint32_t sample_base, int count,
                                                            float* __restrict__ x, int ldx) {
    __shared__ __align__(16) float As[kEmitTK][kEmitTM + 4];
    __shared__ __align__(16) float Bm[kEmitTK][kEmitTN + 4];
    __shared__ __align__(16) float Bl[kEmitTK][kEmitTN + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int row0 = blockIdx.y * kEmitTM, j0 = blockIdx.x * kEmitTN;
    const int H = m.H, N = m.N;
    float acc_m[4][4], acc_l[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc_m[a][b] = acc_l[a][b] = 0.0f;

    const int lr = tid >> 2, lc = (tid & 3) * 4;
    for (int kk = 0; kk < H; kk += kEmitTK) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), bm = a, bl = a;
        if (kk + lc < H) {
            if (row0 + lr < count) a = *reinterpret_cast<const float4*>(v + static_cast<size_t>(row0 + lr) * H + kk + lc);
            if (j0 + lr < N) {
                bm = *reinterpret_cast<const float4*>(m.W4 + static_cast<size_t>(j0 + lr) * H + kk + lc);
                bl = *reinterpret_cast<const float4*>(m.W4 + static_cast<size_t>(N + j0 + lr) * H + kk + lc);
            }
        }
        As[lc + 0][lr] = a.x; As[lc + 1][lr] = a.y; As[lc + 2][lr] = a.z; As[lc + 3][lr] = a.w;
        Bm[lc + 0][lr] = bm.x; Bm[lc + 1][lr] = bm.y; Bm[lc + 2][lr] = bm.z; Bm[lc + 3][lr] = bm.w;
        Bl[lc + 0][lr] = bl.x; Bl[lc + 1][lr] = bl.y; Bl[lc + 2][lr] = bl.z; Bl[lc + 3][lr] = bl.w;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kEmitTK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 m4 = *reinterpret_cast<const float4*>(&Bm[k][tx * 4]);
            const float4 l4 = *reinterpret_cast<const float4*>(&Bl[k][tx * 4]);
            const float av[4] = {a4.x, a4.y, a4.z, a4.w};
            const float mv[4] = {m4.x, m4.y, m4.z, m4.w};
            const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
            for (int a_ = 0; a_ < 4; ++a_)
#pragma unroll
                for (int b_ = 0; b_ < 4; ++b_) {
                    acc_m[a_][b_] = fmaf(av[a_], mv[b_], acc_m[a_][b_]);
                    acc_l[a_][b_] = fmaf(av[a_], lv[b_], acc_l[a_][b_]);
                }
        }
        __syncthreads();
    }

    const uint32_t step = st->step;
    const int jbase = j0 + tx * 4;
    if (jbase >= N) return;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int k = row0 + ty * 4 + s;
        if (k >= count) continue;
        float eps[4];
        normal4(static_cast<uint32_t>(jbase >> 2), sample_base + static_cast<uint32_t>(k), kStreamEmission, step,
                key.seed_lo, key.seed_hi, eps);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = jbase + c;
            if (j < N) {
                const float mean = acc_m[s][c] + m.b4[j];
                const float logvar = acc_l[s][c] + m.b4[N + j];
                x[static_cast<size_t>(k) * ldx + j] = fmaf(expf(0.5f * logvar), eps[c], mean);
            }
        }
    }
}

}  // namespace cutoff
