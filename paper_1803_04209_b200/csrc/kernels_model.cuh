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
    if (tid == 0 && (st->error_flags & kErrNoFinisher)) bad = 1;   // raised by the imputation that precedes this push
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
// Censored run-times (Section 4.2): a worker that was killed at the cutoff gets a draw from its own
// predictive distribution of this step, left-truncated at the cutoff time (the largest run-time
// that was observed).  The predictive distribution is the Monte-Carlo one: column j of the sample
// matrix of the last decision.  The draws are iid, so the first one above the threshold, scanning
// cyclically from a start that does not depend on their values (Philox word 0 of counter
// (worker, 0, 0x300, decision number) modulo S), is an exact draw from the truncated distribution;
// if there is none the threshold itself is used.  One CTA; a warp per censored worker.
// ---------------------------------------------------------------------------------------------
constexpr int kImputeThreads = 1024;
constexpr uint32_t kStreamImpute = 0x300u;

__global__ void __launch_bounds__(kImputeThreads) k_impute(float* __restrict__ stage, const uint8_t* __restrict__ censored,
                                                            const float* __restrict__ x, int ldx, int S, int N,
                                                            DevState* __restrict__ st, NoiseKey key) {
    __shared__ float red[kImputeThreads / 32];
    __shared__ float s_threshold;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float m = -INFINITY;
    for (int j = threadIdx.x; j < N; j += kImputeThreads)
        if (!censored[j]) m = fmaxf(m, stage[j]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (warp == 0) {
        m = red[lane];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        if (lane == 0) s_threshold = m;
    }
    __syncthreads();
    const float threshold = s_threshold;
    if (!(threshold > -INFINITY)) {
        // nobody finished, so there is no cutoff time to truncate at: flag the vector; the push kernel that
        // follows sees the flag and leaves the window untouched
        if (threadIdx.x == 0) st->error_flags |= kErrNoFinisher;
        return;
    }
    const float scale = st->scale;
    const uint32_t step = st->step;
    for (int j = warp; j < N; j += kImputeThreads / 32) {
        if (!censored[j]) continue;
        const uint32_t start = philox4x32_10(static_cast<uint32_t>(j), 0u, kStreamImpute, step, key.seed_lo, key.seed_hi).x %
                               static_cast<uint32_t>(S);
        float value = threshold;
        for (int base = 0; base < S; base += 32) {
            const int i = base + lane;
            float v = -INFINITY;
            if (i < S) {
                uint32_t k = start + static_cast<uint32_t>(i);
                if (k >= static_cast<uint32_t>(S)) k -= static_cast<uint32_t>(S);
                v = x[static_cast<size_t>(k) * ldx + j] * scale;
            }
            const uint32_t hit = __ballot_sync(0xffffffffu, v > threshold);
            if (hit) {
                value = __shfl_sync(0xffffffffu, v, __ffs(hit) - 1);
                break;
            }
        }
        if (lane == 0) stage[j] = value;
    }
}

// ---------------------------------------------------------------------------------------------
// Encoder, part 1: input projections of both RNNs, cached per ring slot,
//   R[dir][slot][i] = sum_j Wx_dir[i][j] * x_slot[j]          (raw seconds: the normaliser is applied by part 2,
//                                                              so a slot's projection never has to be redone)
// One warp per hidden unit i; the weight row is read once for all slots of the launch.
// newest_only = 1: only the slot of the vector pushed last (launched after every push);
// newest_only = 0: every slot (after the ring or the weights were replaced).  Both run the same
// arithmetic per slot, so a cached projection equals a recomputed one bit for bit.
// ---------------------------------------------------------------------------------------------
constexpr int kProjWarps = 8;
constexpr int kProjChunk = 8;

__global__ void __launch_bounds__(kProjWarps * 32) k_enc_proj(ModelDev m, const float* __restrict__ ring,
                                                               const DevState* __restrict__ st, int newest_only,
                                                               float* __restrict__ proj /*[2][W slots][H]*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i = blockIdx.x * kProjWarps + warp;
    const int dir = blockIdx.y;
    if (i >= m.H) return;
    const float* Wx = (dir ? m.Wxb : m.Wxf) + static_cast<size_t>(i) * m.N;
    const int slot_first = newest_only ? static_cast<int>((st->push_count + m.W - 1) % m.W) : 0;
    const int n_slots = newest_only ? 1 : m.W;
    for (int s0 = 0; s0 < n_slots; s0 += kProjChunk) {
        float acc[kProjChunk];
        const float* row[kProjChunk];
#pragma unroll
        for (int tt = 0; tt < kProjChunk; ++tt) {
            acc[tt] = 0.0f;
            row[tt] = ring + static_cast<size_t>(slot_first + min(s0 + tt, n_slots - 1)) * m.N;
        }
        if ((m.N & 3) == 0) {
            // 16-byte loads, four independent iterations in flight
#pragma unroll 4
            for (int j = 4 * lane; j < m.N; j += 128) {
                const float4 w = *reinterpret_cast<const float4*>(Wx + j);
#pragma unroll
                for (int tt = 0; tt < kProjChunk; ++tt) {
                    if (s0 + tt >= n_slots) break;          // uniform: one slot after a push
                    const float4 xv = *reinterpret_cast<const float4*>(row[tt] + j);
                    acc[tt] = fmaf(w.x, xv.x, acc[tt]);
                    acc[tt] = fmaf(w.y, xv.y, acc[tt]);
                    acc[tt] = fmaf(w.z, xv.z, acc[tt]);
                    acc[tt] = fmaf(w.w, xv.w, acc[tt]);
                }
            }
        } else {
            for (int j = lane; j < m.N; j += 32) {
                const float w = Wx[j];
#pragma unroll
                for (int tt = 0; tt < kProjChunk; ++tt) {
                    if (s0 + tt >= n_slots) break;
                    acc[tt] = fmaf(w, row[tt][j], acc[tt]);
                }
            }
        }
#pragma unroll
        for (int tt = 0; tt < kProjChunk; ++tt) {
            float v = acc[tt];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lane == 0 && s0 + tt < n_slots)
                proj[(static_cast<size_t>(dir) * m.W + slot_first + s0 + tt) * m.H + i] = v;
        }
    }
}

// Input projection of window position t (0 = oldest) for hidden unit i: the cached raw projection of the ring slot
// that holds position t, scaled by 1 / s (Section 3.1.3: observations are divided by twice the mean of the first
// window), plus the bias.
__device__ __forceinline__ float window_projection(const ModelDev& m, const float* __restrict__ proj, int dir, int t, int i,
                                                   uint32_t pushes, float inv_scale) {
    const int slot = static_cast<int>((pushes + static_cast<uint32_t>(t)) % static_cast<uint32_t>(m.W));
    return fmaf(proj[(static_cast<size_t>(dir) * m.W + slot) * m.H + i], inv_scale, (dir ? m.bb : m.bf)[i]);
}

// ---------------------------------------------------------------------------------------------
// Encoder, part 2: the two recurrences (h_left forward, h_right backward; Section 3.1.3).
//   a_t = relu(P[0][t] + Whf a_{t-1}),  b_t = relu(P[1][t] + Whb b_{t+1}).
// One CTA per direction; the state lives in shared memory.  hlr[dir][t][i] is written.
// ---------------------------------------------------------------------------------------------
constexpr int kRnnThreads = 1024;

__global__ void __launch_bounds__(kRnnThreads) k_enc_rnn(ModelDev m, const float* __restrict__ proj,
                                                          const DevState* __restrict__ st,
                                                          float* __restrict__ hlr /*[2][W][H]*/) {
    extern __shared__ float sm_rnn[];
    float* state = sm_rnn;
    float* next = sm_rnn + m.H;
    const int dir = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* Wh = dir ? m.Whb : m.Whf;
    const float* init = dir ? m.b0 : m.a0;
    const uint32_t pushes = st->push_count;
    const float inv_scale = st->inv_scale;
    for (int i = threadIdx.x; i < m.H; i += kRnnThreads) state[i] = init[i];
    __syncthreads();
    for (int s = 0; s < m.W; ++s) {
        const int t = dir ? (m.W - 1 - s) : s;
        for (int i = warp; i < m.H; i += kRnnThreads / 32) {
            const float* wrow = Wh + static_cast<size_t>(i) * m.H;
            float acc = 0.0f;
            for (int j = lane; j < m.H; j += 32) acc = fmaf(wrow[j], state[j], acc);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) next[i] = fmaxf(acc + window_projection(m, proj, dir, t, i, pushes, inv_scale), 0.0f);
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
// Encoder, part 2, latency version for H <= 128: the recurrence matrix never leaves the registers.
// One CTA per direction, 4 threads per hidden unit; thread (i, q) owns columns q*H/4 .. of row i.
// The state is double-buffered in shared memory, so a step costs one __syncthreads.
// ---------------------------------------------------------------------------------------------
template <int HQ>   // HQ = H / 4 <= 32
__global__ void __launch_bounds__(16 * HQ) k_enc_rnn_resident(ModelDev m, const float* __restrict__ wh_threads,
                                                              const float* __restrict__ proj,
                                                              const DevState* __restrict__ dev_state,
                                                              float* __restrict__ hlr /*[2][W][H]*/) {
    static_assert(HQ <= 32, "a thread keeps its HQ weights in registers");
    constexpr int H = 4 * HQ, T = 16 * HQ, PAD = HQ + 4;
    extern __shared__ __align__(16) float sm_rr[];
    float* state = sm_rr;                         // [2][4][PAD]
    float* sproj = state + 2 * 4 * PAD;           // [W][H]
    const int dir = blockIdx.x;
    const int t = threadIdx.x, i = t >> 2, q = t & 3;
    // wh_threads holds both recurrence matrices regrouped per thread, [dir][j4][thread][4]: the j4-th group of
    // four weights of thread (i, q) is Wh[i][q*HQ + 4*j4 ..], so that consecutive threads read consecutive 16 bytes
    const float4* Wh = reinterpret_cast<const float4*>(wh_threads) + static_cast<size_t>(dir) * (HQ / 4) * T;
    const float* init = dir ? m.b0 : m.a0;
    float w[HQ];
#pragma unroll
    for (int j4 = 0; j4 < HQ / 4; ++j4) {
        const float4 v = Wh[static_cast<size_t>(j4) * T + t];
        w[4 * j4 + 0] = v.x; w[4 * j4 + 1] = v.y; w[4 * j4 + 2] = v.z; w[4 * j4 + 3] = v.w;
    }
    {
        const uint32_t pushes = dev_state->push_count;
        const float inv_scale = dev_state->inv_scale;
        for (int idx = t; idx < m.W * H; idx += T) sproj[idx] = window_projection(m, proj, dir, idx / H, idx % H, pushes, inv_scale);
    }
    if (t < H) state[(t / HQ) * PAD + (t % HQ)] = init[t];
    __syncthreads();
    int cur = 0;
    for (int s = 0; s < m.W; ++s) {
        const int tt = dir ? (m.W - 1 - s) : s;
        const float* st = state + cur * 4 * PAD + q * PAD;
        float acc = 0.0f;
#pragma unroll
        for (int j4 = 0; j4 < HQ / 4; ++j4) {
            const float4 v = *reinterpret_cast<const float4*>(st + 4 * j4);
            acc = fmaf(w[4 * j4 + 0], v.x, acc); acc = fmaf(w[4 * j4 + 1], v.y, acc);
            acc = fmaf(w[4 * j4 + 2], v.z, acc); acc = fmaf(w[4 * j4 + 3], v.w, acc);
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        if (q == 0) {
            const float v = fmaxf(acc + sproj[tt * H + i], 0.0f);
            state[(cur ^ 1) * 4 * PAD + (i / HQ) * PAD + (i % HQ)] = v;
            hlr[(static_cast<size_t>(dir) * m.W + tt) * H + i] = v;
        }
        __syncthreads();
        cur ^= 1;
    }
}

inline size_t enc_rnn_resident_smem_floats(int H, int W) {
    return 2 * 4 * (H / 4 + 4) + static_cast<size_t>(W) * H;
}

// ---------------------------------------------------------------------------------------------
// Encoder, part 2, for 256 <= H <= 640: the recurrence matrix of a direction is split over the shared
// memories of a cluster of 8 CTAs (H/8 rows each), so it is read from global memory once.  Every CTA
// keeps the whole state (double-buffered); after a step each row's new value is written into the next
// state buffer of all 8 CTAs through distributed shared memory, and one cluster barrier (a hardware
// barrier: no thread leaves before the last step) separates the steps.
// 8 threads per row: thread p of a row takes the 16-byte column chunks p, p+8, ...; rows are padded by
// 8 floats so that the four rows of a warp fall into different banks.  Grid: 16 CTAs (2 clusters).
// ---------------------------------------------------------------------------------------------
constexpr int kRnnClusterSize = 8;

inline size_t enc_rnn_cluster_smem_floats(int H, int W) {
    const int R = H / kRnnClusterSize;
    return static_cast<size_t>(R) * (H + 8) + 2 * static_cast<size_t>(H) + static_cast<size_t>(W) * R;
}

__global__ void __cluster_dims__(kRnnClusterSize, 1, 1) __launch_bounds__(1024)
k_enc_rnn_cluster(ModelDev m, const float* __restrict__ proj, const DevState* __restrict__ dev_state,
                  float* __restrict__ hlr /*[2][W][H]*/) {
    extern __shared__ __align__(16) float sm_rc[];
    launch_dependents();      // the chain kernel may set itself up on the SMs this kernel leaves free
    const int H = m.H, W = m.W, R = H / kRnnClusterSize, ldw = H + 8;
    float* sW = sm_rc;                         // [R][ldw]  rows rank*R .. of the recurrence matrix
    float* state = sW + static_cast<size_t>(R) * ldw;      // [2][H]
    float* sproj = state + 2 * H;              // [W][R]
    uint32_t rank;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int dir = blockIdx.x / kRnnClusterSize;
    const int row = threadIdx.x >> 3, part = threadIdx.x & 7;          // blockDim.x = 8 R
    const int i = static_cast<int>(rank) * R + row;                    // hidden unit of this thread's row
    const float* Wh = (dir ? m.Whb : m.Whf) + static_cast<size_t>(rank) * R * H;
    const float* init = dir ? m.b0 : m.a0;
    // R * H / 4 = blockDim.x * H / 32 chunks of 16 bytes: every thread moves H / 32 of them, eight loads in flight
    for (int base = 0; base < R * (H / 4); base += 8 * blockDim.x) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int idx = base + u * blockDim.x + threadIdx.x;
            if (idx < R * (H / 4)) v[u] = *reinterpret_cast<const float4*>(Wh + static_cast<size_t>(idx / (H / 4)) * H + 4 * (idx % (H / 4)));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int idx = base + u * blockDim.x + threadIdx.x;
            if (idx < R * (H / 4)) *reinterpret_cast<float4*>(sW + static_cast<size_t>(idx / (H / 4)) * ldw + 4 * (idx % (H / 4))) = v[u];
        }
    }
    for (int k = threadIdx.x; k < H; k += blockDim.x) state[k] = init[k];
    {
        const uint32_t pushes = dev_state->push_count;
        const float inv_scale = dev_state->inv_scale;
        for (int idx = threadIdx.x; idx < W * R; idx += blockDim.x)
            sproj[idx] = window_projection(m, proj, dir, idx / R, static_cast<int>(rank) * R + idx % R, pushes, inv_scale);
    }
    // every CTA of the cluster has started and initialised its buffers before anyone writes into them
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    const float* wrow = sW + static_cast<size_t>(row) * ldw;
    int cur = 0;
    for (int s = 0; s < W; ++s) {
        const int t = dir ? (W - 1 - s) : s;
        const float* st = state + cur * H;
        float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;      // four chains: the sum's order is fixed all the same
        for (int c = part; c < H / 4; c += 8) {
            const float4 w = *reinterpret_cast<const float4*>(wrow + 4 * c);
            const float4 v = *reinterpret_cast<const float4*>(st + 4 * c);
            a0 = fmaf(w.x, v.x, a0); a1 = fmaf(w.y, v.y, a1);
            a2 = fmaf(w.z, v.z, a2); a3 = fmaf(w.w, v.w, a3);
        }
        float acc = (a0 + a1) + (a2 + a3);
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        acc += __shfl_xor_sync(0xffffffffu, acc, 4);
        const float v = fmaxf(acc + sproj[t * R + row], 0.0f);
        // thread `part` of the row delivers the new value to CTA `part` of the cluster
        {
            const uint32_t local = static_cast<uint32_t>(__cvta_generic_to_shared(state + (cur ^ 1) * H + i));
            uint32_t remote;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(static_cast<uint32_t>(part)));
            asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
        }
        if (part == 0) hlr[(static_cast<size_t>(dir) * W + t) * H + i] = v;
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        cur ^= 1;
    }
}

// ---------------------------------------------------------------------------------------------
// Per-sample chain: guide steps over the window, transition, first emission layer.
//
// SPL samples are worked on by a group of G = D/4 adjacent lanes.  Lane g of the group owns, of
// every hidden layer, the units i = 4(g + G m) .. 4(g + G m) + 3 (m = 0, 1, ...) and the four
// latent dimensions 4g..4g+3 (exactly one Philox call per noise stream and sample).  Every lane
// keeps the whole latent vector of its samples in registers.  A layer pair
//      hidden = act(A z + a),   out += B hidden
// is evaluated four hidden units at a time as two small outer-product updates: A is staged
// transposed ([D][H]) and B as it is ([out][H]), so that the four weights a lane needs for one
// input or output dimension are one 16-byte shared-memory load, which the G lanes of a group read
// from consecutive addresses and all groups of a warp read as a broadcast.  Partial outputs are
// summed over the group with xor-shuffles.  Each weight read serves all SPL samples of the lane.
// ---------------------------------------------------------------------------------------------
template <int D> struct ChainShape {
    static constexpr int G = D / 4;                   // lanes per group
    static constexpr int SPL = D <= 16 ? 2 : 1;       // samples per lane
    // threads of the phase-staged kernel: its shared memory allows one CTA per SM at D = 32, so that CTA is wide
    static constexpr int kThreads = D <= 16 ? 128 : 384;
    static constexpr int kSamplesPerCta = kThreads / G * SPL;
};

__device__ __forceinline__ float softplusf(float x) { return x > 20.0f ? x : log1pf(expf(x)); }

// tanh(x) = 1 - 2 / (exp(2x) + 1) with the hardware exp2 and reciprocal: absolute error below 3e-7.
__device__ __forceinline__ float tanh_fast(float x) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 2.8853900817779268f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e + 1.0f));
    return fmaf(-2.0f, r, 1.0f);
}

__device__ __forceinline__ float round_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

__device__ __forceinline__ void stage_vector(float* dst, const float* __restrict__ src, int n) {
    for (int i = threadIdx.x; i < n; i += blockDim.x) dst[i] = src[i];
}

__device__ __forceinline__ float4 lds4(const float* p) { return *reinterpret_cast<const float4*>(p); }

// hidden[s][c] = sum_k A^T[k][i0 + c] * z[s][k] + bias[i0 + c]       (A^T staged as [D][H])
template <int D, int SPL>
__device__ __forceinline__ void hidden_block(const float* sAT, const float* sbias, int H, int i0,
                                             const float (&z)[SPL][D], float (&hid)[SPL][4]) {
    const float4 b = lds4(sbias + i0);
#pragma unroll
    for (int s = 0; s < SPL; ++s) { hid[s][0] = b.x; hid[s][1] = b.y; hid[s][2] = b.z; hid[s][3] = b.w; }
#pragma unroll
    for (int k = 0; k < D; ++k) {
        const float4 w = lds4(sAT + k * H + i0);
#pragma unroll
        for (int s = 0; s < SPL; ++s) {
            hid[s][0] = fmaf(w.x, z[s][k], hid[s][0]);
            hid[s][1] = fmaf(w.y, z[s][k], hid[s][1]);
            hid[s][2] = fmaf(w.z, z[s][k], hid[s][2]);
            hid[s][3] = fmaf(w.w, z[s][k], hid[s][3]);
        }
    }
}

// out[s][o] += sum_c B[o][i0 + c] * hid[s][c]                        (B staged as [M][H])
template <int M, int SPL>
__device__ __forceinline__ void output_block(const float* sB, int H, int i0, const float (&hid)[SPL][4],
                                             float (&out)[SPL][M]) {
#pragma unroll
    for (int o = 0; o < M; ++o) {
        const float4 w = lds4(sB + o * H + i0);
#pragma unroll
        for (int s = 0; s < SPL; ++s)
            out[s][o] = fmaf(w.w, hid[s][3], fmaf(w.z, hid[s][2], fmaf(w.y, hid[s][1], fmaf(w.x, hid[s][0], out[s][o]))));
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
    const size_t guide = 2 * static_cast<size_t>(H) * D + H + static_cast<size_t>(W) * H + static_cast<size_t>(D) * D;
    const size_t trans = 3 * static_cast<size_t>(H) * D + H;
    return guide > trans ? guide : trans;
}

__device__ __forceinline__ void stage_vector4(float* dst, const float* __restrict__ src, int n) {   // n % 4 == 0
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* d4 = reinterpret_cast<float4*>(dst);
    for (int i = threadIdx.x; i < n / 4; i += blockDim.x) d4[i] = s4[i];
}

struct ChainNoise {
    NoiseKey key;
    uint32_t step;
    uint32_t sample0;          // global index of the lane's first sample
};

// Guide: z_t = mu + sigma * eps for t = 0..W-1 (Section 3.1.3).  z holds z_{T-l-1} on entry, z_T on exit.
template <int D>
__device__ __forceinline__ void chain_guide(const ModelDev& m, const float* sWzT, const float* sWmu, const float* sWsig,
                                            const float* sbz, const float* shl, int g, const ChainNoise& nz,
                                            float (&z)[ChainShape<D>::SPL][D]) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    const int H = m.H, W = m.W;
    for (int t = 0; t < W; ++t) {
        float mu[SPL][D];
#pragma unroll
        for (int s = 0; s < SPL; ++s)
#pragma unroll
            for (int d = 0; d < D; ++d) mu[s][d] = 0.0f;
        const float* hl = shl + t * H;
        for (int i0 = 4 * g; i0 < H; i0 += 4 * G) {
            float hid[SPL][4];
            hidden_block<D, SPL>(sWzT, sbz, H, i0, z, hid);
            const float4 lr = lds4(hl + i0);
            const float lrv[4] = {lr.x, lr.y, lr.z, lr.w};
#pragma unroll
            for (int s = 0; s < SPL; ++s)
#pragma unroll
                for (int c = 0; c < 4; ++c) hid[s][c] = (tanh_fast(hid[s][c]) + lrv[c]) * (1.0f / 3.0f);
            output_block<D, SPL>(sWmu, H, i0, hid, mu);
        }
#pragma unroll
        for (int s = 0; s < SPL; ++s) {
            group_allreduce<G, D>(mu[s]);
#pragma unroll
            for (int d = 0; d < D; ++d) mu[s][d] += m.bmu[d];
        }
#pragma unroll
        for (int s = 0; s < SPL; ++s) {
            float eps[4], mu_own[4], z_own[4];
            normal4(static_cast<uint32_t>(g), nz.sample0 + s, static_cast<uint32_t>(t), nz.step, nz.key.seed_lo,
                    nz.key.seed_hi, eps);
            select_own<G, D>(mu[s], 0, g, mu_own);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float pre = m.bsig[4 * g + c];
                const float* wrow = sWsig + (4 * g + c) * D;
#pragma unroll
                for (int e4 = 0; e4 < D / 4; ++e4) {
                    const float4 w = lds4(wrow + 4 * e4);
                    pre = fmaf(w.x, mu[s][4 * e4 + 0], pre);
                    pre = fmaf(w.y, mu[s][4 * e4 + 1], pre);
                    pre = fmaf(w.z, mu[s][4 * e4 + 2], pre);
                    pre = fmaf(w.w, mu[s][4 * e4 + 3], pre);
                }
                z_own[c] = fmaf(softplusf(pre), eps[c], mu_own[c]);
            }
            group_allgather<G, D>(z_own, z[s]);
        }
    }
}

// Transition: z_{T+1} = mean + exp(logvar / 2) * eps with [mean | logvar] = W2 relu(W1 z + b1) + b2.
template <int D>
__device__ __forceinline__ void chain_transition(const ModelDev& m, const float* sW1T, const float* sW2, const float* sb1,
                                                 int g, const ChainNoise& nz, float (&z)[ChainShape<D>::SPL][D]) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    const int H = m.H;
    float head[SPL][2 * D];
#pragma unroll
    for (int s = 0; s < SPL; ++s)
#pragma unroll
        for (int o = 0; o < 2 * D; ++o) head[s][o] = 0.0f;
    for (int i0 = 4 * g; i0 < H; i0 += 4 * G) {
        float hid[SPL][4];
        hidden_block<D, SPL>(sW1T, sb1, H, i0, z, hid);
#pragma unroll
        for (int s = 0; s < SPL; ++s)
#pragma unroll
            for (int c = 0; c < 4; ++c) hid[s][c] = fmaxf(hid[s][c], 0.0f);
        output_block<2 * D, SPL>(sW2, H, i0, hid, head);
    }
#pragma unroll
    for (int s = 0; s < SPL; ++s) {
        group_allreduce<G, 2 * D>(head[s]);
        float eps[4], mean_own[4], logvar_own[4], z_own[4];
        normal4(static_cast<uint32_t>(g), nz.sample0 + s, kStreamTransition, nz.step, nz.key.seed_lo, nz.key.seed_hi, eps);
        select_own<G, 2 * D>(head[s], 0, g, mean_own);
        select_own<G, 2 * D>(head[s], D, g, logvar_own);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float mean = mean_own[c] + m.b2[4 * g + c];
            const float logvar = logvar_own[c] + m.b2[D + 4 * g + c];
            z_own[c] = fmaf(expf(0.5f * logvar), eps[c], mean);
        }
        group_allgather<G, D>(z_own, z[s]);
    }
}

// Emission hidden layer: v = relu(W3 z + b3), written for the samples k0 .. k0+SPL-1 that exist.
template <int D>
__device__ __forceinline__ void chain_emission_hidden(const ModelDev& m, const float* sW3T, const float* sb3, int g,
                                                      const float (&z)[ChainShape<D>::SPL][D], int k0, int count,
                                                      int round_v, float* __restrict__ v_out) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    const int H = m.H;
    for (int i0 = 4 * g; i0 < H; i0 += 4 * G) {
        float hid[SPL][4];
        hidden_block<D, SPL>(sW3T, sb3, H, i0, z, hid);
#pragma unroll
        for (int s = 0; s < SPL; ++s) {
            float4 o;
            o.x = fmaxf(hid[s][0], 0.0f); o.y = fmaxf(hid[s][1], 0.0f);
            o.z = fmaxf(hid[s][2], 0.0f); o.w = fmaxf(hid[s][3], 0.0f);
            if (round_v) { o.x = round_tf32(o.x); o.y = round_tf32(o.y); o.z = round_tf32(o.z); o.w = round_tf32(o.w); }
            if (k0 + s < count) *reinterpret_cast<float4*>(v_out + static_cast<size_t>(k0 + s) * H + i0) = o;
        }
    }
}

// Variant 1: weights staged phase by phase (any model size whose largest phase fits in shared memory).
template <int D>
__global__ void __launch_bounds__(ChainShape<D>::kThreads) k_chain(ModelDev m, const float* __restrict__ hlr,
                                                          const DevState* __restrict__ st, NoiseKey key,
                                                          uint32_t sample_base, int count, int round_v,
                                                          float* __restrict__ v_out /*[count][H]*/) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    extern __shared__ __align__(16) float sm[];
    const int H = m.H, W = m.W;
    const int g = threadIdx.x % G;
    const int k0 = (blockIdx.x * (ChainShape<D>::kThreads / G) + threadIdx.x / G) * SPL;      // first sample of the lane
    const ChainNoise nz{key, st->step, sample_base + static_cast<uint32_t>(k0)};

    float* sWzT = sm;                   // [D][H]
    float* sWmu = sWzT + H * D;         // [D][H]
    float* sWsig = sWmu + H * D;        // [D][D]
    float* sbz = sWsig + D * D;         // [H]
    float* shl = sbz + H;               // [W][H]  h_left + h_right
    stage_vector4(sWzT, m.WzT, H * D);
    stage_vector4(sWmu, m.Wmu, H * D);
    stage_vector4(sWsig, m.Wsig, D * D);
    stage_vector4(sbz, m.bz, H);
    for (int i = threadIdx.x; i < W * H; i += blockDim.x) shl[i] = hlr[i] + hlr[W * H + i];
    __syncthreads();
    float z[SPL][D];
#pragma unroll
    for (int s = 0; s < SPL; ++s)
#pragma unroll
        for (int d = 0; d < D; ++d) z[s][d] = m.z0[d];
    chain_guide<D>(m, sWzT, sWmu, sWsig, sbz, shl, g, nz, z);
    __syncthreads();

    float* sW1T = sm;                   // [D][H]
    float* sW2 = sW1T + H * D;          // [2D][H]
    float* sb1 = sW2 + 2 * H * D;       // [H]
    stage_vector4(sW1T, m.W1T, H * D);
    stage_vector4(sW2, m.W2, 2 * H * D);
    stage_vector4(sb1, m.b1, H);
    __syncthreads();
    chain_transition<D>(m, sW1T, sW2, sb1, g, nz, z);
    __syncthreads();

    float* sW3T = sm;                   // [D][H]
    float* sb3 = sW3T + H * D;          // [H]
    stage_vector4(sW3T, m.W3T, H * D);
    stage_vector4(sb3, m.b3, H);
    __syncthreads();
    chain_emission_hidden<D>(m, sW3T, sb3, g, z, k0, count, round_v, v_out);
}

// Variant 2: every weight of the chain resident in shared memory, one persistent CTA per SM.
// The weights are staged once; after that the warps never synchronise: warp w of the grid takes
// the sample batches blockIdx + gridDim * w, + (warps in the grid), ... (a batch = the samples one warp covers).
constexpr int kChainResidentThreads = 512;

inline size_t chain_resident_smem_floats(int D, int H, int W) {
    return 6 * static_cast<size_t>(H) * D + static_cast<size_t>(D) * D + 3 * static_cast<size_t>(H) +
           static_cast<size_t>(W) * H;
}

template <int D>
__global__ void __launch_bounds__(kChainResidentThreads, 1)
k_chain_resident(ModelDev m, const float* __restrict__ hlr, const DevState* __restrict__ st, NoiseKey key,
                 uint32_t sample_base, int count, int round_v, float* __restrict__ v_out /*[count][H]*/) {
    constexpr int G = ChainShape<D>::G, SPL = ChainShape<D>::SPL;
    constexpr int kBatch = 32 / G * SPL;                // samples per warp and pass
    extern __shared__ __align__(16) float sm[];
    const int H = m.H, W = m.W;
    float* sWzT = sm;                   // [D][H]
    float* sWmu = sWzT + H * D;         // [D][H]
    float* sW1T = sWmu + H * D;         // [D][H]
    float* sW2 = sW1T + H * D;          // [2D][H]
    float* sW3T = sW2 + 2 * H * D;      // [D][H]
    float* sWsig = sW3T + H * D;        // [D][D]
    float* sbz = sWsig + D * D;         // [H]
    float* sb1 = sbz + H;               // [H]
    float* sb3 = sb1 + H;               // [H]
    float* shl = sb3 + H;               // [W][H]
    stage_vector4(sWzT, m.WzT, H * D);
    stage_vector4(sWmu, m.Wmu, H * D);
    stage_vector4(sW1T, m.W1T, H * D);
    stage_vector4(sW2, m.W2, 2 * H * D);
    stage_vector4(sW3T, m.W3T, H * D);
    stage_vector4(sWsig, m.Wsig, D * D);
    stage_vector4(sbz, m.bz, H);
    stage_vector4(sb1, m.b1, H);
    stage_vector4(sb3, m.b3, H);
    for (int i = threadIdx.x; i < W * H; i += kChainResidentThreads) shl[i] = hlr[i] + hlr[W * H + i];
    __syncthreads();

    const int lane = threadIdx.x & 31, g = lane % G;
    const int warps_in_grid = gridDim.x * (kChainResidentThreads / 32);
    const int n_batches = ceil_div(count, kBatch);
    const uint32_t step = st->step;
    // consecutive batches go to different CTAs, so that a small decision still spreads over all SMs
    for (int b = blockIdx.x + gridDim.x * (threadIdx.x >> 5); b < n_batches; b += warps_in_grid) {
        const int k0 = b * kBatch + (lane / G) * SPL;
        const ChainNoise nz{key, step, sample_base + static_cast<uint32_t>(k0)};
        float z[SPL][D];
#pragma unroll
        for (int s = 0; s < SPL; ++s)
#pragma unroll
            for (int d = 0; d < D; ++d) z[s][d] = m.z0[d];
        chain_guide<D>(m, sWzT, sWmu, sWsig, sbz, shl, g, nz, z);
        chain_transition<D>(m, sW1T, sW2, sb1, g, nz, z);
        chain_emission_hidden<D>(m, sW3T, sb3, g, z, k0, count, round_v, v_out);
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
