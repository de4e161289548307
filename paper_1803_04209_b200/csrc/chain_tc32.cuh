// Per-sample chain on the tcgen05 tensor cores for latent size 32 and hidden width up to 512
// (tf32 operands).  Same structure as chain_tc.cuh -- per 128-sample tile, every layer pair is
//      hidden = act(A z + a)   (M=128, N=H in halves of 256, K=32)   -> TMEM columns [0, H)
//      out    = B hidden (+b)  (M=128, N=32 per MMA, K=H in chunks of 32)
// with the epilogue warps turning each 32-column chunk of the hidden layer into the next A operand --
// but the weight operands (384 KB at H = 512) do not fit in shared memory, so they are staged phase
// by phase from their swizzled image in global memory into two 64 KB regions:
//      guide steps   region A = Wz,            region B = Wmu
//      transition    region A = W1, then (once its MMAs are done) the log-variance rows of W2;
//                    region B = the mean rows of W2
//      emission      region A = W3
// The 16 epilogue warps do the staging between their last read of a result and their next barrier
// arrival, so the MMA warp needs no extra synchronisation: a barrier it waits on completes only
// after every warp has finished its share of the copy.
// One tile is in flight per CTA (the hidden pre-activations may take all 512 TMEM columns); the
// second results (mu: 32 columns; mean | logvar: 64 columns) reuse columns [0, 64), which is why the
// first two chunks of a phase are produced before the first of them is multiplied.
//
// LITERAL = true runs the networks as Section 3.1.3 prints them (see chain_tc.cuh for the formulas) on the
// same skeleton: after the guide steps come the gate (Wg1, Wg2), the proposal (Wh1, Wh2; its result is combined
// with the gate and the linear map Wl z + bl, which the epilogue threads compute from the latent tile, into G;
// relu(G) then takes the latent tile's place for one more small product with Ws, which stays resident), and the
// first, affine, emission layer u = Wi1 z' + bi1.  Staging: guide A = Wz, B = Wmu; gate A = Wg1, B = Wg2;
// proposal A = Wh1, B = Wh2; emission A = Wi1.
#pragma once
#include "chain_tc.cuh"

namespace cutoff {
namespace tc {

constexpr int kChain32D = 32;

struct ChainTc32Args {
    const float* image;         // swizzled tiles: Wz, W1, W3 (H x 32 each), Wmu, W2 mean rows, W2 logvar rows (H/32 x 32 x 32 each)
                                // literal: Wz, Wg1, Wh1, Wi1 (H x 32 each), Wmu, Wg2, Wh2 (H/32 x 32 x 32 each), Ws (32 x 32)
    const float *bz, *b1, *b3, *bmu, *bsig, *Wsig, *b2, *z0;      // literal: b1 = bg1, b3 = bh1, b2 unused
    const float *bi1 = nullptr, *bg2 = nullptr, *bh2 = nullptr, *Wl = nullptr, *bl = nullptr, *bs = nullptr;   // literal only
    const float* hlr;           // [2][W][H]
    DevState* st;
    NoiseKey key;
    uint32_t sample_base;
    int count, H, W, round_v;
    float* v_out;               // [count][H]
};

inline size_t chain_tc32_image_floats(int H, bool literal = false) {
    return literal ? static_cast<size_t>(H) * 32 * 7 + 1024 : static_cast<size_t>(H) * 32 * 6;
}

inline size_t chain_tc32_smem_bytes(int H, int W, bool literal = false) {
    const size_t tiles = 2 * static_cast<size_t>(H) * 128 + 3 * 16384 + 4096; // regions A, B; Z; two hidden chunks; Ws
    const size_t floats = 4 * static_cast<size_t>(H) + static_cast<size_t>(W) * H + 2 * 32 * 32 + 7 * 32 + 64;
    (void)literal;
    return 1024 + tiles + floats * 4 + 256;
}

// Copy `bytes` (a multiple of 16) from global to shared memory with the 512 epilogue threads.
__device__ __forceinline__ void stage_region(uint8_t* dst, const float* __restrict__ src, uint32_t bytes, int epi_thread) {
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* d4 = reinterpret_cast<float4*>(dst);
    for (uint32_t i = epi_thread; i < bytes / 16; i += kChainEpiWarps * 32) d4[i] = s4[i];
}

template <bool LITERAL>
__global__ void __launch_bounds__(kChainTcThreads, 1) k_chain_tc32(ChainTc32Args a) {
    extern __shared__ uint8_t smem_raw[];
    const int H = a.H, W = a.W;
    const int n_chunks = H / 32;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - raw);
    const uint32_t region_bytes = static_cast<uint32_t>(H) * 128u;
    const uint32_t t_ra = base, t_rb = base + region_bytes;
    const uint32_t t_z = t_rb + region_bytes, t_hb = t_z + 16384u, t_ws = t_hb + 32768u;
    uint8_t* g_ra = gen;
    uint8_t* g_rb = gen + region_bytes;
    float* sbzs = reinterpret_cast<float*>(gen + 2 * region_bytes + 3 * 16384 + 4096);
    float* sb1 = sbzs + H;                   // b1 (literal: bg1)
    float* sb3 = sb1 + H;                    // b3 (literal: bh1)
    float* sbi1 = sb3 + H;                   // literal: bi1
    float* slr = sbi1 + H;                   // [W][H]
    float* sWsig = slr + W * H;              // [32][32]
    float* sWl = sWsig + 1024;               // [32][32] (literal)
    float* sbmu = sWl + 1024;
    float* sbsig = sbmu + 32;
    float* sb2 = sbsig + 32;                 // [64] mean | log-variance biases of the transition (compact)
    float* sbg2 = sb2 + 64;                  // literal: bg2, bh2, bl, bs, 32 each
    float* sbh2 = sbg2 + 32;
    float* sbl = sbh2 + 32;
    float* sbs = sbl + 32;
    float* sz0 = sbs + 32;                   // [32]
    const uint32_t bars = smem_u32(sz0 + 32);
    const uint32_t bar_z = bars, bar_p = bars + 8, bar_h = bars + 16, bar_hfree = bars + 32, bar_acc2 = bars + 48,
                   bar_drain = bars + 56;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sz0 + 32 + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sz0 + 32 + 18);
    // image layout in global memory (floats)
    const size_t tile_f = static_cast<size_t>(H) * 32;
    // compact: Wz W1 W3 | Wmu W2(mean) W2(logvar);  literal: Wz Wg1 Wh1 Wi1 | Wmu Wg2 Wh2 | Ws
    const float* img_wz = a.image;
    const float* img_w1 = img_wz + tile_f;                                    // literal: Wg1
    const float* img_w3 = img_w1 + tile_f;                                    // literal: Wh1
    const float* img_wi1 = img_w3 + tile_f;                                   // literal only
    const float* img_wmu = LITERAL ? img_wi1 + tile_f : img_w3 + tile_f;
    const float* img_w2m = img_wmu + tile_f;                                  // literal: Wg2
    const float* img_w2v = img_w2m + tile_f;                                  // literal: Wh2
    const float* img_ws = img_w2v + tile_f;                                   // literal only: 32 x 32

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int epi_thread = threadIdx.x - 32;               // 0..511 for the epilogue warps

    for (int i = threadIdx.x; i < H; i += kChainTcThreads) {
        sbzs[i] = a.bz[i];
        sb1[i] = a.b1[i];
        sb3[i] = a.b3[i];
    }
    for (int i = threadIdx.x; i < W * H; i += kChainTcThreads) slr[i] = (a.hlr[i] + a.hlr[W * H + i]) * (1.0f / 3.0f);
    for (int i = threadIdx.x; i < 1024; i += kChainTcThreads) sWsig[i] = a.Wsig[i];
    if (threadIdx.x < 32) {
        sbmu[threadIdx.x] = a.bmu[threadIdx.x];
        sbsig[threadIdx.x] = a.bsig[threadIdx.x];
        sz0[threadIdx.x] = a.z0[threadIdx.x];
    }
    if (!LITERAL) {
        if (threadIdx.x < 64) sb2[threadIdx.x] = a.b2[threadIdx.x];
    } else {
        for (int i = threadIdx.x; i < H; i += kChainTcThreads) sbi1[i] = a.bi1[i];
        for (int i = threadIdx.x; i < 1024; i += kChainTcThreads) {
            sWl[i] = a.Wl[i];
            reinterpret_cast<float*>(gen + 2 * region_bytes + 3 * 16384)[i] = img_ws[i];    // the Ws tile stays resident
        }
        if (threadIdx.x < 32) {
            sbg2[threadIdx.x] = a.bg2[threadIdx.x];
            sbh2[threadIdx.x] = a.bh2[threadIdx.x];
            sbl[threadIdx.x] = a.bl[threadIdx.x];
            sbs[threadIdx.x] = a.bs[threadIdx.x];
        }
    }
    if (threadIdx.x == 0) {
        mbar_init(bar_z, kChainEpiWarps);
        mbar_init(bar_p, 1);
        mbar_init(bar_h, kChainEpiWarps);
        mbar_init(bar_h + 8, kChainEpiWarps);
        mbar_init(bar_hfree, 1);
        mbar_init(bar_hfree + 8, 1);
        mbar_init(bar_acc2, 1);
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (LITERAL) fence_proxy_async();                             // the Ws tile was written with ordinary stores
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int n_tiles = ceil_div(a.count, 128);
    const int n_phases = LITERAL ? W + 3 : W + 2;                 // guide steps; transition (literal: gate, proposal); emission layer
    const int ph_last = n_phases - 1;                             // the emission layer: no second GEMM
    const int n_lo = H < 256 ? H : 256, n_hi = H - n_lo;          // the hidden layer is multiplied in two halves

    if (warp == 0) {
        // ---------------- MMA issuer -------------------------------------------------------------------
        const uint32_t idesc_lo = instr_desc_tf32(n_lo), idesc_hi = instr_desc_tf32(n_hi > 0 ? n_hi : 16);
        const uint32_t idesc_32 = instr_desc_tf32(32);
        uint32_t nz = 0, nu = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
            for (int ph = 0; ok && ph < n_phases; ++ph) {
                ok = mbar_wait(bar_z, nz & 1u, abort_flag, a.st);
                if (!ok) break;
                ++nz;
                tc_fence_after();
                if (lane == 0) {
                    const uint64_t a_desc = make_smem_desc(t_z);
                    const uint64_t b_lo = make_smem_desc(t_ra), b_hi = make_smem_desc(t_ra + 256u * 128u);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_tf32(tmem_base, a_desc + 2 * k, b_lo + 2 * k, idesc_lo, k != 0 ? 1u : 0u);
                    if (n_hi > 0) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_tf32(tmem_base + 256u, a_desc + 2 * k, b_hi + 2 * k, idesc_hi, k != 0 ? 1u : 0u);
                    }
                    umma_commit(bar_p);
                }
                __syncwarp();
                if (ph == ph_last) continue;
                // second GEMM.  Its result reuses columns [0, 64): wait for the first two chunks before multiplying the first.
                for (int c = 0; c < n_chunks; ++c, ++nu) {
                    const uint32_t b = nu & 1u;
                    ok = mbar_wait(bar_h + 8 * b, (nu >> 1) & 1u, abort_flag, a.st);
                    if (!ok) break;
                    if (c == 0 && n_chunks > 1) {
                        ok = mbar_wait(bar_h + 8 * (b ^ 1u), ((nu + 1u) >> 1) & 1u, abort_flag, a.st);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    if (lane == 0) {
                        const uint64_t a_desc = make_smem_desc(t_hb + b * 16384u);
                        const uint64_t b_first = make_smem_desc(t_rb + c * 4096u);          // Wmu, or the mean rows of W2
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_tf32(tmem_base, a_desc + 2 * k, b_first + 2 * k, idesc_32, (c | k) != 0 ? 1u : 0u);
                        if (!LITERAL && ph == W) {                                         // log-variance rows of W2 (region A)
                            const uint64_t b_second = make_smem_desc(t_ra + c * 4096u);
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_tf32(tmem_base + 32u, a_desc + 2 * k, b_second + 2 * k, idesc_32, (c | k) != 0 ? 1u : 0u);
                        }
                        umma_commit(bar_hfree + 8 * b);
                        if (c == n_chunks - 1) umma_commit(bar_acc2);
                    }
                    __syncwarp();
                }
                if (LITERAL && ok && ph == W + 1) {
                    // scale of the gated transition: Ws relu(G); relu(G) now sits in the latent tile
                    ok = mbar_wait(bar_z, nz & 1u, abort_flag, a.st);
                    if (!ok) break;
                    ++nz;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint64_t a_desc = make_smem_desc(t_z), b_desc = make_smem_desc(t_ws);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_tf32(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc_32, k != 0 ? 1u : 0u);
                        umma_commit(bar_acc2);
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok) {
            if (lane == 0) umma_commit(bar_drain);
            __syncwarp();
            mbar_wait_quiet(bar_drain, 0u);
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ---------------------------------------------------------------------
        const int q = warp & 3, cg = (warp - 1) >> 2;
        const int row = q * 32 + lane;
        const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t step = a.st->step;
        uint32_t np = 0, na = 0, nu = 0;
        float gate_own[8], lin_own[8], G_own[8];                   // literal: gate, linear map and G of this thread's dimensions
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
            const int k = tile * 128 + row;
            const uint32_t sample = a.sample_base + static_cast<uint32_t>(k);
            // weights of the guide steps; the regions' last readers (the previous tile's MMAs) are done:
            // this warp has seen the previous tile's last bar_p complete
            stage_region(g_ra, img_wz, region_bytes, epi_thread);
            stage_region(g_rb, img_wmu, region_bytes, epi_thread);
            st_shared_v4(t_z + sw128(row, 2 * cg), tf32_rna(sz0[8 * cg + 0]), tf32_rna(sz0[8 * cg + 1]),
                         tf32_rna(sz0[8 * cg + 2]), tf32_rna(sz0[8 * cg + 3]));
            st_shared_v4(t_z + sw128(row, 2 * cg + 1), tf32_rna(sz0[8 * cg + 4]), tf32_rna(sz0[8 * cg + 5]),
                         tf32_rna(sz0[8 * cg + 6]), tf32_rna(sz0[8 * cg + 7]));
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_z);

            for (int ph = 0; ok && ph < n_phases; ++ph) {
                ok = mbar_wait(bar_p, np & 1u, abort_flag, a.st);
                if (!ok) break;
                ++np;
                tc_fence_after();
                if (!LITERAL && ph == W) {
                    // W1 has been multiplied: its region now takes the log-variance rows of W2
                    stage_region(g_ra, img_w2v, region_bytes, epi_thread);
                    fence_proxy_async();
                }
                if (LITERAL && (ph == W || ph == W + 1)) {
                    // Wg1 (Wh1) has been multiplied: its region takes the next first-layer matrix, Wh1 (Wi1)
                    stage_region(g_ra, ph == W ? img_w3 : img_wi1, region_bytes, epi_thread);
                    fence_proxy_async();
                }
                const float* bias = ph < W ? sbzs : (ph == W ? sb1 : (ph == W + 1 ? sb3 : sbi1));
                const float* lr = slr + (ph < W ? ph : 0) * H;
                for (int c = 0; c < n_chunks; ++c) {
                    const int col0 = c * 32 + cg * 8;
                    uint32_t acc[8];
                    tmem_ld8(tmem_base + lane_off + col0, acc);
                    tmem_ld_wait();
                    const float4 b_lo = *reinterpret_cast<const float4*>(bias + col0);
                    const float4 b_hi = *reinterpret_cast<const float4*>(bias + col0 + 4);
                    const float bv[8] = {b_lo.x, b_lo.y, b_lo.z, b_lo.w, b_hi.x, b_hi.y, b_hi.z, b_hi.w};
                    float h[8];
                    if (ph < W) {
                        const float4 l_lo = *reinterpret_cast<const float4*>(lr + col0);
                        const float4 l_hi = *reinterpret_cast<const float4*>(lr + col0 + 4);
                        const float lv[8] = {l_lo.x, l_lo.y, l_lo.z, l_lo.w, l_hi.x, l_hi.y, l_hi.z, l_hi.w};
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            float t;                                   // tanh by the hardware instruction (chain_tc.cuh)
                            asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(__uint_as_float(acc[i]) + bv[i]));
                            h[i] = fmaf(t, 1.0f / 3.0f, lv[i]);
                        }
                    } else if (!LITERAL || ph < ph_last) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) h[i] = fmaxf(__uint_as_float(acc[i]) + bv[i], 0.0f);
                    } else {                                       // literal: the first emission layer is affine
#pragma unroll
                        for (int i = 0; i < 8; ++i) h[i] = __uint_as_float(acc[i]) + bv[i];
                    }
                    if (ph < ph_last) {
                        const uint32_t b = nu & 1u;
                        if (nu >= 2) {
                            ok = mbar_wait(bar_hfree + 8 * b, ((nu >> 1) - 1u) & 1u, abort_flag, a.st);
                            if (!ok) break;
                        }
                        const uint32_t dst = t_hb + b * 16384u;
                        st_shared_v4(dst + sw128(row, 2 * cg), tf32_rna(h[0]), tf32_rna(h[1]), tf32_rna(h[2]), tf32_rna(h[3]));
                        st_shared_v4(dst + sw128(row, 2 * cg + 1), tf32_rna(h[4]), tf32_rna(h[5]), tf32_rna(h[6]), tf32_rna(h[7]));
                        fence_proxy_async();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_h + 8 * b);
                        ++nu;
                    } else if (k < a.count) {
                        if (a.round_v) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) h[i] = tf32_rna(h[i]);
                        }
                        store8(a.v_out + static_cast<size_t>(k) * H + col0, h);          // one whole 32-byte sector
                    }
                }
                if (!ok || ph == ph_last) continue;

                // ---- second result: the next latent (this thread: dimensions 8cg .. 8cg+7) ----------------
                ok = mbar_wait(bar_acc2, na & 1u, abort_flag, a.st);
                if (!ok) break;
                ++na;
                tc_fence_after();
                float z_own[8], eps[8];
                const uint32_t stream = ph < W ? static_cast<uint32_t>(ph) : kStreamTransition;
                if (!LITERAL || ph != W) {                          // the gate phase draws nothing
                    normal4_fast(static_cast<uint32_t>(2 * cg), sample, stream, step, a.key.seed_lo, a.key.seed_hi, eps);
                    normal4_fast(static_cast<uint32_t>(2 * cg + 1), sample, stream, step, a.key.seed_lo, a.key.seed_hi, eps + 4);
                }
                if (ph < W) {
                    uint32_t mu_lo[16], mu_hi[16], own_bits[8];
                    tmem_ld16(tmem_base + lane_off, mu_lo);
                    tmem_ld16(tmem_base + lane_off + 16, mu_hi);
                    tmem_ld8(tmem_base + lane_off + 8 * cg, own_bits);
                    tmem_ld_wait();
                    float mu[32];
#pragma unroll
                    for (int d = 0; d < 16; ++d) {
                        mu[d] = __uint_as_float(mu_lo[d]) + sbmu[d];
                        mu[16 + d] = __uint_as_float(mu_hi[d]) + sbmu[16 + d];
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float* wrow = sWsig + (8 * cg + c) * 32;
                        float pre = sbsig[8 * cg + c];
#pragma unroll
                        for (int e = 0; e < 32; ++e) pre = fmaf(wrow[e], mu[e], pre);
                        z_own[c] = fmaf(softplus_fast(pre), eps[c], __uint_as_float(own_bits[c]) + sbmu[8 * cg + c]);
                    }
                    // the guide's weights are done with after its last step: bring in W1 and the mean rows of W2
                    if (ph == W - 1) {
                        stage_region(g_ra, img_w1, region_bytes, epi_thread);
                        stage_region(g_rb, img_w2m, region_bytes, epi_thread);
                    }
                } else if (!LITERAL) {
                    uint32_t mean_bits[8], lv_bits[8];
                    tmem_ld8(tmem_base + lane_off + 8 * cg, mean_bits);
                    tmem_ld8(tmem_base + lane_off + 32 + 8 * cg, lv_bits);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        z_own[c] = fmaf(exp_half_fast(__uint_as_float(lv_bits[c]) + sb2[32 + 8 * cg + c]), eps[c],
                                        __uint_as_float(mean_bits[c]) + sb2[8 * cg + c]);
                    stage_region(g_ra, img_w3, region_bytes, epi_thread);      // W2 is done with: bring in W3
                } else if (ph == W) {
                    // gate g, and the linear map Wl z + bl from the latent tile (which stays as it is for the proposal)
                    uint32_t res[8];
                    tmem_ld8(tmem_base + lane_off + 8 * cg, res);
                    tmem_ld_wait();
                    float zf[32];
#pragma unroll
                    for (int e4 = 0; e4 < 8; ++e4) {
                        const float4 v4 = ld_shared_v4(t_z + sw128(row, e4));
                        zf[4 * e4 + 0] = v4.x; zf[4 * e4 + 1] = v4.y; zf[4 * e4 + 2] = v4.z; zf[4 * e4 + 3] = v4.w;
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        gate_own[c] = sigmoid_fast(__uint_as_float(res[c]) + sbg2[8 * cg + c]);
                        const float* wrow = sWl + (8 * cg + c) * 32;
                        float lin = sbl[8 * cg + c];
#pragma unroll
                        for (int e = 0; e < 32; ++e) lin = fmaf(wrow[e], zf[e], lin);
                        lin_own[c] = lin;
                    }
                    stage_region(g_rb, img_w2v, region_bytes, epi_thread);     // Wg2 is done with: bring in Wh2
                    fence_proxy_async();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_z);                         // the proposal reads the same latent tile
                    continue;
                } else {
                    // proposal h -> G = (1 - g) * lin + g * h; relu(G) replaces the latent tile for the scale product
                    uint32_t res[8];
                    tmem_ld8(tmem_base + lane_off + 8 * cg, res);
                    tmem_ld_wait();
                    float r[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float prop = __uint_as_float(res[c]) + sbh2[8 * cg + c];
                        G_own[c] = fmaf(gate_own[c], prop - lin_own[c], lin_own[c]);
                        r[c] = tf32_rna(fmaxf(G_own[c], 0.0f));
                    }
                    st_shared_v4(t_z + sw128(row, 2 * cg), r[0], r[1], r[2], r[3]);
                    st_shared_v4(t_z + sw128(row, 2 * cg + 1), r[4], r[5], r[6], r[7]);
                    fence_proxy_async();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_z);
                    // z' = G + softplus(Ws relu(G) + bs) * eps
                    ok = mbar_wait(bar_acc2, na & 1u, abort_flag, a.st);
                    if (!ok) break;
                    ++na;
                    tc_fence_after();
                    tmem_ld8(tmem_base + lane_off + 8 * cg, res);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        z_own[c] = fmaf(softplus_fast(__uint_as_float(res[c]) + sbs[8 * cg + c]), eps[c], G_own[c]);
                }
                st_shared_v4(t_z + sw128(row, 2 * cg), tf32_rna(z_own[0]), tf32_rna(z_own[1]), tf32_rna(z_own[2]), tf32_rna(z_own[3]));
                st_shared_v4(t_z + sw128(row, 2 * cg + 1), tf32_rna(z_own[4]), tf32_rna(z_own[5]), tf32_rna(z_own[6]), tf32_rna(z_own[7]));
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_z);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

}  // namespace tc
}  // namespace cutoff
