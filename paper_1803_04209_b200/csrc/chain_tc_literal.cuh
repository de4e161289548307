// Per-sample chain of the literal model variant (Section 3.1.3 as printed) on the tcgen05 tensor cores,
// for latent size 16 and hidden width 64..256, operands in tf32: the guide steps, then the gated transition
//      g = sigmoid(Wg2 relu(Wg1 z + bg1) + bg2)        h = Wh2 relu(Wh1 z + bh1) + bh2
//      G = (1 - g) * (Wl z + bl) + g * h               H = softplus(Ws relu(G) + bs)        z' = G + H * eps
// and the first (affine) layer of the emission mean, u = Wi1 z' + bi1, which goes to global memory for
// the three emission products.
//
// Same machinery as k_chain_tc (chain_tc.cuh): two tiles of 128 samples in flight per CTA, every layer pair
// as two UMMA groups with the hidden layer handed over in 32-column chunks through shared memory, all weight
// operands resident in shared memory.  Phases: W guide steps; gate (Wg1, Wg2); proposal (Wh1, Wh2), whose
// second result is combined with the gate and the linear map (computed by the epilogue threads from the
// latent tile) into G, after which relu(G) takes the place of the latent tile and one more small product
// with Ws gives the scale; first emission layer (Wi1, no activation).
// Latent rows are 128 bytes wide although K = 16: [Wz | Wg1] and [Wh1 | Wi1] share one tile each.
#pragma once
#include "chain_tc.cuh"

namespace cutoff {
namespace tc {

struct ChainTclArgs {
    const float* image;         // swizzled operand tiles: [Wz|Wg1] (H x 32), [Wh1|Wi1] (H x 32), Wmu, Wg2, Wh2 (H/32 x 16 x 32 each), Ws (16 x 32)
    const float *bz, *bg1, *bh1, *bi1, *bmu, *bsig, *Wsig, *bg2, *bh2, *Wl, *bl, *bs, *z0;
    const float* hlr;           // [2][W][H] h_left, h_right
    DevState* st;
    NoiseKey key;
    uint32_t sample_base;
    int count, H, W;
    float* u_out;               // [count][H], rounded to tf32
};

inline size_t chain_tcl_image_floats(int H) { return static_cast<size_t>(H) * (32 + 32 + 16 + 16 + 16) + 16 * 32; }

inline size_t chain_tcl_smem_bytes(int H, int W) {
    const size_t tiles = chain_tcl_image_floats(H) * 4 + 2 * 128 * 128 /*Z x2*/ + 4 * 128 * 128 /*hidden chunks: 2 per slot*/;
    const size_t floats = 4 * static_cast<size_t>(H) + static_cast<size_t>(W) * H + 2 * 16 * 16 + 7 * 16;
    return 1024 + tiles + floats * 4 + 256;
}

__device__ __forceinline__ float sigmoid_fast(float x) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e + 1.0f));
    return r;
}

__device__ __forceinline__ float4 ld_shared_v4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}

__global__ void __launch_bounds__(kChainTcThreads, 1) k_chain_tc_literal(ChainTclArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const int H = a.H, W = a.W;
    const int n_chunks = H / 32;                                  // a chunk = 32 hidden units = one K block
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - raw);
    // weight operand tiles
    const uint32_t t_zg = base;                                   // [Wz | Wg1]
    const uint32_t t_hi = t_zg + H * 128;                         // [Wh1 | Wi1]
    const uint32_t t_wmu = t_hi + H * 128;
    const uint32_t t_wg2 = t_wmu + H * 64;
    const uint32_t t_wh2 = t_wg2 + H * 64;
    const uint32_t t_ws = t_wh2 + H * 64;                         // 16 rows x 128 bytes
    const uint32_t image_bytes = static_cast<uint32_t>(H) * 448u + 2048u;
    const uint32_t t_act = base + image_bytes;                    // Z0, Z1, then 4 hidden-chunk buffers: 6 x 16 KB
    // fp32 side tables
    float* sbzs = reinterpret_cast<float*>(gen + image_bytes + 6 * 16384);    // bz
    float* sbg1 = sbzs + H;
    float* sbh1 = sbg1 + H;
    float* sbi1 = sbh1 + H;
    float* slr = sbi1 + H;                   // [W][H]  (h_left + h_right) / 3
    float* sWsig = slr + W * H;              // [16][16]
    float* sWl = sWsig + 256;                // [16][16]
    float* sbmu = sWl + 256;
    float* sbsig = sbmu + 16;
    float* sbg2 = sbsig + 16;
    float* sbh2 = sbg2 + 16;
    float* sbl = sbh2 + 16;
    float* sbs = sbl + 16;
    float* sz0 = sbs + 16;                   // [16]
    const uint32_t bars = smem_u32(sz0 + 16);                     // 2 slots x 7 barriers, then the drain barrier
    const uint32_t bar_drain = bars + 2 * 56;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sz0 + 16 + 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sz0 + 16 + 34);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- one-time set-up: operand image, side tables, barriers, TMEM --------------------------------
    {
        const float4* src = reinterpret_cast<const float4*>(a.image);
        float4* dst = reinterpret_cast<float4*>(gen);
        for (uint32_t i = threadIdx.x; i < image_bytes / 16; i += kChainTcThreads) dst[i] = src[i];
        for (int i = threadIdx.x; i < H; i += kChainTcThreads) {
            sbzs[i] = a.bz[i];
            sbg1[i] = a.bg1[i];
            sbh1[i] = a.bh1[i];
            sbi1[i] = a.bi1[i];
        }
        for (int i = threadIdx.x; i < W * H; i += kChainTcThreads) slr[i] = (a.hlr[i] + a.hlr[W * H + i]) * (1.0f / 3.0f);
        for (int i = threadIdx.x; i < 256; i += kChainTcThreads) {
            sWsig[i] = a.Wsig[i];
            sWl[i] = a.Wl[i];
        }
        if (threadIdx.x < 16) {
            sbmu[threadIdx.x] = a.bmu[threadIdx.x];
            sbsig[threadIdx.x] = a.bsig[threadIdx.x];
            sbg2[threadIdx.x] = a.bg2[threadIdx.x];
            sbh2[threadIdx.x] = a.bh2[threadIdx.x];
            sbl[threadIdx.x] = a.bl[threadIdx.x];
            sbs[threadIdx.x] = a.bs[threadIdx.x];
            sz0[threadIdx.x] = a.z0[threadIdx.x];
        }
    }
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < 2; ++s) {
            const uint32_t b0 = bars + 56 * s;
            mbar_init(b0, kChainEpiWarps);           // latent tile (or relu(G)) ready
            mbar_init(b0 + 8, 1);                    // hidden pre-activations ready
            mbar_init(b0 + 16, kChainEpiWarps);      // hidden chunk buffer 0 written
            mbar_init(b0 + 24, kChainEpiWarps);      // hidden chunk buffer 1 written
            mbar_init(b0 + 32, 1);                   // hidden chunk buffer 0 multiplied
            mbar_init(b0 + 40, 1);                   // hidden chunk buffer 1 multiplied
            mbar_init(b0 + 48, 1);                   // second result ready
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_proxy_async();          // the operand image was written with ordinary stores; the MMAs read it asynchronously
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    ChainSlot slot[2];
#pragma unroll
    for (uint32_t s = 0; s < 2; ++s) {
        const uint32_t b0 = bars + 56 * s;
        slot[s].t_z = t_act + s * 16384u;
        slot[s].t_hb = t_act + 2 * 16384u + s * 32768u;
        slot[s].tmem = tmem_base + s * 256u;
        slot[s].bar_z = b0; slot[s].bar_p = b0 + 8; slot[s].bar_h = b0 + 16; slot[s].bar_hfree = b0 + 32;
        slot[s].bar_acc2 = b0 + 48;
        slot[s].nz = slot[s].np = slot[s].na = slot[s].nu = 0;
        slot[s].tile = -1;
    }
    const int n_tiles = ceil_div(a.count, 128);
    const int ph_gate = W, ph_prop = W + 1, ph_emit = W + 2, n_phases = W + 3;
    // The second results of a tile (16 columns each) reuse the first columns of the tile's pre-activation block:
    // those are multiplied only after every warp has read chunk 0.

    if (warp == 0) {
        // ---------------- MMA issuer -------------------------------------------------------------------
        const uint32_t idesc_h = instr_desc_tf32(H), idesc_16 = instr_desc_tf32(16);
        bool ok = true;
        for (int t0 = blockIdx.x; ok && t0 < n_tiles; t0 += 2 * gridDim.x) {
            slot[0].tile = t0;
            slot[1].tile = t0 + static_cast<int>(gridDim.x) < n_tiles ? t0 + static_cast<int>(gridDim.x) : -1;
            for (int ph = 0; ok && ph < n_phases; ++ph) {
#pragma unroll
                for (int s = 0; s < 2; ++s) {                       // first GEMM of both tiles
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    ok = mbar_wait(sl.bar_z, sl.nz & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.nz;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t b_tile = ph < ph_gate ? t_zg : (ph == ph_gate ? t_zg + 64u : (ph == ph_prop ? t_hi : t_hi + 64u));
                        const uint64_t a_desc = make_smem_desc(sl.t_z), b_desc = make_smem_desc(b_tile);
                        umma_tf32(sl.tmem, a_desc, b_desc, idesc_h, 0u);
                        umma_tf32(sl.tmem, a_desc + 2, b_desc + 2, idesc_h, 1u);
                        umma_commit(sl.bar_p);
                    }
                    __syncwarp();
                }
                if (ph == ph_emit) continue;                       // the first emission layer has no second GEMM here
                const uint32_t b_base = ph < ph_gate ? t_wmu : (ph == ph_gate ? t_wg2 : t_wh2);
#pragma unroll
                for (int s = 0; s < 2; ++s) {                       // second GEMM, chunk by chunk as the epilogue delivers
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    for (int c = 0; c < n_chunks; ++c, ++sl.nu) {
                        const uint32_t b = sl.nu & 1u;
                        ok = mbar_wait(sl.bar_h + 8 * b, (sl.nu >> 1) & 1u, abort_flag, a.st);
                        if (!ok) break;
                        tc_fence_after();
                        if (lane == 0) {
                            const uint64_t a_desc = make_smem_desc(sl.t_hb + b * 16384u);
                            const uint64_t b_desc = make_smem_desc(b_base + c * (16u * 128u));
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_tf32(sl.tmem, a_desc + 2 * k, b_desc + 2 * k, idesc_16, (c | k) != 0 ? 1u : 0u);
                            umma_commit(sl.bar_hfree + 8 * b);
                            if (c == n_chunks - 1) umma_commit(sl.bar_acc2);
                        }
                        __syncwarp();
                    }
                }
                if (ph != ph_prop) continue;
#pragma unroll
                for (int s = 0; s < 2; ++s) {                       // scale: Ws relu(G), relu(G) sits in the latent tile
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    ok = mbar_wait(sl.bar_z, sl.nz & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.nz;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint64_t a_desc = make_smem_desc(sl.t_z), b_desc = make_smem_desc(t_ws);
                        umma_tf32(sl.tmem, a_desc, b_desc, idesc_16, 0u);
                        umma_tf32(sl.tmem, a_desc + 2, b_desc + 2, idesc_16, 1u);
                        umma_commit(sl.bar_acc2);
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
        const int row = q * 32 + lane;                                            // TMEM lane = sample of the tile
        const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t step = a.st->step;
        float gate_own[2][4], lin_own[2][4], G_own[2][4];                         // per tile in flight, latent dimensions 4cg..4cg+3
        bool ok = true;
        for (int t0 = blockIdx.x; ok && t0 < n_tiles; t0 += 2 * gridDim.x) {
            slot[0].tile = t0;
            slot[1].tile = t0 + static_cast<int>(gridDim.x) < n_tiles ? t0 + static_cast<int>(gridDim.x) : -1;
#pragma unroll
            for (int s = 0; s < 2; ++s) {                           // initial latent z_{T-l-1} of both tiles
                if (slot[s].tile < 0) continue;
                st_shared_v4(slot[s].t_z + sw128(row, cg), tf32_rna(sz0[4 * cg + 0]), tf32_rna(sz0[4 * cg + 1]),
                             tf32_rna(sz0[4 * cg + 2]), tf32_rna(sz0[4 * cg + 3]));
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(slot[s].bar_z);
            }
            for (int ph = 0; ok && ph < n_phases; ++ph) {
                const float* bias = ph < ph_gate ? sbzs : (ph == ph_gate ? sbg1 : (ph == ph_prop ? sbh1 : sbi1));
                const float* lr = slr + (ph < ph_gate ? ph : 0) * H;
                // ---- hidden layer of both tiles: bias, activation, next A operand (or u) -----------------
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    ok = mbar_wait(sl.bar_p, sl.np & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.np;
                    tc_fence_after();
                    const int k = sl.tile * 128 + row;
                    for (int c = 0; c < n_chunks; ++c) {
                        const int col0 = c * 32 + cg * 8;
                        uint32_t acc[8];
                        tmem_ld8(sl.tmem + lane_off + col0, acc);
                        tmem_ld_wait();
                        const float4 b_lo = *reinterpret_cast<const float4*>(bias + col0);
                        const float4 b_hi = *reinterpret_cast<const float4*>(bias + col0 + 4);
                        const float bv[8] = {b_lo.x, b_lo.y, b_lo.z, b_lo.w, b_hi.x, b_hi.y, b_hi.z, b_hi.w};
                        float h[8];
                        if (ph < ph_gate) {
                            const float4 l_lo = *reinterpret_cast<const float4*>(lr + col0);
                            const float4 l_hi = *reinterpret_cast<const float4*>(lr + col0 + 4);
                            const float lv[8] = {l_lo.x, l_lo.y, l_lo.z, l_lo.w, l_hi.x, l_hi.y, l_hi.z, l_hi.w};
#pragma unroll
                            for (int i = 0; i < 8; ++i) {          // tanh, then (tanh + h_left + h_right) / 3
                                float t;                                   // tanh by the hardware instruction (chain_tc.cuh)
                                asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(__uint_as_float(acc[i]) + bv[i]));
                                h[i] = fmaf(t, 1.0f / 3.0f, lv[i]);
                            }
                        } else if (ph < ph_emit) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) h[i] = fmaxf(__uint_as_float(acc[i]) + bv[i], 0.0f);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) h[i] = __uint_as_float(acc[i]) + bv[i];
                        }
                        if (ph < ph_emit) {
                            const uint32_t b = sl.nu & 1u;
                            if (sl.nu >= 2) {                      // the buffer's previous contents must have been multiplied
                                ok = mbar_wait(sl.bar_hfree + 8 * b, ((sl.nu >> 1) - 1u) & 1u, abort_flag, a.st);
                                if (!ok) break;
                            }
                            const uint32_t dst = sl.t_hb + b * 16384u;
                            st_shared_v4(dst + sw128(row, 2 * cg), tf32_rna(h[0]), tf32_rna(h[1]), tf32_rna(h[2]), tf32_rna(h[3]));
                            st_shared_v4(dst + sw128(row, 2 * cg + 1), tf32_rna(h[4]), tf32_rna(h[5]), tf32_rna(h[6]), tf32_rna(h[7]));
                            fence_proxy_async();
                            tc_fence_before();                     // our TMEM reads of this chunk precede the MMAs it unblocks
                            __syncwarp();
                            if (lane == 0) mbar_arrive(sl.bar_h + 8 * b);
                            ++sl.nu;
                        } else if (k < a.count) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) h[i] = tf32_rna(h[i]);
                            store8(a.u_out + static_cast<size_t>(k) * H + col0, h);          // one whole 32-byte sector
                        }
                    }
                }
                if (!ok || ph == ph_emit) continue;
                // ---- second result of both tiles ----------------------------------------------------------
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    ok = mbar_wait(sl.bar_acc2, sl.na & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.na;
                    tc_fence_after();
                    const uint32_t sample = a.sample_base + static_cast<uint32_t>(sl.tile * 128 + row);
                    uint32_t res_bits[16];
                    tmem_ld16(sl.tmem + lane_off, res_bits);
                    tmem_ld_wait();
                    float own[4];                                   // this thread's four of the 16 results
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        own[c] = 0.0f;
#pragma unroll
                        for (int gg = 0; gg < 4; ++gg)
                            if (gg == cg) own[c] = __uint_as_float(res_bits[4 * gg + c]);
                    }
                    if (ph < ph_gate) {
                        // guide: z = mu + softplus(Wsig mu + bsig) * eps
                        float mu[16];
#pragma unroll
                        for (int d = 0; d < 16; ++d) mu[d] = __uint_as_float(res_bits[d]) + sbmu[d];
                        float eps[4], z_own[4];
                        normal4_fast(static_cast<uint32_t>(cg), sample, static_cast<uint32_t>(ph), step, a.key.seed_lo, a.key.seed_hi, eps);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float* wrow = sWsig + (4 * cg + c) * 16;
                            float pre = sbsig[4 * cg + c];
#pragma unroll
                            for (int e = 0; e < 16; ++e) pre = fmaf(wrow[e], mu[e], pre);
                            z_own[c] = fmaf(softplus_fast(pre), eps[c], own[c] + sbmu[4 * cg + c]);
                        }
                        st_shared_v4(sl.t_z + sw128(row, cg), tf32_rna(z_own[0]), tf32_rna(z_own[1]), tf32_rna(z_own[2]), tf32_rna(z_own[3]));
                        fence_proxy_async();
                    } else if (ph == ph_gate) {
                        // gate g, and the linear map Wl z + bl from the latent tile (it stays as it is for the proposal)
                        float z[16];
#pragma unroll
                        for (int e4 = 0; e4 < 4; ++e4) {
                            const float4 v = ld_shared_v4(sl.t_z + sw128(row, e4));
                            z[4 * e4 + 0] = v.x; z[4 * e4 + 1] = v.y; z[4 * e4 + 2] = v.z; z[4 * e4 + 3] = v.w;
                        }
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            gate_own[s][c] = sigmoid_fast(own[c] + sbg2[4 * cg + c]);
                            const float* wrow = sWl + (4 * cg + c) * 16;
                            float lin = sbl[4 * cg + c];
#pragma unroll
                            for (int e = 0; e < 16; ++e) lin = fmaf(wrow[e], z[e], lin);
                            lin_own[s][c] = lin;
                        }
                    } else {
                        // proposal h -> G = (1 - g) * lin + g * h; relu(G) replaces the latent tile for the scale product
                        float r[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float prop = own[c] + sbh2[4 * cg + c];
                            G_own[s][c] = fmaf(gate_own[s][c], prop - lin_own[s][c], lin_own[s][c]);
                            r[c] = tf32_rna(fmaxf(G_own[s][c], 0.0f));
                        }
                        st_shared_v4(sl.t_z + sw128(row, cg), r[0], r[1], r[2], r[3]);
                        fence_proxy_async();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(sl.bar_z);
                }
                if (!ok || ph != ph_prop) continue;
                // ---- scale of both tiles: z' = G + softplus(Ws relu(G) + bs) * eps ---------------------------
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    ok = mbar_wait(sl.bar_acc2, sl.na & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.na;
                    tc_fence_after();
                    const uint32_t sample = a.sample_base + static_cast<uint32_t>(sl.tile * 128 + row);
                    uint32_t res_bits[16];
                    tmem_ld16(sl.tmem + lane_off, res_bits);
                    tmem_ld_wait();
                    float eps[4], z_own[4];
                    normal4_fast(static_cast<uint32_t>(cg), sample, kStreamTransition, step, a.key.seed_lo, a.key.seed_hi, eps);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float pre = 0.0f;
#pragma unroll
                        for (int gg = 0; gg < 4; ++gg)
                            if (gg == cg) pre = __uint_as_float(res_bits[4 * gg + c]);
                        z_own[c] = fmaf(softplus_fast(pre + sbs[4 * cg + c]), eps[c], G_own[s][c]);
                    }
                    st_shared_v4(sl.t_z + sw128(row, cg), tf32_rna(z_own[0]), tf32_rna(z_own[1]), tf32_rna(z_own[2]), tf32_rna(z_own[3]));
                    fence_proxy_async();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(sl.bar_z);
                }
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
