// Per-sample chain (guide steps, transition, first emission layer) on the tcgen05 tensor cores,
// for latent size 16 and hidden width 64..256, operands in tf32.  One kernel template serves both model
// variants: the compact one (transition = one hidden layer with a [mean | logvar] head, then the emission's
// hidden layer v) and the networks as Section 3.1.3 prints them (LITERAL: gated transition
//      g = sigmoid(Wg2 relu(Wg1 z + bg1) + bg2)        h = Wh2 relu(Wh1 z + bh1) + bh2
//      G = (1 - g) * (Wl z + bl) + g * h               H = softplus(Ws relu(G) + bs)        z' = G + H * eps
// then the affine first layer of the emission mean, u = Wi1 z' + bi1).
//
// A CTA walks over tiles of 128 samples; sample r of the tile is TMEM lane r.  Every layer pair
//      hidden = act(A z + a)          (M=128, N=H, K=16)
//      out    = B hidden (+ b)        (M=128, N=16 or 32, K=H)
// is two UMMA groups.  The first writes the hidden pre-activations to TMEM columns [0, H); the
// epilogue warps read them 64 hidden units ("chunk") at a time, apply bias and activation, round
// to tf32 and store the chunk as two K-major, 128-byte-swizzled A operand tiles in the buffer of
// the tile's slot; the MMA warp multiplies that chunk with the matching K blocks of B while the
// epilogue produces the same chunk of the other tile in flight.  The second result (mu; mean | logvar; gate;
// proposal) is read back by all epilogue warps, which draw the noise, form the next latent and store it as the
// next A operand.  In the literal variant the proposal's result is combined with the gate and the linear map
// (computed by the epilogue threads from the latent tile) into G, relu(G) then takes the place of the latent
// tile and one more small product with Ws gives the scale.
// The last layer's hidden vector (v, or u) goes to global memory for the emission output GEMMs.
//
// All weight operands live in shared memory for the whole kernel: the host prepares their
// swizzled image once, the CTA copies it in at start.  Latent rows are 128 bytes wide (32 tf32)
// although K = 16: two first-layer matrices share one tile (columns 0..15 and 16..31: [Wz | W1], or
// [Wz | Wg1] and [Wh1 | Wi1]), so the MMA for the second of them simply starts 64 bytes into the rows.
//
// Warp 0 issues the MMAs and owns TMEM; warps 1..16 are the epilogue: warp w serves TMEM lanes
// 32*(w%4).. and column group cg = (w-1)/4: 16 of each chunk's 64 columns and the latent
// dimensions 4cg..4cg+3 (one Philox call per stream and sample, as everywhere else).
// Every mbarrier wait is bounded (see async.cuh).
#pragma once
#include "emit_tc.cuh"

namespace cutoff {
namespace tc {

constexpr int kChainEpiWarps = 16;
constexpr int kChainTcThreads = (1 + kChainEpiWarps) * 32;
constexpr int kChainD = 16;

struct ChainTcArgs {
    // swizzled operand tiles.  compact: [Wz|W1] (H x 32), W3 (H x 32), Wmu (H/32 x 16 x 32), W2 (H/32 x 32 x 32);
    // literal: [Wz|Wg1] (H x 32), [Wh1|Wi1] (H x 32), Wmu, Wg2, Wh2 (H/32 x 16 x 32 each), Ws (16 x 32)
    const float* image;
    // compact: b1, b3 = biases of the transition's and the emission's hidden layer, b2 = [mean | logvar] bias (32);
    // literal: b1 = bg1, b3 = bh1, b2 unused
    const float *bz, *b1, *b3, *bmu, *bsig, *Wsig, *b2, *z0;
    const float *bi1, *bg2, *bh2, *Wl, *bl, *bs;       // literal variant only
    const float* hlr;           // [2][W][H] h_left, h_right
    DevState* st;
    NoiseKey key;
    uint32_t sample_base;
    int count, H, W, round_v;   // round_v: round v to tf32 (compact; u of the literal variant always is)
    float* v_out;               // [count][H]
};

inline size_t chain_tc_image_floats(int H, bool literal = false) {
    return literal ? static_cast<size_t>(H) * (32 + 32 + 16 + 16 + 16) + 16 * 32 : static_cast<size_t>(H) * (32 + 32 + 16 + 32);
}

inline size_t chain_tc_smem_bytes(int H, int W, bool literal = false) {
    const size_t tiles = chain_tc_image_floats(H, literal) * 4 + 2 * 128 * 128 /*Z x2*/ + 4 * 128 * 128 /*hidden chunks: 2 per slot*/;
    const size_t floats = literal ? 4 * static_cast<size_t>(H) + static_cast<size_t>(W) * H + 2 * 16 * 16 + 7 * 16
                                  : 3 * static_cast<size_t>(H) + static_cast<size_t>(W) * H + 16 * 16 + 16 + 16 + 32 + 16;
    return 1024 + tiles + floats * 4 + 256;
}

// byte offset of the 16-byte chunk `chunk` of row `row` in a K-major tile with 128-byte swizzled rows
__device__ __forceinline__ uint32_t sw128(int row, int chunk) {
    return static_cast<uint32_t>((row >> 3) * 1024 + (row & 7) * 128 + ((chunk ^ (row & 7)) << 4));
}

__device__ __forceinline__ uint32_t instr_desc_tf32(int n) {      // D = f32, A = B = tf32, K-major, M = 128
    return (1u << 4) | (2u << 7) | (2u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | ((128u >> 4) << 24);
}

// Round to tf32 (nearest, ties away from zero) with two integer instructions instead of the conversion instruction,
// which shares the slow special-function pipe with tanh: add half a unit of the 13 dropped bits to the magnitude,
// clear them.  The same bits as cvt.rna.tf32.f32 for every finite value (an overflow of the mantissa carries into
// the exponent, as it should).
__device__ __forceinline__ float tf32_rna(float x) {
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

__device__ __forceinline__ float softplus_fast(float x) {          // ln(1 + e^x)
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 1.4426950408889634f));
    return x > 15.0f ? x : 0.6931471805599453f * __log2f(1.0f + e);
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

// One of the two tiles a CTA has in flight: its shared-memory operands, TMEM columns and barriers,
// and how many times each barrier has completed (both roles count the same sequence).
struct ChainSlot {
    uint32_t t_z;            // latent A operand [128 x 128 B]
    uint32_t t_hb;           // two hidden-chunk A operands [128 x 128 B] each
    uint32_t tmem;           // first of the slot's 256 TMEM columns
    uint32_t bar_z, bar_p, bar_h, bar_hfree, bar_acc2;     // bar_h, bar_hfree: two barriers each
    uint32_t nz, np, na, nu;
    int tile;                // current tile, -1 if the slot is idle
};

template <bool LITERAL>
__global__ void __launch_bounds__(kChainTcThreads, 1) k_chain_tc(ChainTcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const int H = a.H, W = a.W;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - raw);
    // weight operand tiles
    const uint32_t t_in0 = base;                                  // [Wz | W1]   or [Wz | Wg1]
    const uint32_t t_in1 = t_in0 + H * 128;                       // W3          or [Wh1 | Wi1]
    const uint32_t t_wmu = t_in1 + H * 128;
    const uint32_t t_out1 = t_wmu + H * 64;                       // W2 (32 rows per K block) or Wg2 (16 rows)
    const uint32_t t_out2 = t_out1 + H * 64;                      // literal: Wh2
    const uint32_t t_ws = t_out2 + H * 64;                        // literal: Ws, 16 rows x 128 bytes
    const uint32_t image_bytes = static_cast<uint32_t>(H) * 448u + (LITERAL ? 2048u : 0u);
    const uint32_t t_act = base + image_bytes;                    // Z0, Z1, then 4 hidden-chunk buffers: 6 x 16 KB
    // fp32 side tables
    float* sbzs = reinterpret_cast<float*>(gen + image_bytes + 6 * 16384);    // bz
    float* sb1 = sbzs + H;
    float* sb3 = sb1 + H;
    float* sbi1 = sb3 + H;                   // literal only
    float* slr = sb3 + (LITERAL ? 2 : 1) * H;        // [W][H]  (h_left + h_right) / 3
    float* sWsig = slr + W * H;              // [16][16]
    float* sWl = sWsig + 256;                // [16][16], literal only
    float* sbmu = sWsig + (LITERAL ? 512 : 256);
    float* sbsig = sbmu + 16;
    float* sb2 = sbsig + 16;                 // compact: [32]
    float* sbg2 = sbsig + 16;                // literal: bg2, bh2, bl, bs, 16 each
    float* sbh2 = sbg2 + 16;
    float* sbl = sbh2 + 16;
    float* sbs = sbl + 16;
    float* sz0 = LITERAL ? sbs + 16 : sb2 + 32;      // [16]
    const uint32_t bars = smem_u32(sz0 + 16);                     // 2 slots x 7 barriers, then the drain barrier
    const uint32_t bar_drain = bars + 2 * 56;
    const uint32_t bar_img = bar_drain + 8;                       // the operand image has landed
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sz0 + 16 + 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sz0 + 16 + 34);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- one-time set-up: barriers, operand image (bulk copies, while the side tables are filled), TMEM ----------
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
        mbar_init(bar_img, 1);
        *abort_flag = 0;
        fence_barrier_init();
        mbar_arrive_expect_tx(bar_img, image_bytes);
        for (uint32_t off = 0; off < image_bytes; off += 32768u) {
            const uint32_t n = image_bytes - off < 32768u ? image_bytes - off : 32768u;
            bulk_load_1d(base + off, reinterpret_cast<const uint8_t*>(a.image) + off, n, bar_img);
        }
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // up to here nothing an earlier kernel of the stream writes has been touched (the image and the biases are
    // weights): the encoder's states and the device state come after this point
    dependency_wait();
    launch_dependents();
    {
        for (int i = threadIdx.x; i < H; i += kChainTcThreads) {
            sbzs[i] = a.bz[i];
            sb1[i] = a.b1[i];
            sb3[i] = a.b3[i];
            if (LITERAL) sbi1[i] = a.bi1[i];
        }
        for (int i = threadIdx.x; i < W * H; i += kChainTcThreads) slr[i] = (a.hlr[i] + a.hlr[W * H + i]) * (1.0f / 3.0f);
        for (int i = threadIdx.x; i < 256; i += kChainTcThreads) {
            sWsig[i] = a.Wsig[i];
            if (LITERAL) sWl[i] = a.Wl[i];
        }
        if (threadIdx.x < 16) {
            sbmu[threadIdx.x] = a.bmu[threadIdx.x];
            sbsig[threadIdx.x] = a.bsig[threadIdx.x];
            sz0[threadIdx.x] = a.z0[threadIdx.x];
            if (LITERAL) {
                sbg2[threadIdx.x] = a.bg2[threadIdx.x];
                sbh2[threadIdx.x] = a.bh2[threadIdx.x];
                sbl[threadIdx.x] = a.bl[threadIdx.x];
                sbs[threadIdx.x] = a.bs[threadIdx.x];
            }
        }
        if (!LITERAL && threadIdx.x < 32) sb2[threadIdx.x] = a.b2[threadIdx.x];
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // nothing starts before the weights are in place; if they never arrive every role skips its loop
    const bool image_ok = mbar_wait(bar_img, 0u, abort_flag, a.st);

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
    const int n_tiles = image_ok ? ceil_div(a.count, 128) : 0;
    // phases: W guide steps, then transition and emission hidden layer -- or gate, proposal (+ scale), first emission layer
    const int n_phases = LITERAL ? W + 3 : W + 2;
    const int ph_last = n_phases - 1;                             // its hidden layer goes to global memory, no second GEMM
    // The second result of a tile (16 columns; mean | logvar: 32) reuses the first columns of the tile's
    // pre-activation block: those are multiplied only after every warp has read chunk 0.

    // A hidden layer goes to the second GEMM in chunks of 64 units (two K blocks).  Each slot has one chunk buffer
    // (its two 16 KB tiles); the chunks of the two tiles in flight are produced alternately -- (chunk 0, slot 0),
    // (chunk 0, slot 1), (chunk 1, slot 0), ... -- so a slot's buffer is being multiplied while the other slot's is
    // written, and both roles walk the same order.  sl.nu counts a slot's chunks: chunk n completes phase n of
    // bar_h (written) and of bar_hfree (multiplied).
    const int n_chunks64 = H / 64;

    if (warp == 0) {
        // ---------------- MMA issuer -------------------------------------------------------------------
        const uint32_t idesc_h = instr_desc_tf32(H), idesc_16 = instr_desc_tf32(16), idesc_head = instr_desc_tf32(32);
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
                        const uint32_t b_tile = ph < W ? t_in0 : (ph == W ? t_in0 + 64u : (ph == W + 1 ? t_in1 : t_in1 + 64u));
                        const uint64_t a_desc = make_smem_desc(sl.t_z), b_desc = make_smem_desc(b_tile);
                        umma_tf32(sl.tmem, a_desc, b_desc, idesc_h, 0u);
                        umma_tf32(sl.tmem, a_desc + 2, b_desc + 2, idesc_h, 1u);
                        umma_commit(sl.bar_p);
                    }
                    __syncwarp();
                }
                if (ph == ph_last) continue;                       // the last hidden layer has no second GEMM here
                const uint32_t b_base = ph < W ? t_wmu : (ph == W ? t_out1 : t_out2);
                const uint32_t slab = LITERAL || ph < W ? 16u * 128u : 32u * 128u;
                const uint32_t idesc2 = LITERAL || ph < W ? idesc_16 : idesc_head;
                for (int c = 0; ok && c < n_chunks64; ++c) {        // second GEMM, chunk by chunk as the epilogue delivers
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        ChainSlot& sl = slot[s];
                        if (!ok || sl.tile < 0) continue;
                        ok = mbar_wait(sl.bar_h, sl.nu & 1u, abort_flag, a.st);
                        if (!ok) continue;
                        ++sl.nu;
                        tc_fence_after();
                        if (lane == 0) {
#pragma unroll
                            for (int kb = 0; kb < 2; ++kb) {
                                const uint64_t a_desc = make_smem_desc(sl.t_hb + kb * 16384u);
                                const uint64_t b_desc = make_smem_desc(b_base + (2 * c + kb) * slab);
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    umma_tf32(sl.tmem, a_desc + 2 * k, b_desc + 2 * k, idesc2, (c | kb | k) != 0 ? 1u : 0u);
                            }
                            umma_commit(sl.bar_hfree);
                            if (c == n_chunks64 - 1) umma_commit(sl.bar_acc2);
                        }
                        __syncwarp();
                    }
                }
                if (!LITERAL || ph != W + 1) continue;
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
        const uint32_t hb_off = static_cast<uint32_t>(cg >> 1) * 16384u;          // K block of the chunk this warp writes
        const int hb_chunk = 4 * (cg & 1);                                        // its first 16-byte chunk in a row
        float gate_own[2][4], lin_own[2][4], G_own[2][4];     // literal: per tile in flight, latent dimensions 4cg..4cg+3
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
                const float* bias = ph < W ? sbzs : (ph == W ? sb1 : (ph == W + 1 ? sb3 : sbi1));
                const float* lr = slr + (ph < W ? ph : 0) * H;
                // ---- hidden layer of both tiles: bias, activation, next A operand (or v) -----------------
                for (int c = 0; ok && c < n_chunks64; ++c) {
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        ChainSlot& sl = slot[s];
                        if (!ok || sl.tile < 0) continue;
                        if (c == 0) {
                            ok = mbar_wait(sl.bar_p, sl.np & 1u, abort_flag, a.st);
                            if (!ok) continue;
                            ++sl.np;
                            tc_fence_after();
                        }
                        const int col0 = c * 64 + cg * 16;
                        uint32_t acc[16];
                        tmem_ld16(sl.tmem + lane_off + col0, acc);
                        tmem_ld_wait();
                        float h[16];
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const float4 bq = *reinterpret_cast<const float4*>(bias + col0 + 4 * g);
                            const float bv[4] = {bq.x, bq.y, bq.z, bq.w};
                            if (ph < W) {
                                const float4 lq = *reinterpret_cast<const float4*>(lr + col0 + 4 * g);
                                const float lv[4] = {lq.x, lq.y, lq.z, lq.w};
#pragma unroll
                                for (int i = 0; i < 4; ++i) {      // tanh, then (tanh + h_left + h_right) / 3
                                    float t;
                                    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(__uint_as_float(acc[4 * g + i]) + bv[i]));
                                    h[4 * g + i] = fmaf(t, 1.0f / 3.0f, lv[i]);
                                }
                            } else if (LITERAL && ph == ph_last) {  // u = Wi1 z' + bi1: no activation
#pragma unroll
                                for (int i = 0; i < 4; ++i) h[4 * g + i] = __uint_as_float(acc[4 * g + i]) + bv[i];
                            } else {
#pragma unroll
                                for (int i = 0; i < 4; ++i) h[4 * g + i] = fmaxf(__uint_as_float(acc[4 * g + i]) + bv[i], 0.0f);
                            }
                        }
                        if (ph != ph_last) {
                            if (sl.nu >= 1) {                      // the buffer's previous contents must have been multiplied
                                ok = mbar_wait(sl.bar_hfree, (sl.nu - 1u) & 1u, abort_flag, a.st);
                                if (!ok) continue;
                            }
                            const uint32_t dst = sl.t_hb + hb_off;
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                st_shared_v4(dst + sw128(row, hb_chunk + g), tf32_rna(h[4 * g]), tf32_rna(h[4 * g + 1]),
                                             tf32_rna(h[4 * g + 2]), tf32_rna(h[4 * g + 3]));
                            fence_proxy_async();
                            tc_fence_before();                     // our TMEM reads of this chunk precede the MMAs it unblocks
                            __syncwarp();
                            if (lane == 0) mbar_arrive(sl.bar_h);
                            ++sl.nu;
                        } else {
                            const int k = sl.tile * 128 + row;
                            if (k < a.count) {
                                if (LITERAL || a.round_v) {
#pragma unroll
                                    for (int i = 0; i < 16; ++i) h[i] = tf32_rna(h[i]);
                                }
                                store8(a.v_out + static_cast<size_t>(k) * H + col0, h);          // whole 32-byte sectors
                                store8(a.v_out + static_cast<size_t>(k) * H + col0 + 8, h + 8);
                            }
                        }
                    }
                }
                if (!ok || ph == ph_last) continue;
                // ---- second result of both tiles: the next latent (literal: gate, then G and relu(G)) ------------
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    const uint32_t sample = a.sample_base + static_cast<uint32_t>(sl.tile * 128 + row);
                    float eps[4];                                   // drawn before the wait: the noise does not depend on the result
                    if (!LITERAL || ph < W)
                        normal4_fast(static_cast<uint32_t>(cg), sample, ph < W ? static_cast<uint32_t>(ph) : kStreamTransition, step,
                                     a.key.seed_lo, a.key.seed_hi, eps);
                    ok = mbar_wait(sl.bar_acc2, sl.na & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.na;
                    tc_fence_after();
                    float z_own[4];
                    bool store_z = true;
                    if (ph < W) {
                        // guide: z = mu + softplus(Wsig mu + bsig) * eps
                        uint32_t mu_bits[16];
                        tmem_ld16(sl.tmem + lane_off, mu_bits);
                        tmem_ld_wait();
                        float mu[16];
#pragma unroll
                        for (int d = 0; d < 16; ++d) mu[d] = __uint_as_float(mu_bits[d]) + sbmu[d];
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float* wrow = sWsig + (4 * cg + c) * 16;
                            float pre = sbsig[4 * cg + c];
#pragma unroll
                            for (int e = 0; e < 16; ++e) pre = fmaf(wrow[e], mu[e], pre);
                            float own = 0.0f;
#pragma unroll
                            for (int gg = 0; gg < 4; ++gg)
                                if (gg == cg) own = mu[4 * gg + c];
                            z_own[c] = fmaf(softplus_fast(pre), eps[c], own);
                        }
                    } else if constexpr (!LITERAL) {
                        uint32_t mean_bits[16], lv_bits[16];
                        tmem_ld16(sl.tmem + lane_off, mean_bits);
                        tmem_ld16(sl.tmem + lane_off + 16, lv_bits);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            float mean = 0.0f, lv = 0.0f;
#pragma unroll
                            for (int gg = 0; gg < 4; ++gg)
                                if (gg == cg) { mean = __uint_as_float(mean_bits[4 * gg + c]); lv = __uint_as_float(lv_bits[4 * gg + c]); }
                            z_own[c] = fmaf(exp_half_fast(lv + sb2[16 + 4 * cg + c]), eps[c], mean + sb2[4 * cg + c]);
                        }
                    } else {
                        uint32_t res_bits[16];
                        tmem_ld16(sl.tmem + lane_off, res_bits);
                        tmem_ld_wait();
                        float own[4];                               // this thread's four of the 16 results
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            own[c] = 0.0f;
#pragma unroll
                            for (int gg = 0; gg < 4; ++gg)
                                if (gg == cg) own[c] = __uint_as_float(res_bits[4 * gg + c]);
                        }
                        if (ph == W) {
                            // gate g, and the linear map Wl z + bl from the latent tile (it stays as it is for the proposal)
                            float z[16];
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 zq = ld_shared_v4(sl.t_z + sw128(row, e4));
                                z[4 * e4 + 0] = zq.x; z[4 * e4 + 1] = zq.y; z[4 * e4 + 2] = zq.z; z[4 * e4 + 3] = zq.w;
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
                            store_z = false;
                        } else {
                            // proposal h -> G = (1 - g) * lin + g * h; relu(G) replaces the latent tile for the scale product
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float prop = own[c] + sbh2[4 * cg + c];
                                G_own[s][c] = fmaf(gate_own[s][c], prop - lin_own[s][c], lin_own[s][c]);
                                z_own[c] = fmaxf(G_own[s][c], 0.0f);
                            }
                        }
                    }
                    if (store_z) {
                        st_shared_v4(sl.t_z + sw128(row, cg), tf32_rna(z_own[0]), tf32_rna(z_own[1]), tf32_rna(z_own[2]), tf32_rna(z_own[3]));
                        fence_proxy_async();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(sl.bar_z);
                }
                if (!LITERAL || !ok || ph != W + 1) continue;
                // ---- literal: scale of both tiles, z' = G + softplus(Ws relu(G) + bs) * eps ------------------
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    ChainSlot& sl = slot[s];
                    if (!ok || sl.tile < 0) continue;
                    const uint32_t sample = a.sample_base + static_cast<uint32_t>(sl.tile * 128 + row);
                    float eps[4], z_own[4];
                    normal4_fast(static_cast<uint32_t>(cg), sample, kStreamTransition, step, a.key.seed_lo, a.key.seed_hi, eps);
                    ok = mbar_wait(sl.bar_acc2, sl.na & 1u, abort_flag, a.st);
                    if (!ok) continue;
                    ++sl.na;
                    tc_fence_after();
                    uint32_t res_bits[16];
                    tmem_ld16(sl.tmem + lane_off, res_bits);
                    tmem_ld_wait();
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
