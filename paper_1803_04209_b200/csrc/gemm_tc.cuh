// The emission of the literal model variant (Section 3.1.3) on the 5th-generation tensor cores (tcgen05, kind::tf32):
//   I = Wi2 u + bi2        r = relu(Wj1 I + bj1)        x = I + softplus(Wj2 r + bj2) * eps,      u = Wi1 z' + bi1.
// I = MLP_2(z, Identity, Identity) is affine in u, so the hidden layer of the scale does not need I:
//   Wj1 I + bj1 = (Wj1 Wi2) u + (Wj1 bi2 + bj1) = M u + b',
// with the H x H matrix M and the vector b' formed once when the weights are loaded.  Two kernels remain:
//   k_gemm_relu_tc   r = relu(u M^T + b')                       (K = H instead of K = N)
//   k_emit_dual_tc   x = (u Wi2^T + bi2) + softplus(r Wj2^T + bj2) * eps,  both products in one accumulator.
//
// k_gemm_relu_tc has the pipeline of the emission kernel of emit_tc.cuh: one persistent CTA per SM walks over output
// tiles of 128 rows x 256 columns; a tile is one accumulator of 128 TMEM lanes x 256 fp32 columns,
// filled by UMMA instructions of shape M=128, N=256, K=8; operands arrive by plain per-CTA TMA loads
// (boxes of 128 rows x 32 tf32, 128-byte swizzle; rows or columns outside the matrices read as zero)
// into a 4-stage ring; the accumulator is double-buffered.  Warp 0 loads, warp 1 issues the MMAs,
// warps 2..17 are the epilogue (warp w reads TMEM lanes 32*(w%4).. and the columns
// 32*cg .. 32*cg+31 and 128+32*cg .. 128+32*cg+31 of the tile, cg = (w-2)/4).
// Every mbarrier wait is bounded, as in emit_tc.cuh.
#pragma once
#include "chain_tc.cuh"      // softplus_fast
#include "emit_tc.cuh"
#include "kernels_literal.cuh"

namespace cutoff {
namespace tc {

constexpr int kGemmBN = 256;              // output columns per tile

struct GemmTcArgs {
    const float* bias;      // [Nout]
    float* out;             // [M][ld_out]: relu(A B^T + bias), rounded to tf32 (it is the next product's operand)
    DevState* st;
    int M, Nout, K, ld_out;
};

__device__ __forceinline__ void gemm_epilogue_tile(const GemmTcArgs& a, uint32_t tmem_base, uint32_t acc, int q, int cg,
                                                   int lane, int m0, int w0, uint32_t bar_acc_empty, const float* bias_s) {
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccCols + cg * 32;
    const int row = m0 + q * 32 + lane;
    const bool row_ok = row < a.M;
    const bool wide_store = (a.ld_out & 7) == 0;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        uint32_t bits[2][16];
        tmem_ld16(taddr + 16 * half, bits[0]);
        tmem_ld16(taddr + 128 + 16 * half, bits[1]);
        tmem_ld_wait();
        if (half == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);    // accumulator is free again
        }
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            const int jw = w0 + 128 * part + cg * 32 + 16 * half;
            if (!row_ok || jw >= a.Nout) continue;
            float* dst = a.out + static_cast<size_t>(row) * a.ld_out + jw;
            float out[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 bv = *reinterpret_cast<const float4*>(bias_s + 32 * part + 16 * half + 4 * i);
                const float b[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    out[4 * i + c] = round_tf32(fmaxf(__uint_as_float(bits[part][4 * i + c]) + b[c], 0.0f));
            }
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                if (wide_store && jw + 8 * p + 7 < a.Nout) {
                    store8(dst + 8 * p, out + 8 * p);
                    continue;
                }
#pragma unroll
                for (int i = 2 * p; i < 2 * p + 2; ++i) {
                    const int ji = jw + 4 * i;
                    if (ji + 3 < a.Nout) {
                        *reinterpret_cast<float4*>(dst + 4 * i) =
                            make_float4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
                    } else {
                        for (int c = 0; c < 4 && ji + c < a.Nout; ++c) dst[4 * i + c] = out[4 * i + c];
                    }
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1) k_gemm_relu_tc(const __grid_constant__ CUtensorMap map_a,
                                                          const __grid_constant__ CUtensorMap map_b, GemmTcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                     // operand ring, 1024-byte aligned
    const uint32_t bars = tiles + kStages * kStageBytes;
    // barrier layout (8 bytes each): full[4], empty[4], acc_full[2], acc_empty[2], drain; then tmem base, abort flag
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kStages;
    const uint32_t bar_acc_full = bar_empty + 8 * kStages, bar_acc_empty = bar_acc_full + 16;
    const uint32_t bar_drain = bar_acc_empty + 16;
    uint8_t* gen = smem_raw + (tiles - raw) + kStages * kStageBytes;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 8 * (2 * kStages + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 8 * (2 * kStages + 5) + 8);
    float* bias_all = reinterpret_cast<float*>(gen + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles_w = ceil_div(a.Nout, kGemmBN);
    const int n_tiles_m = ceil_div(a.M, kBM);
    const int total_tiles = n_tiles_w * n_tiles_m;
    const int k_blocks = ceil_div(a.K, kBK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, kEpiWarps);
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------------------------------------------------
        uint32_t stage = 0, phase = 0;
        uint32_t armed_mask = 0, parity_mask = 0;      // per stage: armed at least once / parity of its last phase
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const int m0 = (t / n_tiles_w) * kBM, w0 = (t % n_tiles_w) * kGemmBN;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.st);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t full = bar_full + 8 * stage;
                    const uint32_t dst = tiles + stage * kStageBytes;
                    mbar_arrive_expect_tx(full, kStageBytes);
                    tma_load_2d(dst, &map_a, kb * kBK, m0, full);
                    tma_load_2d(dst + kABytes, &map_b, kb * kBK, w0, full);
                    tma_load_2d(dst + kABytes + kBBytes / 2, &map_b, kb * kBK, w0 + 128, full);
                }
                __syncwarp();
                armed_mask |= 1u << stage;
                parity_mask = (parity_mask & ~(1u << stage)) | (phase << stage);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            // wind down: let every copy that was issued land before the CTA leaves (bounded)
            for (uint32_t s = 0; s < static_cast<uint32_t>(kStages); ++s) {
                if (!((armed_mask >> s) & 1u)) continue;
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_full + 8 * s, (parity_mask >> s) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer -------------------------------------------------------------
        uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            ok = mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag, a.st);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * kAccCols;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.st);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t a_addr = tiles + stage * kStageBytes;
                    const uint64_t a_desc = make_smem_desc(a_addr);
                    const uint64_t b_desc = make_smem_desc(a_addr + kABytes);
#pragma unroll
                    for (int k = 0; k < kBK / 8; ++k)          // 8 tf32 = 32 bytes per instruction
                        umma_tf32(d_tmem, a_desc + 2 * k, b_desc + 2 * k, kInstrDesc, (kb | k) != 0);
                    umma_commit(bar_empty + 8 * stage);         // frees the stage when these MMAs are done
                    if (kb == k_blocks - 1) umma_commit(bar_acc_full + 8 * acc);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok) {
            // make sure no MMA is still running before TMEM is released (bounded)
            if (lane == 0) umma_commit(bar_drain);
            __syncwarp();
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0u) && global_ns() - t0 < kWaitLimitNs) {}
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ---------------------------------------------------------------
        const int q = warp & 3, cg = (warp - 2) >> 2;
        float* bias_s = bias_all + (warp - 2) * 64;
        int w_staged = -1;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const int m0 = (t / n_tiles_w) * kBM, w0 = (t % n_tiles_w) * kGemmBN;
            if (w0 != w_staged) {                       // biases of this warp's 2 x 32 columns, read once per column tile
                const int j = w0 + cg * 32 + lane;
                const float b_lo = j < a.Nout ? __ldg(a.bias + j) : 0.f;
                const float b_hi = j + 128 < a.Nout ? __ldg(a.bias + j + 128) : 0.f;
                __syncwarp();                           // the previous tile's readers are done
                bias_s[lane] = b_lo;
                bias_s[32 + lane] = b_hi;
                __syncwarp();
                w_staged = w0;
            }
            ok = mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, a.st);
            if (!ok) break;
            tc_fence_after();
            gemm_epilogue_tile(a, tmem_base, acc, q, cg, lane, m0, w0, bar_acc_empty, bias_s);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// x = I + softplus(r Wj2^T + bj2) * eps  with  I = u Wi2^T + bi2, both products in one accumulator, so that I
// never goes through memory (an earlier version wrote I out and read it back element by element in the epilogue of
// the scale product: that alone cost 0.14 ms at N=1024, S=65536).  Tiles of 128 samples x 128 workers; the
// accumulator holds I in columns 0..127 and the scale pre-activation in columns 128..255, from two MMAs per
// K step with different operands: (u, Wi2 rows) and (r, Wj2 rows).  A stage of the 3-stage ring is
// [u tile | r tile | Wi2 tile | Wj2 tile], 16 KB each.  Warp roles, accumulator double-buffering and the bounded
// waits are those of k_emit_tc; the epilogue is its epilogue with softplus in place of exp(logvar / 2).
// ---------------------------------------------------------------------------------------------
constexpr int kDualStages = 3;
constexpr int kDualStageBytes = 4 * kABytes;             // 64 KB
constexpr size_t kDualSmemBytes = kDualStages * kDualStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kBiasBytes;
constexpr uint32_t kDualInstrDesc = (1u << 4) | (2u << 7) | (2u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);   // N = 128

struct EmitDualArgs {
    const float* bias_mean;     // bi2 [N]
    const float* bias_scale;    // bj2 [N]
    float* x;                   // [count][ldx]
    DevState* st;
    NoiseKey key;
    uint32_t sample_base;
    int count, N, H, ldx;
};

__device__ __forceinline__ void dual_epilogue_tile(const EmitDualArgs& a, uint32_t tmem_base, uint32_t acc, int q, int cg,
                                                   int lane, int m0, int w0, uint32_t step, uint32_t bar_acc_empty,
                                                   const float* bias_s) {
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccCols + cg * 32;
    const int row = m0 + q * 32 + lane;
    const bool row_ok = row < a.count;
    const uint32_t sample = a.sample_base + static_cast<uint32_t>(row);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        uint32_t mean_bits[16], scale_bits[16];
        tmem_ld16(taddr + 16 * half, mean_bits);
        tmem_ld16(taddr + kBW + 16 * half, scale_bits);
        tmem_ld_wait();
        if (half == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);    // accumulator is free again
        }
        const int jw = w0 + cg * 32 + 16 * half;
        if (row_ok && jw < a.N) {
            float* dst = a.x + static_cast<size_t>(row) * a.ldx + jw;
            float out[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = jw + 4 * i;
                if (j >= a.N) continue;
                float eps[4];
                normal4_fast(static_cast<uint32_t>(j >> 2), sample, kStreamEmission, step, a.key.seed_lo,
                             a.key.seed_hi, eps);
                const float4 bm = *reinterpret_cast<const float4*>(bias_s + 16 * half + 4 * i);
                const float4 bs = *reinterpret_cast<const float4*>(bias_s + 32 + 16 * half + 4 * i);
                const float bmv[4] = {bm.x, bm.y, bm.z, bm.w}, bsv[4] = {bs.x, bs.y, bs.z, bs.w};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    out[4 * i + c] = fmaf(softplus_fast(__uint_as_float(scale_bits[4 * i + c]) + bsv[c]), eps[c],
                                          __uint_as_float(mean_bits[4 * i + c]) + bmv[c]);
            }
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                if (jw + 8 * p + 7 < a.N) {
                    store8(dst + 8 * p, out + 8 * p);
                    continue;
                }
#pragma unroll
                for (int i = 2 * p; i < 2 * p + 2; ++i) {
                    const int ji = jw + 4 * i;
                    if (ji + 3 < a.N) {
                        *reinterpret_cast<float4*>(dst + 4 * i) =
                            make_float4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
                    } else {
                        for (int c = 0; c < 4 && ji + c < a.N; ++c) dst[4 * i + c] = out[4 * i + c];
                    }
                }
            }
        }
    }
}

// map_u, map_r: [rows][H] activations; map_wi2, map_wj2: [N][H] weights; boxes of 128 rows x 32 columns.
__global__ void __launch_bounds__(kThreads, 1) k_emit_dual_tc(const __grid_constant__ CUtensorMap map_u,
                                                               const __grid_constant__ CUtensorMap map_r,
                                                               const __grid_constant__ CUtensorMap map_wi2,
                                                               const __grid_constant__ CUtensorMap map_wj2, EmitDualArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                     // operand ring, 1024-byte aligned
    const uint32_t bars = tiles + kDualStages * kDualStageBytes;
    // barrier layout (8 bytes each): full[3], empty[3], acc_full[2], acc_empty[2], drain; then tmem base, abort flag
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kDualStages;
    const uint32_t bar_acc_full = bar_empty + 8 * kDualStages, bar_acc_empty = bar_acc_full + 16;
    const uint32_t bar_drain = bar_acc_empty + 16;
    uint8_t* gen = smem_raw + (tiles - raw) + kDualStages * kDualStageBytes;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 8 * (2 * kDualStages + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 8 * (2 * kDualStages + 5) + 8);
    float* bias_all = reinterpret_cast<float*>(gen + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles_w = ceil_div(a.N, kBW);
    const int n_tiles_m = ceil_div(a.count, kBM);
    const int total_tiles = n_tiles_w * n_tiles_m;
    const int k_blocks = ceil_div(a.H, kBK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDualStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, kEpiWarps);
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------------------------------------------------
        uint32_t stage = 0, phase = 0;
        uint32_t armed_mask = 0, parity_mask = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const int m0 = (t / n_tiles_w) * kBM, w0 = (t % n_tiles_w) * kBW;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.st);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t full = bar_full + 8 * stage;
                    const uint32_t dst = tiles + stage * kDualStageBytes;
                    mbar_arrive_expect_tx(full, kDualStageBytes);
                    tma_load_2d(dst, &map_u, kb * kBK, m0, full);
                    tma_load_2d(dst + kABytes, &map_r, kb * kBK, m0, full);
                    tma_load_2d(dst + 2 * kABytes, &map_wi2, kb * kBK, w0, full);
                    tma_load_2d(dst + 3 * kABytes, &map_wj2, kb * kBK, w0, full);
                }
                __syncwarp();
                armed_mask |= 1u << stage;
                parity_mask = (parity_mask & ~(1u << stage)) | (phase << stage);
                if (++stage == kDualStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            for (uint32_t s = 0; s < static_cast<uint32_t>(kDualStages); ++s) {
                if (!((armed_mask >> s) & 1u)) continue;
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_full + 8 * s, (parity_mask >> s) & 1u) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer -------------------------------------------------------------
        uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            ok = mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag, a.st);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * kAccCols;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.st);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t s_addr = tiles + stage * kDualStageBytes;
                    const uint64_t u_desc = make_smem_desc(s_addr), r_desc = make_smem_desc(s_addr + kABytes);
                    const uint64_t wi_desc = make_smem_desc(s_addr + 2 * kABytes), wj_desc = make_smem_desc(s_addr + 3 * kABytes);
#pragma unroll
                    for (int k = 0; k < kBK / 8; ++k) {
                        umma_tf32(d_tmem, u_desc + 2 * k, wi_desc + 2 * k, kDualInstrDesc, (kb | k) != 0);          // I
                        umma_tf32(d_tmem + kBW, r_desc + 2 * k, wj_desc + 2 * k, kDualInstrDesc, (kb | k) != 0);    // scale
                    }
                    umma_commit(bar_empty + 8 * stage);
                    if (kb == k_blocks - 1) umma_commit(bar_acc_full + 8 * acc);
                }
                __syncwarp();
                if (++stage == kDualStages) { stage = 0; phase ^= 1u; }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok) {
            if (lane == 0) umma_commit(bar_drain);
            __syncwarp();
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0u) && global_ns() - t0 < kWaitLimitNs) {}
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ---------------------------------------------------------------
        const int q = warp & 3, cg = (warp - 2) >> 2;
        const uint32_t step = a.st->step;
        float* bias_s = bias_all + (warp - 2) * 64;
        int w_staged = -1;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const int m0 = (t / n_tiles_w) * kBM, w0 = (t % n_tiles_w) * kBW;
            if (w0 != w_staged) {                       // biases of this warp's 32 workers, read once per worker tile
                const int j = w0 + cg * 32 + lane;
                const float bm = j < a.N ? __ldg(a.bias_mean + j) : 0.f;
                const float bs = j < a.N ? __ldg(a.bias_scale + j) : 0.f;
                __syncwarp();
                bias_s[lane] = bm;
                bias_s[32 + lane] = bs;
                __syncwarp();
                w_staged = w0;
            }
            ok = mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, a.st);
            if (!ok) break;
            tc_fence_after();
            dual_epilogue_tile(a, tmem_base, acc, q, cg, lane, m0, w0, step, bar_acc_empty, bias_s);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace tc
}  // namespace cutoff
