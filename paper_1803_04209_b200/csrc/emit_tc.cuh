// Emission output layer on the 5th-generation tensor cores (tcgen05), with the noise drawn in
// the epilogue:   [mean | logvar] = W4 v + b4,   x_j = mean_j + exp(logvar_j / 2) * eps_j.
//
// One persistent CTA per SM walks over output tiles of 128 samples x 128 workers.  A tile is one
// accumulator of 128 TMEM lanes (samples) x 256 fp32 columns (128 means, then 128 log-variances),
// filled by UMMA instructions of shape M=128, N=256, K=8 in kind::tf32.  Operands arrive by TMA
// (plain, per-CTA loads) into a 4-stage ring of 128-byte-swizzled K-major tiles; the accumulator
// is double-buffered (2 x 256 of the 512 TMEM columns) so that the epilogue of one tile runs
// while the next tile is multiplied.
//
// Warp roles: warp 0 issues TMA loads, warp 1 owns TMEM and issues the MMAs, warps 2..17 are the
// epilogue (warp w reads TMEM lanes 32*(w%4).., the 32 workers of column group (w-2)/4).
//
// Every wait on an mbarrier is bounded: after about two seconds it records kErrTimeout in the
// device state, raises a CTA-wide abort flag and the kernel winds down (outstanding copies are
// waited for, again bounded, and TMEM is released).
#pragma once
#include <cuda.h>

#include "async.cuh"
#include "common.cuh"
#include "rng.cuh"

namespace cutoff {
namespace tc {

using namespace cutoff::async;

constexpr int kBM = 128;                 // samples per tile (TMEM lanes)
constexpr int kBW = 128;                 // workers per tile
constexpr int kBK = 32;                  // tf32 elements per 128-byte swizzle row
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK * 4;           // 16 KB
constexpr int kBBytes = 2 * kBW * kBK * 4;       // 32 KB: mean rows, then log-variance rows
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kEpiWarps = 16;
constexpr int kThreads = (2 + kEpiWarps) * 32;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 2 * kBW;                // 256 columns per accumulator
constexpr int kBiasBytes = kEpiWarps * 64 * 4;   // per epilogue warp: 32 mean + 32 log-variance biases of its columns
constexpr size_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kBiasBytes;

// instruction descriptor: D = f32, A = B = tf32, both K-major, N = 256, M = 128
constexpr uint32_t kInstrDesc = (1u << 4) | (2u << 7) | (2u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// K-major operand tile, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);      // start address
    d |= static_cast<uint64_t>(1) << 16;                           // leading byte offset (unused here)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                   // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;                           // descriptor version
    d |= static_cast<uint64_t>(2) << 61;                           // SWIZZLE_128B
    return d;
}

__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// One 256-bit store: eight consecutive floats at a 32-byte aligned address.
__device__ __forceinline__ void store8(float* p, const float* v) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}

struct EmitArgs {
    const float* b4;        // [2N]
    float* x;               // [count][ldx]
    DevState* st;
    NoiseKey key;
    uint32_t sample_base;
    int count, N, H, ldx;
};

// Epilogue of one 128 x 128 output tile for one warp: read its 32 lanes x 32 (+32) accumulator columns, hand the
// accumulator back, add the biases, draw the noise and store x = mean + exp(logvar / 2) * eps.
// bias_s: this warp's 32 mean biases, then its 32 log-variance biases, in shared memory (zero beyond worker N).
__device__ __forceinline__ void emit_epilogue_tile(const EmitArgs& a, uint32_t tmem_base, uint32_t acc, int q, int cg,
                                                   int lane, int m0, int w0, uint32_t step, uint32_t bar_acc_empty,
                                                   const float* bias_s) {
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccCols + cg * 32;
    const int row = m0 + q * 32 + lane;
    const bool row_ok = row < a.count;
    const uint32_t sample = a.sample_base + static_cast<uint32_t>(row);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        uint32_t mean_bits[16], logvar_bits[16];
        tmem_ld16(taddr + 16 * half, mean_bits);
        tmem_ld16(taddr + kBW + 16 * half, logvar_bits);
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
                const float4 bl = *reinterpret_cast<const float4*>(bias_s + 32 + 16 * half + 4 * i);
                const float bmv[4] = {bm.x, bm.y, bm.z, bm.w}, blv[4] = {bl.x, bl.y, bl.z, bl.w};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    out[4 * i + c] = fmaf(exp_half_fast(__uint_as_float(logvar_bits[4 * i + c]) + blv[c]), eps[c],
                                          __uint_as_float(mean_bits[4 * i + c]) + bmv[c]);
            }
            // a thread owns 16 consecutive workers of its sample: two 32-byte stores (whole sectors; the row pitch
            // is a multiple of 8 floats), 16-byte or scalar stores on the ragged edge
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

__global__ void __launch_bounds__(kThreads, 1) k_emit_tc(const __grid_constant__ CUtensorMap map_v,
                                                          const __grid_constant__ CUtensorMap map_w4, EmitArgs a) {
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
    const int n_tiles_w = ceil_div(a.N, kBW);
    const int n_tiles_m = ceil_div(a.count, kBM);
    const int total_tiles = n_tiles_w * n_tiles_m;
    const int k_blocks = ceil_div(a.H, kBK);

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
    dependency_wait();            // the hidden vectors and the device state are an earlier kernel's
    launch_dependents();

    if (warp == 0) {
        // ---------------- TMA producer ----------------------------------------------------------
        uint32_t stage = 0, phase = 0;
        uint32_t armed_mask = 0, parity_mask = 0;      // per stage: armed at least once / parity of its last phase
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const int m0 = (t / n_tiles_w) * kBM, w0 = (t % n_tiles_w) * kBW;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.st);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t full = bar_full + 8 * stage;
                    const uint32_t dst = tiles + stage * kStageBytes;
                    mbar_arrive_expect_tx(full, kStageBytes);
                    tma_load_2d(dst, &map_v, kb * kBK, m0, full);
                    tma_load_2d(dst + kABytes, &map_w4, kb * kBK, w0, full);
                    tma_load_2d(dst + kABytes + kBBytes / 2, &map_w4, kb * kBK, a.N + w0, full);
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
        const uint32_t step = a.st->step;
        float* bias_s = bias_all + (warp - 2) * 64;
        int w_staged = -1;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const int m0 = (t / n_tiles_w) * kBM, w0 = (t % n_tiles_w) * kBW;
            if (w0 != w_staged) {                       // biases of this warp's 32 workers, read once per worker tile
                const int j = w0 + cg * 32 + lane;
                const float bm = j < a.N ? __ldg(a.b4 + j) : 0.f;
                const float bl = j < a.N ? __ldg(a.b4 + a.N + j) : 0.f;
                __syncwarp();                           // the previous tile's readers are done
                bias_s[lane] = bm;
                bias_s[32 + lane] = bl;
                __syncwarp();
                w_staged = w0;
            }
            ok = mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, a.st);
            if (!ok) break;
            tc_fence_after();
            emit_epilogue_tile(a, tmem_base, acc, q, cg, lane, m0, w0, step, bar_acc_empty, bias_s);
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
