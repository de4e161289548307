// The emission output layer of emit_tc.cuh on pairs of SMs: one UMMA of shape M=256, N=256, K=8
// (tcgen05.mma.cta_group::2) spans a cluster of two CTAs.  Opt-in (option "pair_emission").
//
// The one-SM kernel streams 48 KB of operands from L2 into shared memory per K block for every 128 x 128 output
// tile (16 KB of hidden vectors, 32 KB of weights).  Here the two CTAs of a cluster take the same 128 workers for
// two neighbouring blocks of 128 samples.  Each CTA loads its own 128 hidden vectors (A: the instruction reads
// rows 0..127 from the leader's shared memory and rows 128..255 from its peer's) and only HALF of the weight tile
// (B: the 128 mean rows in the leader, the 128 log-variance rows in the peer): 32 KB per K block instead of 48.
// Each CTA's tensor memory receives the accumulator of its own 128 samples, 128 lanes x 256 columns (means, then
// log-variances) -- the layout of the one-SM kernel, whose epilogue is used as it is.
//
// Roles per CTA: warp 0 loads its operands by TMA (plain per-CTA loads, not multicast; the loads of both CTAs are
// counted on the leader's "stage full" barrier); warp 1 of the leader (cluster rank 0) issues the MMAs for the
// pair, warp 1 of the peer tells the leader when the peer's epilogue has emptied an accumulator; warps 2..17 are the
// epilogue.  The leader's tcgen05.commit arrives on the "stage free" and "accumulator ready" barriers of BOTH CTAs
// (multicast of the arrive, not of data).  A stage holds two K blocks (64 KB), three stages: with one K block per
// stage the hand-shake across the pair, not the operand stream, set the pace.  Tensor memory is allocated by each
// CTA for itself (all 512 columns, so both start at column 0).  Every wait is bounded as in emit_tc.cuh.
//
// Measured at N=1024, S=65536: 0.177 ms against 0.148 ms of the one-SM kernel (0.235 ms with one K block per
// stage); tensor pipe 27 % active.  The operand stream shrinks as planned (L2 throughput 41 % against 59 %), but
// a K=8 tf32 instruction is short and every stage now costs a round trip between two SMs.  Hence opt-in.
#pragma once
#include "emit_tc.cuh"

namespace cutoff {
namespace tc {

constexpr int kStages2 = 3;
constexpr int kStageK2 = 2;                               // K blocks (of 32) per stage
constexpr int kStage2Bytes = kStageK2 * (kABytes + kBBytes / 2);   // 64 KB: per K block 128 hidden vectors x 32 and this CTA's 128 weight rows x 32
constexpr size_t kSmem2Bytes = kStages2 * kStage2Bytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kBiasBytes;
// instruction descriptor: D = f32, A = B = tf32, both K-major, N = 256, M = 256 (two CTAs x 128)
constexpr uint32_t kInstrDesc2 = (1u << 4) | (2u << 7) | (2u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
// arrive with an expected byte count on a barrier given by its shared::cluster address
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// plain (per-CTA, not multicast) tiled load whose completion is counted on a barrier that may live in the peer CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void umma_tf32_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrive (once the pair's MMAs issued so far are done) on the barrier at this offset in the CTAs of `cta_mask`
// (3: both CTAs of the pair, 1: the leader only)
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask = 3) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(cta_mask) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_emit_tc2(const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_w4, EmitArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                     // operand ring, 1024-byte aligned
    const uint32_t bars = tiles + kStages2 * kStage2Bytes;
    // barrier layout (8 bytes each): full[6], peer_full[6], empty[6], acc_full[2], acc_empty[2], drain;
    // then tmem base, abort flag
    const uint32_t bar_full = bars, bar_peer_full = bars + 8 * kStages2, bar_empty = bars + 16 * kStages2;
    const uint32_t bar_acc_full = bars + 24 * kStages2, bar_acc_empty = bar_acc_full + 16;
    const uint32_t bar_drain = bar_acc_empty + 16;
    uint8_t* gen = smem_raw + (tiles - raw) + kStages2 * kStage2Bytes;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 8 * (3 * kStages2 + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 8 * (3 * kStages2 + 5) + 8);
    float* bias_all = reinterpret_cast<float*>(gen + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                          // 0: leader (issues the MMAs), 1: peer
    const int cluster_id = static_cast<int>(blockIdx.x >> 1), n_clusters = static_cast<int>(gridDim.x >> 1);
    const int n_tiles_w = ceil_div(a.N, kBW);
    const int total_tiles = n_tiles_w * ceil_div(a.count, 2 * kBM);   // a tile: 256 samples (128 per CTA) x 128 workers
    const int k_blocks = ceil_div(a.H, kBK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages2; ++s) {
            mbar_init(bar_full + 8 * s, 2);                           // the producers of both CTAs (the leader's copy is the one used)
            mbar_init(bar_peer_full + 8 * s, 1);                      // [0], [1]: the peer's epilogue has emptied accumulator 0 / 1
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, kEpiWarps);              // this CTA's epilogue warps
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
    cluster_sync_all();                   // the peer's barriers and tensor memory exist before anything reaches across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs): own hidden vectors, own half of the weight tile -------------
        uint32_t stage = 0, phase = 0;
        const uint32_t leader_full = map_to_cta(bar_full, 0u);        // every load of the pair is counted on the leader's barriers
        bool ok = true;
        for (int t = cluster_id; ok && t < total_tiles; t += n_clusters) {
            const int m0 = (t / n_tiles_w) * 2 * kBM + static_cast<int>(rank) * kBM, w0 = (t % n_tiles_w) * kBW;
            const int b_row = rank == 0 ? w0 : a.N + w0;              // mean rows in the leader, log-variance rows in the peer
            for (int kb = 0; kb < k_blocks; kb += kStageK2) {
                ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, a.st);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t full = leader_full + 8 * stage;
                    const uint32_t dst = tiles + stage * kStage2Bytes;
                    mbar_arrive_expect_tx_cluster(full, kStage2Bytes);     // blocks beyond H read as zeros and count all the same
#pragma unroll
                    for (int j = 0; j < kStageK2; ++j) {
                        tma_load_2d_pair(dst + j * (kABytes + kBBytes / 2), &map_v, (kb + j) * kBK, m0, full);
                        tma_load_2d_pair(dst + j * (kABytes + kBBytes / 2) + kABytes, &map_w4, (kb + j) * kBK, b_row, full);
                    }
                }
                __syncwarp();
                if (++stage == kStages2) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            // wind down: the copies still in flight land within microseconds; give them a bounded while
            const unsigned long long t0 = global_ns();
            while (global_ns() - t0 < 200000ull) {}
        }
    } else if (warp == 1 && rank != 0) {
        // ---------------- peer: tell the leader when this CTA's epilogue has emptied an accumulator ---------------
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        const uint32_t leader_peer_free = map_to_cta(bar_peer_full, 0u);
        for (int t = cluster_id; ok && t < total_tiles; t += n_clusters) {
            ok = mbar_wait(bar_acc_empty + 8 * acc, acc_phase, abort_flag, a.st);
            if (!ok) break;
            if (lane == 0) mbar_arrive_cluster(leader_peer_free + 8 * acc);
            __syncwarp();
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else if (warp == 1) {
        // ---------------- leader: MMA issuer for the pair ---------------------------------------------------------
        uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = cluster_id; ok && t < total_tiles; t += n_clusters) {
            ok = mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag, a.st) &&
                 mbar_wait(bar_peer_full + 8 * acc, acc_phase ^ 1u, abort_flag, a.st);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * kAccCols;
            for (int kb = 0; kb < k_blocks; kb += kStageK2) {
                ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, a.st);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < kStageK2; ++j) {
                        const uint32_t a_addr = tiles + stage * kStage2Bytes + j * (kABytes + kBBytes / 2);
                        const uint64_t a_desc = make_smem_desc(a_addr);
                        const uint64_t b_desc = make_smem_desc(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kBK / 8; ++k)
                            umma_tf32_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, kInstrDesc2, (kb | j | k) != 0);
                    }
                    umma_commit_pair(bar_empty + 8 * stage);          // frees the stage in both CTAs
                    if (kb + kStageK2 >= k_blocks) umma_commit_pair(bar_acc_full + 8 * acc);
                }
                __syncwarp();
                if (++stage == kStages2) { stage = 0; phase ^= 1u; }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok) {
            if (lane == 0) umma_commit_pair(bar_drain, 1);
            __syncwarp();
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0u) && global_ns() - t0 < kWaitLimitNs) {}
        }
        __syncwarp();
    } else {
        // ---------------- epilogue (both CTAs): this CTA's 128 samples ---------------------------------------------
        const int q = warp & 3, cg = (warp - 2) >> 2;
        const uint32_t step = a.st->step;
        float* bias_s = bias_all + (warp - 2) * 64;
        int w_staged = -1;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = cluster_id; ok && t < total_tiles; t += n_clusters) {
            const int m0 = (t / n_tiles_w) * 2 * kBM + static_cast<int>(rank) * kBM, w0 = (t % n_tiles_w) * kBW;
            if (w0 != w_staged) {
                const int j = w0 + cg * 32 + lane;
                const float bm = j < a.N ? __ldg(a.b4 + j) : 0.f;
                const float bl = j < a.N ? __ldg(a.b4 + a.N + j) : 0.f;
                __syncwarp();
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
    cluster_sync_all();                   // neither CTA frees its tensor memory or leaves while the other may still reach it
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace tc
}  // namespace cutoff
