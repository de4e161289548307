// C ABI and host orchestration of the cutoff library (see include/cutoff.h).
#include "../../include/cutoff.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "kernels_model.cuh"
#include "kernels_sort.cuh"
#include "emit_tc.cuh"
#include "emit_tc2.cuh"
#include "chain_tc.cuh"
#include "chain_tc32.cuh"
#include "kernels_literal.cuh"
#include "gemm_tc.cuh"
#include "pipe_rates.cuh"
#include "kernels_eval.cuh"
#include "fit_api.cuh"

using namespace cutoff;

namespace {

constexpr uint32_t kBlobMagic = 0x31465443u;   // "CTF1"
constexpr int kNumStages = 5;
constexpr int kMaxChunks = 64;        // passes per decision (also the number of timing event sets)
constexpr int kPartialRows = 2048;    // partial-sum rows shared by all passes of a decision
const char* const kStageNames[kNumStages] = {"encoder", "chain", "emission", "sort", "decide"};

struct TensorSpec { const char* name; size_t rows, cols; };

}  // namespace

struct cutoff_ctx {
    cutoff_config cfg{};
    int N = 0, D = 0, H = 0, W = 0, S = 0;
    int ldx = 0;            // leading dimension of the sample matrix (N rounded up to 8: rows start on 32 bytes)
    int P = 0;              // sort width: N rounded up to a power of two, at least 32
    int sm_count = 0;
    int chunk_rows = 0;     // samples per pass through chain -> emission -> sort
    int alloc_rows = 0;     // rows the pass buffers were allocated for
    int n_chunks = 0;
    int sort_grid = 0;      // CTAs of the sort kernel per chunk (= partial rows per chunk)
    cudaStream_t stream = nullptr;
    bool owns_stream = false;       // the context created `stream` itself (graph mode with a NULL stream)

    float* d_blob = nullptr;        // tensors as loaded
    float* d_WT = nullptr;          // transposed copies WzT, W1T, W3T: 3 x [D][H]
    float* d_WhR = nullptr;         // recurrence matrices regrouped per thread for k_enc_rnn_resident: 2 x H x H
    ModelDev m{};
    bool weights_loaded = false;

    float* d_ring = nullptr;        // [W][N]
    float* d_stage = nullptr;       // [N] landing buffer for host pushes
    uint8_t* d_mask = nullptr;      // [N] censoring mask of the push in progress
    uint8_t* h_mask = nullptr;      // pinned [N]
    bool draws_valid = false;       // d_x holds every predictive draw of the last decision (needed for imputation)
    DevState* d_state = nullptr;
    float* d_proj = nullptr;        // [2][W slots][H] raw input projections of the ring's vectors, kept up to date by every push
    bool proj_stale = true;         // the ring or the weights were replaced: recompute every slot before the next decision
    float* d_hlr = nullptr;         // [2][W][H]
    float* d_v = nullptr;           // [chunk_rows][H]
    float* d_x = nullptr;           // [chunk_rows][ldx]
    float* d_partial = nullptr;     // [n_chunks * sort_grid][N]; a second block of kPartialRows rows holds sums of squares
    float* d_std = nullptr;         // [N] spread of each order statistic (when asked for)
    bool want_std = false;
    bool have_std = false;
    double* d_sums = nullptr;       // [N]
    float* d_E = nullptr;           // [N]
    float* d_omega = nullptr;       // [N]

    CUtensorMap map_v{};            // TMA view of d_v   [alloc_rows][H]
    CUtensorMap map_w4{};           // TMA view of W4    [2N][H]

    bool literal = false;           // the networks as Section 3.1.3 prints them (CUTOFF_FLAG_LITERAL)
    LiteralDev lit{};
    float* d_I = nullptr;           // [alloc_rows][ldx]  emission mean I (padding columns stay zero); fp32 path only
    float* d_r = nullptr;           // [alloc_rows][H]    hidden layer of the emission scale
    float* d_Wj1p = nullptr;        // [H][ldx]           Wj1 with rows padded with zeros to ldx; fp32 path only
    float* d_M = nullptr;           // [H][H] then [H]    M = Wj1 Wi2 and b' = Wj1 bi2 + bj1 (tensor-core path: Wj1 I + bj1 = M u + b')
    CUtensorMap map_r{};            // TMA view of d_r [alloc_rows][H]
    CUtensorMap map_wi2{}, map_M{}, map_wj2{};
    bool use_tc = false;            // emission output layer on tensor cores
    int pair_clusters = 0;          // clusters of two CTAs of the two-SM emission kernel that fit the GPU at once
    bool pair_emission = false;     // option "pair_emission": run the output layer on pairs of SMs (slower as measured; off)
    bool chain_tc = false;          // per-sample chain on tensor cores as well (D = 16, H in {64, 128, 192, 256})
    bool chain_tc32 = false;        // the same for D = 32, H <= 512 (weights staged phase by phase)
    bool chain_tcl = false;         // the literal variant's chain on tensor cores (D = 16, H in {64, 128, 192, 256})
    bool chain_tcl32 = false;       // the same for D = 32, H <= 512 (weights staged phase by phase)
    float* d_chain_image = nullptr; // swizzled tf32 operand tiles of the chain

    float* h_stage = nullptr;       // pinned [N]
    DevState* h_state = nullptr;    // pinned

    uint32_t pushes = 0;            // host mirror of DevState::push_count
    bool pending = false;           // a decision is enqueued and not yet fetched
    bool pending_warmup = false;
    bool have_result = false;
    bool partial_pending = false;   // the sums of a decision are enqueued, its argmax (and counter step) still to come

    bool timing = false;
    cudaEvent_t ev[kNumStages + 1][kMaxChunks]{};   // per chunk, stage boundaries
    bool ev_created = false;
    float stage_ms[kNumStages]{};
    int timed_chunks = 0;

    cudaGraph_t graph = nullptr;            // captured push + decision (CUTOFF_FLAG_GRAPH)
    cudaGraphExec_t graph_exec = nullptr;
    cudaGraph_t graph_dev = nullptr;        // the same without the host-to-device copy (cutoff_step_device)
    cudaGraphExec_t graph_dev_exec = nullptr;
    int graph_kernels = 0;                  // kernels one replay launches
    bool decided_once = false;              // a decision has run outside capture (function attributes are set)

    int64_t launches = 0;
    std::string last_error;
};

namespace {

#define CU_CHECK(ctx, call)                                                                          \
    do {                                                                                             \
        cudaError_t err__ = (call);                                                                  \
        if (err__ != cudaSuccess) {                                                                  \
            if (ctx) (ctx)->last_error = std::string(#call) + ": " + cudaGetErrorString(err__);      \
            return err__ == cudaErrorMemoryAllocation ? CUTOFF_ERR_NOMEM : CUTOFF_ERR_CUDA;          \
        }                                                                                            \
    } while (0)

// Makes the context's device current for the duration of an entry point and puts the caller's
// current device back on exit.
struct DeviceGuard {
    int prev = -1;
    bool changed = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int device) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != device) {
            err = cudaSetDevice(device);
            changed = err == cudaSuccess;
        }
    }
    ~DeviceGuard() {
        if (changed && prev >= 0) cudaSetDevice(prev);
    }
    DeviceGuard(const DeviceGuard&) = delete;
    DeviceGuard& operator=(const DeviceGuard&) = delete;
};

std::vector<TensorSpec> tensor_specs(size_t N, size_t D, size_t H) {
    return {
        {"Wxf", H, N}, {"Whf", H, H}, {"bf", 1, H}, {"a0", 1, H},
        {"Wxb", H, N}, {"Whb", H, H}, {"bb", 1, H}, {"b0", 1, H},
        {"Wz", H, D}, {"bz", 1, H}, {"Wmu", D, H}, {"bmu", 1, D}, {"Wsig", D, D}, {"bsig", 1, D}, {"z0", 1, D},
        {"W1", H, D}, {"b1", 1, H}, {"W2", 2 * D, H}, {"b2", 1, 2 * D},
        {"W3", H, D}, {"b3", 1, H}, {"W4", 2 * N, H}, {"b4", 1, 2 * N},
    };
}

// The literal variant: the guide tensors (the first 15) are the same, then the gated transition and the
// emission networks I and J.
std::vector<TensorSpec> tensor_specs_literal(size_t N, size_t D, size_t H) {
    std::vector<TensorSpec> v = tensor_specs(N, D, H);
    v.resize(15);
    const TensorSpec rest[] = {
        {"Wg1", H, D}, {"bg1", 1, H}, {"Wg2", D, H}, {"bg2", 1, D},
        {"Wh1", H, D}, {"bh1", 1, H}, {"Wh2", D, H}, {"bh2", 1, D},
        {"Wl", D, D}, {"bl", 1, D}, {"Ws", D, D}, {"bs", 1, D},
        {"Wi1", H, D}, {"bi1", 1, H}, {"Wi2", N, H}, {"bi2", 1, N},
        {"Wj1", H, N}, {"bj1", 1, H}, {"Wj2", N, H}, {"bj2", 1, N},
    };
    v.insert(v.end(), std::begin(rest), std::end(rest));
    return v;
}

// Round to tf32 as the tensor cores will see the value (nearest, ties away from zero), kept as an fp32 bit pattern.
float host_tf32(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    u = (u + 0x1000u) & 0xFFFFE000u;
    std::memcpy(&f, &u, 4);
    return f;
}

// Float index of element (row, col) inside one K-major operand slab of rows x 32 with 128-byte rows whose 16-byte
// chunks are XOR-swizzled with the row index modulo 8 (the layout the tensor cores read from shared memory).
size_t swz(size_t row, size_t col) {
    return (row >> 3) * 256 + (row & 7) * 32 + ((((col >> 2) ^ (row & 7)) << 2) | (col & 3));
}

// A first-layer matrix w [rows][cols] (cols <= 32) into columns col0 .. col0 + cols - 1 of a swizzled tile of
// `rows` rows x 32, rounded to tf32: the B operand of hidden = act(W z + b), K = the latent size.
void put_first_layer(float* tile, const float* w, size_t rows, size_t cols, size_t col0) {
    for (size_t n = 0; n < rows; ++n)
        for (size_t k = 0; k < cols; ++k) tile[swz(n, col0 + k)] = host_tf32(w[n * cols + k]);
}

// A second-layer matrix w [out_rows][H] as H / 32 K blocks of `block_rows` rows x 32 (out_rows <= block_rows; the
// other rows stay as they are), swizzled and rounded to tf32: the B operand of out = W hidden, K = H.
void put_second_layer(float* tiles, const float* w, size_t out_rows, size_t H, size_t block_rows) {
    for (size_t kb = 0; kb < H / 32; ++kb)
        for (size_t o = 0; o < out_rows; ++o)
            for (size_t jj = 0; jj < 32; ++jj) tiles[kb * block_rows * 32 + swz(o, jj)] = host_tf32(w[o * H + kb * 32 + jj]);
}

// Launch `kernel` so that it may begin while the kernel before it in the stream is still running (programmatic
// dependent launch): the kernel itself waits, by dependency_wait(), before it touches that kernel's results.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int next_pow2(int n) {
    int p = 1;
    while (p < n) p <<= 1;
    return p;
}

void free_all(cutoff_ctx* c) {
    cudaFree(c->d_I); cudaFree(c->d_r); cudaFree(c->d_Wj1p); cudaFree(c->d_M);
    cudaFree(c->d_blob); cudaFree(c->d_WT); cudaFree(c->d_WhR); cudaFree(c->d_chain_image); cudaFree(c->d_mask);
    if (c->h_mask) cudaFreeHost(c->h_mask); cudaFree(c->d_ring); cudaFree(c->d_stage);
    cudaFree(c->d_state); cudaFree(c->d_proj); cudaFree(c->d_hlr); cudaFree(c->d_v); cudaFree(c->d_x);
    cudaFree(c->d_partial); cudaFree(c->d_std); cudaFree(c->d_sums); cudaFree(c->d_E); cudaFree(c->d_omega);
    if (c->h_stage) cudaFreeHost(c->h_stage);
    if (c->h_state) cudaFreeHost(c->h_state);
    if (c->owns_stream && c->stream) cudaStreamDestroy(c->stream);
    if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
    if (c->graph) cudaGraphDestroy(c->graph);
    if (c->graph_dev_exec) cudaGraphExecDestroy(c->graph_dev_exec);
    if (c->graph_dev) cudaGraphDestroy(c->graph_dev);
    if (c->ev_created)
        for (auto& row : c->ev)
            for (auto& e : row)
                if (e) cudaEventDestroy(e);
}

// Work split: how many samples go through chain -> emission -> sort at a time, and how many
// CTAs the sort kernel uses per pass.
void plan_chunks(cutoff_ctx* c, int chunk_rows_wanted) {
    int rows = chunk_rows_wanted > 0 ? chunk_rows_wanted : c->S;
    if (rows > c->S) rows = c->S;
    if (rows > c->alloc_rows) rows = c->alloc_rows;
    if (ceil_div(c->S, rows) > kMaxChunks) rows = ceil_div(c->S, kMaxChunks);
    c->chunk_rows = rows;
    c->n_chunks = ceil_div(c->S, rows);
    // CTAs of the sort kernel per pass: enough to fill the GPU, within the partial-sum rows available
    int want, cap;
    if (c->P <= 1024) { want = ceil_div(rows, kSortWarps); cap = c->sm_count * 2; }
    else { want = rows; cap = c->sm_count * 8; }
    if (cap > kPartialRows / c->n_chunks) cap = kPartialRows / c->n_chunks;
    c->sort_grid = want < cap ? want : cap;
}

template <int E, bool SQ>
void launch_sort_warp_sq(cutoff_ctx* c, int count, float* partial) {
    const size_t smem = sort_tma_smem_bytes<E>(c->ldx);
    launch_dependent(k_sort_sum_tma<E, SQ>, dim3(c->sort_grid), dim3(kSortWarps * 32), smem, c->stream,
                     c->d_x, c->ldx, c->N, count, partial, partial + static_cast<size_t>(kPartialRows) * c->N, c->d_state);
}

template <int E>
void launch_sort_warp(cutoff_ctx* c, int count, float* partial) {
    if (c->want_std) launch_sort_warp_sq<E, true>(c, count, partial);
    else launch_sort_warp_sq<E, false>(c, count, partial);
}

template <int WPR>
void launch_sort_cta(cutoff_ctx* c, int count, float* partial) {
    float* partial_sq = partial + static_cast<size_t>(kPartialRows) * c->N;
    if (c->want_std) k_sort_sum_cta<WPR, true><<<c->sort_grid, WPR * 32, 0, c->stream>>>(c->d_x, c->ldx, c->N, count, partial, partial_sq);
    else k_sort_sum_cta<WPR, false><<<c->sort_grid, WPR * 32, 0, c->stream>>>(c->d_x, c->ldx, c->N, count, partial, partial_sq);
}

int launch_sort(cutoff_ctx* c, int count, float* partial) {
    switch (c->P) {
        case 32: launch_sort_warp<1>(c, count, partial); break;
        case 64: launch_sort_warp<2>(c, count, partial); break;
        case 128: launch_sort_warp<4>(c, count, partial); break;
        case 256: launch_sort_warp<8>(c, count, partial); break;
        case 512: launch_sort_warp<16>(c, count, partial); break;
        case 1024: launch_sort_warp<32>(c, count, partial); break;
        case 2048: launch_sort_cta<2>(c, count, partial); break;
        case 4096: launch_sort_cta<4>(c, count, partial); break;
        default: return CUTOFF_ERR_UNSUPPORTED;
    }
    c->launches += 1;
    return CUTOFF_OK;
}

template <int D>
void launch_chain_t(cutoff_ctx* c, uint32_t sample_base, int count, size_t smem) {
    const NoiseKey key{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    const int round_v = c->cfg.precision != CUTOFF_PRECISION_FP32;
    const size_t resident = chain_resident_smem_floats(c->D, c->H, c->W) * sizeof(float);
    if (resident <= 200 * 1024) {
        // all weights fit: one persistent CTA per SM, as many as there are warp batches to hand out
        const int batch = 32 / ChainShape<D>::G * ChainShape<D>::SPL;
        const int batches = ceil_div(count, batch);
        const int grid = batches < c->sm_count ? batches : c->sm_count;
        k_chain_resident<D><<<grid, kChainResidentThreads, resident, c->stream>>>(c->m, c->d_hlr, c->d_state, key,
                                                                                sample_base, count, round_v, c->d_v);
    } else {
        k_chain<D><<<ceil_div(count, ChainShape<D>::kSamplesPerCta), ChainShape<D>::kThreads, smem, c->stream>>>(
            c->m, c->d_hlr, c->d_state, key, sample_base, count, round_v, c->d_v);
    }
}

void launch_chain_tc(cutoff_ctx* c, uint32_t sample_base, int count) {
    tc::ChainTcArgs a{};
    const ModelDev& m = c->m;
    a.image = c->d_chain_image;
    a.bz = m.bz; a.b1 = m.b1; a.b3 = m.b3; a.bmu = m.bmu; a.bsig = m.bsig; a.Wsig = m.Wsig; a.b2 = m.b2; a.z0 = m.z0;
    if (c->chain_tcl) {
        const LiteralDev& l = c->lit;
        a.b1 = l.bg1; a.b3 = l.bh1; a.b2 = nullptr;
        a.bi1 = l.bi1; a.bg2 = l.bg2; a.bh2 = l.bh2; a.Wl = l.Wl; a.bl = l.bl; a.bs = l.bs;
    }
    a.hlr = c->d_hlr; a.st = c->d_state;
    a.key = NoiseKey{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    a.sample_base = sample_base; a.count = count; a.H = c->H; a.W = c->W; a.round_v = 1; a.v_out = c->d_v;
    const int tiles = ceil_div(count, 128);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    if (c->chain_tcl) launch_dependent(tc::k_chain_tc<true>, dim3(grid), dim3(tc::kChainTcThreads), tc::chain_tc_smem_bytes(c->H, c->W, true), c->stream, a);
    else launch_dependent(tc::k_chain_tc<false>, dim3(grid), dim3(tc::kChainTcThreads), tc::chain_tc_smem_bytes(c->H, c->W), c->stream, a);
    c->launches += 1;
}

void launch_chain_tc32(cutoff_ctx* c, uint32_t sample_base, int count) {
    tc::ChainTc32Args a;
    const ModelDev& m = c->m;
    a.image = c->d_chain_image;
    a.bz = m.bz; a.b1 = m.b1; a.b3 = m.b3; a.bmu = m.bmu; a.bsig = m.bsig; a.Wsig = m.Wsig; a.b2 = m.b2; a.z0 = m.z0;
    if (c->chain_tcl32) {
        const LiteralDev& l = c->lit;
        a.b1 = l.bg1; a.b3 = l.bh1; a.b2 = nullptr;
        a.bi1 = l.bi1; a.bg2 = l.bg2; a.bh2 = l.bh2; a.Wl = l.Wl; a.bl = l.bl; a.bs = l.bs;
    }
    a.hlr = c->d_hlr; a.st = c->d_state;
    a.key = NoiseKey{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    a.sample_base = sample_base; a.count = count; a.H = c->H; a.W = c->W; a.round_v = 1; a.v_out = c->d_v;
    const int tiles = ceil_div(count, 128);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    if (c->chain_tcl32) tc::k_chain_tc32<true><<<grid, tc::kChainTcThreads, tc::chain_tc32_smem_bytes(c->H, c->W, true), c->stream>>>(a);
    else tc::k_chain_tc32<false><<<grid, tc::kChainTcThreads, tc::chain_tc32_smem_bytes(c->H, c->W), c->stream>>>(a);
    c->launches += 1;
}

template <int D>
void launch_chain_literal_t(cutoff_ctx* c, uint32_t sample_base, int count) {
    const NoiseKey key{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    const size_t smem = chain_smem_floats(c->D, c->H, c->W) * sizeof(float);
    k_chain_literal<D><<<ceil_div(count, ChainShape<D>::kSamplesPerCta), ChainShape<D>::kThreads, smem, c->stream>>>(
        c->m, c->lit, c->d_hlr, c->d_state, key, sample_base, count, c->use_tc ? 1 : 0, c->d_v);
}

void launch_chain(cutoff_ctx* c, uint32_t sample_base, int count) {
    if (c->chain_tcl) { launch_chain_tc(c, sample_base, count); return; }
    if (c->chain_tcl32) { launch_chain_tc32(c, sample_base, count); return; }
    if (c->literal) {
        switch (c->D) {
            case 4: launch_chain_literal_t<4>(c, sample_base, count); break;
            case 8: launch_chain_literal_t<8>(c, sample_base, count); break;
            case 16: launch_chain_literal_t<16>(c, sample_base, count); break;
            default: launch_chain_literal_t<32>(c, sample_base, count); break;
        }
        c->launches += 1;
        return;
    }
    if (c->chain_tc) { launch_chain_tc(c, sample_base, count); return; }
    if (c->chain_tc32) { launch_chain_tc32(c, sample_base, count); return; }
    const size_t smem = chain_smem_floats(c->D, c->H, c->W) * sizeof(float);
    switch (c->D) {
        case 4: launch_chain_t<4>(c, sample_base, count, smem); break;
        case 8: launch_chain_t<8>(c, sample_base, count, smem); break;
        case 16: launch_chain_t<16>(c, sample_base, count, smem); break;
        default: launch_chain_t<32>(c, sample_base, count, smem); break;
    }
    c->launches += 1;
}

// 2-D fp32 tensor map over a row-major [rows][cols] matrix, boxes of 128 rows x 32 columns
// (one 128-byte-swizzled K-major operand tile).  The driver entry point is looked up at run time.
int make_tile_map(cutoff_ctx* c, CUtensorMap* map, const float* base, uint64_t rows, uint64_t cols, uint64_t ld = 0) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        CU_CHECK(c, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) {
            if (c) c->last_error = "cuTensorMapEncodeTiled is not available from this driver";
            return CUTOFF_ERR_CUDA;
        }
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {(ld ? ld : cols) * sizeof(float)};
    const cuuint32_t box[2] = {tc::kBK, tc::kBM};
    const cuuint32_t elem[2] = {1, 1};
    const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box,
                              elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (c) c->last_error = "cuTensorMapEncodeTiled failed with code " + std::to_string(static_cast<int>(r));
        return CUTOFF_ERR_CUDA;
    }
    return CUTOFF_OK;
}

void launch_emission_tc(cutoff_ctx* c, uint32_t sample_base, int count) {
    tc::EmitArgs a;
    a.b4 = c->m.b4; a.x = c->d_x; a.st = c->d_state;
    a.key = NoiseKey{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    a.sample_base = sample_base; a.count = count; a.N = c->N; a.H = c->H; a.ldx = c->ldx;
    if (c->pair_emission && c->pair_clusters > 0 && count > tc::kBM) {
        // pairs of SMs share a weight tile: 256 samples x 128 workers per cluster and tile
        const int pair_tiles = ceil_div(c->N, tc::kBW) * ceil_div(count, 2 * tc::kBM);
        const int clusters = pair_tiles < c->pair_clusters ? pair_tiles : c->pair_clusters;
        tc::k_emit_tc2<<<2 * clusters, tc::kThreads, tc::kSmem2Bytes, c->stream>>>(c->map_v, c->map_w4, a);
        c->launches += 1;
        return;
    }
    const int tiles = ceil_div(c->N, tc::kBW) * ceil_div(count, tc::kBM);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    launch_dependent(tc::k_emit_tc, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, c->stream, c->map_v, c->map_w4, a);
    c->launches += 1;
}

// Literal emission (Section 3.1.3): I = u Wi2^T + bi2, r = relu(I Wj1^T + bj1), x = I + softplus(r Wj2^T + bj2) * eps.
void launch_gemm_relu_tc(cutoff_ctx* c, const CUtensorMap& map_a, const CUtensorMap& map_b, const tc::GemmTcArgs& a) {
    const int tiles = ceil_div(a.Nout, tc::kGemmBN) * ceil_div(a.M, tc::kBM);
    const int grid = tiles < c->sm_count ? tiles : c->sm_count;
    tc::k_gemm_relu_tc<<<grid, tc::kThreads, tc::kSmemBytes, c->stream>>>(map_a, map_b, a);
    c->launches += 1;
}

void launch_emission_literal(cutoff_ctx* c, uint32_t sample_base, int count) {
    const NoiseKey key{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    const LiteralDev& l = c->lit;
    if (c->use_tc) {
        // r = relu(M u + b') with M = Wj1 Wi2 (I is affine in u), then x = (Wi2 u + bi2) + softplus(Wj2 r + bj2) * eps
        tc::GemmTcArgs a{};
        a.st = c->d_state; a.M = count; a.bias = c->d_M + static_cast<size_t>(c->H) * c->H; a.out = c->d_r;
        a.ld_out = c->H; a.Nout = c->H; a.K = c->H;
        launch_gemm_relu_tc(c, c->map_v, c->map_M, a);
        tc::EmitDualArgs e;
        e.bias_mean = l.bi2; e.bias_scale = l.bj2; e.x = c->d_x; e.st = c->d_state; e.key = key;
        e.sample_base = sample_base; e.count = count; e.N = c->N; e.H = c->H; e.ldx = c->ldx;
        const int tiles = ceil_div(c->N, tc::kBW) * ceil_div(count, tc::kBM);
        tc::k_emit_dual_tc<<<tiles < c->sm_count ? tiles : c->sm_count, tc::kThreads, tc::kDualSmemBytes, c->stream>>>(
            c->map_v, c->map_r, c->map_wi2, c->map_wj2, e);
        c->launches += 1;
        return;
    }
    GemmFmaArgs a{};
    a.st = c->d_state; a.key = key; a.sample_base = sample_base; a.M = count;
    a.A = c->d_v; a.lda = c->H; a.B = l.Wi2; a.ldb = c->H; a.bias = l.bi2; a.out = c->d_I; a.ld_out = c->ldx;
    a.Nout = c->N; a.K = c->H;
    k_gemm_fma<kEpiAffine><<<dim3(ceil_div(a.Nout, kEmitTN), ceil_div(count, kEmitTM)), kEmitThreads, 0, c->stream>>>(a);
    a.A = c->d_I; a.lda = c->ldx; a.B = l.Wj1; a.ldb = l.ldn; a.bias = l.bj1; a.out = c->d_r; a.ld_out = c->H;
    a.Nout = c->H; a.K = c->ldx;                                   // the padding columns of both operands are zero
    k_gemm_fma<kEpiRelu><<<dim3(ceil_div(a.Nout, kEmitTN), ceil_div(count, kEmitTM)), kEmitThreads, 0, c->stream>>>(a);
    a.A = c->d_r; a.lda = c->H; a.B = l.Wj2; a.ldb = c->H; a.bias = l.bj2; a.add = c->d_I; a.out = c->d_x; a.ld_out = c->ldx;
    a.Nout = c->N; a.K = c->H;
    k_gemm_fma<kEpiScaleNoise><<<dim3(ceil_div(a.Nout, kEmitTN), ceil_div(count, kEmitTM)), kEmitThreads, 0, c->stream>>>(a);
    c->launches += 3;
}

void launch_emission(cutoff_ctx* c, uint32_t sample_base, int count) {
    if (c->literal) { launch_emission_literal(c, sample_base, count); return; }
    if (c->use_tc) { launch_emission_tc(c, sample_base, count); return; }
    const NoiseKey key{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    dim3 grid(ceil_div(c->N, kEmitTN), ceil_div(count, kEmitTM));
    k_emit_fma<<<grid, kEmitThreads, 0, c->stream>>>(c->m, c->d_v, c->d_state, key, sample_base, count, c->d_x, c->ldx);
    c->launches += 1;
}

template <int HQ>
void launch_rnn_resident(cutoff_ctx* c) {
    const size_t smem = enc_rnn_resident_smem_floats(c->H, c->W) * sizeof(float);
    k_enc_rnn_resident<HQ><<<2, 16 * HQ, smem, c->stream>>>(c->m, c->d_WhR, c->d_proj, c->d_state, c->d_hlr);
}

// Input projections: of the newest vector after a push, of every slot when the ring or the weights changed.
void launch_projection(cutoff_ctx* c, bool newest_only) {
    dim3 grid(ceil_div(c->H, kProjWarps), 2);
    k_enc_proj<<<grid, kProjWarps * 32, 0, c->stream>>>(c->m, c->d_ring, c->d_state, newest_only ? 1 : 0, c->d_proj);
    c->launches += 1;
}

void refresh_projections(cutoff_ctx* c) {
    if (!c->proj_stale) return;
    launch_projection(c, false);
    c->proj_stale = false;
}

void launch_encoder(cutoff_ctx* c) {
    refresh_projections(c);
    // H <= 128: one CTA per direction with the recurrence matrix in registers.  From H = 256 on a thread's share no
    // longer fits its registers, and a cluster of 8 CTAs per direction does the step in less time than one CTA that
    // keeps part of the matrix in shared memory (H = 256: 17 against 21 us).
    const size_t cluster_smem = enc_rnn_cluster_smem_floats(c->H, c->W) * sizeof(float);
    const size_t resident_smem = enc_rnn_resident_smem_floats(c->H, c->W) * sizeof(float);
    if (c->H == 32 && resident_smem <= 200 * 1024) launch_rnn_resident<8>(c);
    else if (c->H == 64 && resident_smem <= 200 * 1024) launch_rnn_resident<16>(c);
    else if (c->H == 128 && resident_smem <= 200 * 1024) launch_rnn_resident<32>(c);
    else if (c->H >= 256 && c->H % 32 == 0 && c->H <= 1024 && cluster_smem <= 200 * 1024)
        k_enc_rnn_cluster<<<2 * kRnnClusterSize, c->H, cluster_smem, c->stream>>>(c->m, c->d_proj, c->d_state, c->d_hlr);
    else
        k_enc_rnn<<<2, kRnnThreads, 2 * c->H * sizeof(float), c->stream>>>(c->m, c->d_proj, c->d_state, c->d_hlr);
    c->launches += 1;
}

int ensure_events(cutoff_ctx* c) {
    if (c->ev_created) return CUTOFF_OK;
    for (auto& row : c->ev)
        for (auto& e : row) CU_CHECK(c, cudaEventCreate(&e));
    c->ev_created = true;
    return CUTOFF_OK;
}

// Enqueue one decision's kernels.  decide = false stops after the per-position sums (a context that holds
// only part of a decision's samples: the argmax follows once the sums of all parts are added).
int enqueue_decision(cutoff_ctx* c, bool decide = true) {
    const bool timed = c->timing;
    if (timed) {
        const int rc = ensure_events(c);
        if (rc) return rc;
        cudaEventRecord(c->ev[0][0], c->stream);
    }
    launch_encoder(c);
    if (timed) cudaEventRecord(c->ev[1][0], c->stream);
    for (int ch = 0; ch < c->n_chunks; ++ch) {
        const int row0 = ch * c->chunk_rows;
        const int count = (c->S - row0) < c->chunk_rows ? (c->S - row0) : c->chunk_rows;
        const uint32_t base = static_cast<uint32_t>(c->cfg.sample_offset) + static_cast<uint32_t>(row0);
        if (timed && ch > 0) cudaEventRecord(c->ev[1][ch], c->stream);
        launch_chain(c, base, count);
        if (timed) cudaEventRecord(c->ev[2][ch], c->stream);
        launch_emission(c, base, count);
        if (timed) cudaEventRecord(c->ev[3][ch], c->stream);
        const int rc = launch_sort(c, count, c->d_partial + static_cast<size_t>(ch) * c->sort_grid * c->N);
        if (rc) return rc;
        if (timed) cudaEventRecord(c->ev[4][ch], c->stream);
    }
    const int64_t total = c->cfg.total_samples > 0 ? c->cfg.total_samples : c->S;
    launch_dependent(k_colsum_decide, dim3(ceil_div(c->N, 32)), dim3(kColsumThreads), 0, c->stream,
                     c->d_partial, c->n_chunks * c->sort_grid, c->N, c->d_sums, 1.0 / static_cast<double>(total), c->d_state,
                     c->d_E, c->d_omega, c->want_std ? c->d_partial + static_cast<size_t>(kPartialRows) * c->N : nullptr,
                     c->d_std, decide ? 1 : 0);
    c->have_std = c->want_std;
    c->launches += 1;
    if (timed) cudaEventRecord(c->ev[5][0], c->stream);
    c->timed_chunks = timed ? c->n_chunks : 0;
    CU_CHECK(c, cudaMemcpyAsync(c->h_state, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaGetLastError());
    return CUTOFF_OK;
}

int collect_timing(cutoff_ctx* c) {
    for (float& v : c->stage_ms) v = 0.0f;
    if (c->timed_chunks == 0) return CUTOFF_OK;
    float ms = 0.0f;
    CU_CHECK(c, cudaEventElapsedTime(&ms, c->ev[0][0], c->ev[1][0]));
    c->stage_ms[0] = ms;
    for (int ch = 0; ch < c->timed_chunks; ++ch) {
        for (int s = 1; s <= 3; ++s) {
            CU_CHECK(c, cudaEventElapsedTime(&ms, c->ev[s][ch], c->ev[s + 1][ch]));
            c->stage_ms[s] += ms;
        }
    }
    CU_CHECK(c, cudaEventElapsedTime(&ms, c->ev[4][c->timed_chunks - 1], c->ev[5][0]));
    c->stage_ms[4] = ms;
    return CUTOFF_OK;
}

bool valid_latent(int D) { return D == 4 || D == 8 || D == 16 || D == 32; }

// Kernels that need more than 48 KB of dynamic shared memory must be told so once per device.  Done at
// context creation, with the context's device current, for every kernel this context's shape can launch
// (a function attribute belongs to the device's copy of the kernel, not to the process).
template <typename Kernel>
cudaError_t allow_smem(Kernel kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
}

template <int E>
cudaError_t allow_smem_sort() {
    cudaError_t e = allow_smem(k_sort_sum_tma<E, false>, 100 * 1024);
    if (e == cudaSuccess) e = allow_smem(k_sort_sum_tma<E, true>, 100 * 1024);
    return e;
}

template <int D>
cudaError_t allow_smem_chain() {
    cudaError_t e = allow_smem(k_chain<D>, 220 * 1024);
    if (e == cudaSuccess) e = allow_smem(k_chain_resident<D>, 220 * 1024);
    if (e == cudaSuccess) e = allow_smem(k_chain_literal<D>, 220 * 1024);
    return e;
}

cudaError_t set_kernel_attributes(const cutoff_ctx* c) {
    cudaError_t e = cudaSuccess;
    switch (c->P) {
        case 32: e = allow_smem_sort<1>(); break;
        case 64: e = allow_smem_sort<2>(); break;
        case 128: e = allow_smem_sort<4>(); break;
        case 256: e = allow_smem_sort<8>(); break;
        case 512: e = allow_smem_sort<16>(); break;
        case 1024: e = allow_smem_sort<32>(); break;
        default: break;
    }
    if (e != cudaSuccess) return e;
    switch (c->D) {
        case 4: e = allow_smem_chain<4>(); break;
        case 8: e = allow_smem_chain<8>(); break;
        case 16: e = allow_smem_chain<16>(); break;
        default: e = allow_smem_chain<32>(); break;
    }
    if (e != cudaSuccess) return e;
    switch (c->H) {
        case 32: e = allow_smem(k_enc_rnn_resident<8>, 200 * 1024); break;
        case 64: e = allow_smem(k_enc_rnn_resident<16>, 200 * 1024); break;
        case 128: e = allow_smem(k_enc_rnn_resident<32>, 200 * 1024); break;
        default: break;
    }
    if (e == cudaSuccess) e = allow_smem(k_enc_rnn_cluster, 200 * 1024);
    if (e != cudaSuccess || !c->use_tc) return e;
    e = allow_smem(tc::k_emit_tc, tc::kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(tc::k_emit_tc2, tc::kSmem2Bytes);
    if (e == cudaSuccess) e = allow_smem(tc::k_gemm_relu_tc, tc::kSmemBytes);
    if (e == cudaSuccess) e = allow_smem(tc::k_emit_dual_tc, tc::kDualSmemBytes);
    if (e == cudaSuccess) e = allow_smem(tc::k_chain_tc<false>, 227 * 1024);
    if (e == cudaSuccess) e = allow_smem(tc::k_chain_tc<true>, 227 * 1024);
    if (e == cudaSuccess) e = allow_smem(tc::k_chain_tc32<false>, 227 * 1024);
    if (e == cudaSuccess) e = allow_smem(tc::k_chain_tc32<true>, 227 * 1024);
    return e;
}

}  // namespace

extern "C" {

const char* cutoff_strerror(int code) {
    switch (code) {
        case CUTOFF_OK: return "ok";
        case CUTOFF_WARMUP: return "warm-up: fewer than lag+1 observations, cutoff = all workers";
        case CUTOFF_DEGENERATE: return "no cutoff has a positive expected time, cutoff = all workers";
        case CUTOFF_ERR_BAD_ARG: return "bad argument";
        case CUTOFF_ERR_BAD_BLOB: return "weight blob does not match the context or is malformed";
        case CUTOFF_ERR_BAD_VALUE: return "run-times must be finite and greater than zero";
        case CUTOFF_ERR_CUDA: return "CUDA error";
        case CUTOFF_ERR_UNSUPPORTED: return "not supported";
        case CUTOFF_ERR_NOMEM: return "out of device memory";
        case CUTOFF_ERR_STATE: return "call out of order";
        case CUTOFF_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case CUTOFF_ERR_TOO_LARGE: return "request exceeds a fixed built-in capacity (see CUTOFF_STATIC_MAX_N)";
        default: return "unknown code";
    }
}

const char* cutoff_last_error(cutoff_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

const char* cutoff_stage_name(int i) { return (i >= 0 && i < kNumStages) ? kStageNames[i] : ""; }

int cutoff_create(cutoff_ctx** out, const cutoff_config* cfg) {
    if (!out || !cfg) return CUTOFF_ERR_BAD_ARG;
    if (cfg->n_workers < 1 || cfg->hidden < 4 || cfg->lag < 0 || cfg->n_samples < 1 || cfg->sample_offset < 0 ||
        cfg->total_samples < 0 || cfg->device < 0)
        return CUTOFF_ERR_BAD_ARG;
    if (cfg->precision < CUTOFF_PRECISION_FP32 || cfg->precision > CUTOFF_PRECISION_BF16W) return CUTOFF_ERR_BAD_ARG;
    if (!valid_latent(cfg->latent_dim) || cfg->hidden % cfg->latent_dim != 0) return CUTOFF_ERR_UNSUPPORTED;
    if (cfg->n_workers > 4096 || cfg->hidden > 1024 || cfg->lag > 255) return CUTOFF_ERR_UNSUPPORTED;
    if (cfg->sample_offset + cfg->n_samples > (1ll << 32)) return CUTOFF_ERR_UNSUPPORTED;
    if (cfg->total_samples > 0 && cfg->total_samples < cfg->n_samples) return CUTOFF_ERR_BAD_ARG;

    cutoff_ctx* c = new (std::nothrow) cutoff_ctx();
    if (!c) return CUTOFF_ERR_NOMEM;
    c->cfg = *cfg;
    c->N = cfg->n_workers; c->D = cfg->latent_dim; c->H = cfg->hidden; c->W = cfg->lag + 1; c->S = cfg->n_samples;
    c->ldx = (c->N + 7) & ~7;
    c->P = next_pow2(c->N) < 32 ? 32 : next_pow2(c->N);
    c->stream = static_cast<cudaStream_t>(cfg->stream);
    c->literal = (cfg->flags & CUTOFF_FLAG_LITERAL) != 0;

    auto fail = [&](int rc) { free_all(c); delete c; return rc; };
#define CREATE_CHECK(call)                                                                         \
    do {                                                                                           \
        cudaError_t err__ = (call);                                                                \
        if (err__ != cudaSuccess) return fail(err__ == cudaErrorMemoryAllocation ? CUTOFF_ERR_NOMEM : CUTOFF_ERR_CUDA); \
    } while (0)

    DeviceGuard guard(cfg->device);
    CREATE_CHECK(guard.err);
    if ((cfg->flags & CUTOFF_FLAG_GRAPH) && !c->stream) {
        // the default stream cannot be captured: graph mode without a caller stream runs on its own
        CREATE_CHECK(cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking));
        c->owns_stream = true;
    }
    cudaDeviceProp prop;
    CREATE_CHECK(cudaGetDeviceProperties(&prop, cfg->device));
    c->sm_count = prop.multiProcessorCount;
    if (chain_smem_floats(c->D, c->H, c->W) * sizeof(float) > 220 * 1024) return fail(CUTOFF_ERR_UNSUPPORTED);

    // Pass buffers hold up to 2 GiB of samples; by default one pass covers all S samples.
    {
        // per sample: x and v; literal variant: also r, and I on the fp32 path
        const bool tensor_path = cfg->precision != CUTOFF_PRECISION_FP32;
        const int64_t row_floats = c->ldx + c->H + (c->literal ? c->H + (tensor_path ? 0 : c->ldx) : 0);
        int64_t cap = (2ll << 30) / (row_floats * static_cast<int64_t>(sizeof(float)));
        if (cap < 1024) cap = 1024;
        c->alloc_rows = cap < c->S ? static_cast<int>(cap) : c->S;
    }
    if (ceil_div(c->S, kMaxChunks) > c->alloc_rows) return fail(CUTOFF_ERR_UNSUPPORTED);   // S too large for the pass buffers
    plan_chunks(c, c->alloc_rows);
    c->use_tc = cfg->precision != CUTOFF_PRECISION_FP32;
    c->chain_tc = !c->literal && c->use_tc && c->D == tc::kChainD && c->H % 64 == 0 && c->H <= 256 &&
                  tc::chain_tc_smem_bytes(c->H, c->W) <= 227 * 1024;
    c->chain_tcl = c->literal && c->use_tc && c->D == tc::kChainD && c->H % 64 == 0 && c->H <= 256 &&
                   tc::chain_tc_smem_bytes(c->H, c->W, true) <= 227 * 1024;
    c->chain_tc32 = !c->literal && c->use_tc && c->D == tc::kChain32D && c->H % 32 == 0 && c->H <= 512 &&
                    (c->H <= 256 || (c->H - 256) % 16 == 0) && tc::chain_tc32_smem_bytes(c->H, c->W) <= 227 * 1024;
    c->chain_tcl32 = c->literal && c->use_tc && c->D == tc::kChain32D && c->H % 32 == 0 && c->H <= 512 &&
                     (c->H <= 256 || (c->H - 256) % 16 == 0) && tc::chain_tc32_smem_bytes(c->H, c->W, true) <= 227 * 1024;

    size_t blob_floats = 0;
    for (const auto& t : c->literal ? tensor_specs_literal(c->N, c->D, c->H) : tensor_specs(c->N, c->D, c->H))
        blob_floats += (t.rows * t.cols + 7) / 8 * 8;            // each tensor starts on a 32-byte boundary
    CREATE_CHECK(cudaMalloc(&c->d_blob, blob_floats * sizeof(float)));
    CREATE_CHECK(cudaMalloc(&c->d_WT, sizeof(float) * 4 * c->H * c->D));
    if (c->literal) {
        CREATE_CHECK(cudaMalloc(&c->d_r, sizeof(float) * static_cast<size_t>(c->alloc_rows) * c->H));
        if (c->use_tc) {
            CREATE_CHECK(cudaMalloc(&c->d_M, sizeof(float) * (static_cast<size_t>(c->H) * c->H + c->H)));
        } else {
            CREATE_CHECK(cudaMalloc(&c->d_I, sizeof(float) * static_cast<size_t>(c->alloc_rows) * c->ldx));
            CREATE_CHECK(cudaMalloc(&c->d_Wj1p, sizeof(float) * static_cast<size_t>(c->H) * c->ldx));
            // the padding columns of I are never written and must read as zero
            CREATE_CHECK(cudaMemsetAsync(c->d_I, 0, sizeof(float) * static_cast<size_t>(c->alloc_rows) * c->ldx, c->stream));
        }
    }
    CREATE_CHECK(cudaMalloc(&c->d_WhR, sizeof(float) * 2 * c->H * c->H));
    if (c->chain_tc) CREATE_CHECK(cudaMalloc(&c->d_chain_image, sizeof(float) * tc::chain_tc_image_floats(c->H)));
    if (c->chain_tc32) CREATE_CHECK(cudaMalloc(&c->d_chain_image, sizeof(float) * tc::chain_tc32_image_floats(c->H)));
    if (c->chain_tcl) CREATE_CHECK(cudaMalloc(&c->d_chain_image, sizeof(float) * tc::chain_tc_image_floats(c->H, true)));
    if (c->chain_tcl32) CREATE_CHECK(cudaMalloc(&c->d_chain_image, sizeof(float) * tc::chain_tc32_image_floats(c->H, true)));
    CREATE_CHECK(cudaMalloc(&c->d_ring, sizeof(float) * c->W * c->N));
    CREATE_CHECK(cudaMalloc(&c->d_stage, sizeof(float) * c->N));
    CREATE_CHECK(cudaMalloc(&c->d_mask, c->N));
    CREATE_CHECK(cudaMallocHost(&c->h_mask, c->N));
    CREATE_CHECK(cudaMalloc(&c->d_state, sizeof(DevState)));
    CREATE_CHECK(cudaMalloc(&c->d_proj, sizeof(float) * 2 * c->W * c->H));
    CREATE_CHECK(cudaMalloc(&c->d_hlr, sizeof(float) * 2 * c->W * c->H));
    CREATE_CHECK(cudaMalloc(&c->d_v, sizeof(float) * static_cast<size_t>(c->alloc_rows) * c->H));
    CREATE_CHECK(cudaMalloc(&c->d_x, sizeof(float) * static_cast<size_t>(c->alloc_rows) * c->ldx));
    CREATE_CHECK(cudaMalloc(&c->d_partial, sizeof(float) * 2 * static_cast<size_t>(kPartialRows) * c->N));
    CREATE_CHECK(cudaMalloc(&c->d_std, sizeof(float) * c->N));
    CREATE_CHECK(cudaMalloc(&c->d_sums, sizeof(double) * c->N));
    CREATE_CHECK(cudaMalloc(&c->d_E, sizeof(float) * c->N));
    CREATE_CHECK(cudaMalloc(&c->d_omega, sizeof(float) * c->N));
    if (c->use_tc) {
        int rc = make_tile_map(c, &c->map_v, c->d_v, static_cast<uint64_t>(c->alloc_rows), static_cast<uint64_t>(c->H));
        if (!rc && c->literal)
            rc = make_tile_map(c, &c->map_M, c->d_M, static_cast<uint64_t>(c->H), static_cast<uint64_t>(c->H));
        if (!rc && c->literal)
            rc = make_tile_map(c, &c->map_r, c->d_r, static_cast<uint64_t>(c->alloc_rows), static_cast<uint64_t>(c->H));
        if (rc) return fail(rc);
    }
    CREATE_CHECK(set_kernel_attributes(c));
    if (c->use_tc && !c->literal) {
        // how many two-CTA clusters of the two-SM emission kernel the GPU can hold at once
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3(2 * c->sm_count);
        lc.blockDim = dim3(tc::kThreads);
        lc.dynamicSmemBytes = tc::kSmem2Bytes;
        cudaLaunchAttribute at{};
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
        lc.attrs = &at;
        lc.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, tc::k_emit_tc2, &lc) == cudaSuccess && n > 0) c->pair_clusters = n;
        else cudaGetLastError();
    }
    CREATE_CHECK(cudaMallocHost(&c->h_stage, sizeof(float) * c->N));
    CREATE_CHECK(cudaMallocHost(&c->h_state, sizeof(DevState)));
    CREATE_CHECK(cudaMemsetAsync(c->d_state, 0, sizeof(DevState), c->stream));
    CREATE_CHECK(cudaMemsetAsync(c->d_ring, 0, sizeof(float) * c->W * c->N, c->stream));
    CREATE_CHECK(cudaStreamSynchronize(c->stream));
#undef CREATE_CHECK
    *out = c;
    return CUTOFF_OK;
}

void cutoff_destroy(cutoff_ctx* ctx) {
    if (!ctx) return;
    DeviceGuard guard(ctx->cfg.device);
    cudaStreamSynchronize(ctx->stream);
    free_all(ctx);
    delete ctx;
}

int cutoff_load_weights(cutoff_ctx* c, const void* blob, size_t nbytes) {
    if (!c || !blob) return CUTOFF_ERR_BAD_ARG;
    if (nbytes < 6 * sizeof(uint32_t)) return CUTOFF_ERR_BAD_BLOB;
    uint32_t hdr[6];
    std::memcpy(hdr, blob, sizeof(hdr));
    if (hdr[0] != kBlobMagic || hdr[1] != 1u) return CUTOFF_ERR_BAD_BLOB;
    if (hdr[2] != static_cast<uint32_t>(c->N) || hdr[3] != static_cast<uint32_t>(c->D) ||
        hdr[4] != static_cast<uint32_t>(c->H) || hdr[5] != (c->literal ? 1u : 0u))
        return CUTOFF_ERR_BAD_BLOB;
    const auto specs = c->literal ? tensor_specs_literal(c->N, c->D, c->H) : tensor_specs(c->N, c->D, c->H);
    size_t total = 0;
    for (const auto& t : specs) total += t.rows * t.cols;
    if (nbytes != sizeof(hdr) + total * sizeof(float)) return CUTOFF_ERR_BAD_BLOB;
    const float* src = reinterpret_cast<const float*>(static_cast<const char*>(blob) + sizeof(hdr));
    for (size_t i = 0; i < total; ++i)
        if (!std::isfinite(src[i])) return CUTOFF_ERR_BAD_BLOB;

    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    // device layout: every tensor starts on a 32-byte boundary (16-byte loads and tensor maps need aligned bases)
    std::vector<size_t> off(specs.size());
    size_t o = 0;
    for (size_t i = 0; i < specs.size(); ++i) { off[i] = o; o += (specs[i].rows * specs[i].cols + 7) / 8 * 8; }
    std::vector<float> host(o, 0.0f);
    {
        size_t so = 0;
        for (size_t i = 0; i < specs.size(); ++i) {
            const size_t n = specs[i].rows * specs[i].cols;
            std::memcpy(host.data() + off[i], src + so, n * sizeof(float));
            so += n;
        }
    }
    if (c->use_tc) {
        // Weights of the products that run on the tensor cores, as the tensor cores will see them, kept as
        // fp32 bit patterns: bf16 (nearest even) for the bf16-weight precision, else tf32 (nearest, ties
        // away from zero).  Compact variant: W4; literal variant: Wi2, Wj1, Wj2.
        const std::vector<size_t> rounded = c->literal ? std::vector<size_t>{29, 31, 33} : std::vector<size_t>{21};
        for (size_t t : rounded) {
            float* wt = host.data() + off[t];
            for (size_t i = 0; i < specs[t].rows * specs[t].cols; ++i) {
                uint32_t u;
                std::memcpy(&u, &wt[i], 4);
                if (c->cfg.precision == CUTOFF_PRECISION_BF16W) u = (u + 0x7FFFu + ((u >> 16) & 1u)) & 0xFFFF0000u;
                else u = (u + 0x1000u) & 0xFFFFE000u;
                std::memcpy(&wt[i], &u, 4);
            }
        }
    }
    CU_CHECK(c, cudaMemcpy(c->d_blob, host.data(), host.size() * sizeof(float), cudaMemcpyHostToDevice));
    // transposed copies [D][H] of the latent-to-hidden matrices for the per-sample chain
    const size_t D = c->D, H = c->H;
    const int n_transposed = c->literal ? 4 : 3;
    std::vector<float> wT(n_transposed * H * D);
    const size_t src_off[4] = {off[8], off[15], off[19], c->literal ? off[27] : 0};   // Wz, W1 | Wg1, W3 | Wh1, - | Wi1
    for (int t = 0; t < n_transposed; ++t) {
        const float* w = host.data() + src_off[t];
        for (size_t i = 0; i < H; ++i)
            for (size_t d = 0; d < D; ++d) wT[t * H * D + d * H + i] = w[i * D + d];
    }
    CU_CHECK(c, cudaMemcpy(c->d_WT, wT.data(), wT.size() * sizeof(float), cudaMemcpyHostToDevice));

    if (H == 32 || H == 64 || H == 128) {
        // recurrence matrices regrouped per thread of k_enc_rnn_resident (the widths that kernel serves; the layout
        // needs H / 4 to be a multiple of 4): [dir][j4][thread = 4*i + q][4]
        const size_t HQ = H / 4, T = 4 * H;
        std::vector<float> whr(2 * H * H);
        const size_t src_off[2] = {off[1], off[5]};                   // Whf, Whb: each [H][H]
        for (int dir = 0; dir < 2; ++dir) {
            const float* w = host.data() + src_off[dir];
            for (size_t i = 0; i < H; ++i)
                for (size_t q = 0; q < 4; ++q)
                    for (size_t j = 0; j < HQ; ++j)
                        whr[dir * H * H + ((j / 4) * T + (4 * i + q)) * 4 + (j % 4)] = w[i * H + q * HQ + j];
        }
        CU_CHECK(c, cudaMemcpy(c->d_WhR, whr.data(), whr.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    // Operand tiles of the tensor-core chain kernels as they will sit in shared memory: tf32 (nearest, ties away),
    // K-major rows of 32 values, 16-byte chunks XOR-swizzled with the row index modulo 8.
    if (c->chain_tc || c->chain_tcl || c->chain_tc32 || c->chain_tcl32) {
        const bool lit = c->chain_tcl || c->chain_tcl32;
        const float* wz = host.data() + off[8];                  // first layers, [H][D]: Wz; W1 or Wg1; W3 or Wh1; Wi1
        const float* wa = host.data() + off[15];
        const float* wb = host.data() + off[19];
        const float* wi1 = lit ? host.data() + off[27] : nullptr;
        const float* wmu = host.data() + off[10];                // second layers, [D][H] ([2D][H] for W2): Wmu; W2 or Wg2; Wh2
        const float* wc = host.data() + off[17];
        const float* wh2 = lit ? host.data() + off[21] : nullptr;
        const float* ws = lit ? host.data() + off[25] : nullptr; // [D][D]
        const size_t tile = H * 32;
        std::vector<float> img;
        if (c->chain_tc || c->chain_tcl) {
            // D = 16: two first-layer matrices share a tile (columns 0..15 and 16..31); second-layer K blocks of 16 rows
            // (W2: 32).  compact: [Wz|W1], W3, Wmu, W2;  literal: [Wz|Wg1], [Wh1|Wi1], Wmu, Wg2, Wh2, Ws (16 rows)
            img.assign(tc::chain_tc_image_floats(c->H, lit), 0.0f);
            float* t_in0 = img.data();
            float* t_in1 = t_in0 + tile;
            float* t_wmu = t_in1 + tile;
            float* t_out1 = t_wmu + H * 16;
            put_first_layer(t_in0, wz, H, D, 0);
            put_first_layer(t_in0, wa, H, D, 16);
            put_first_layer(t_in1, wb, H, D, 0);
            put_second_layer(t_wmu, wmu, D, H, 16);
            if (lit) {
                float* t_out2 = t_out1 + H * 16;
                put_first_layer(t_in1, wi1, H, D, 16);
                put_second_layer(t_out1, wc, D, H, 16);
                put_second_layer(t_out2, wh2, D, H, 16);
                put_first_layer(t_out2 + H * 16, ws, D, D, 0);
            } else {
                put_second_layer(t_out1, wc, 2 * D, H, 32);
            }
        } else {
            // D = 32: every matrix has a tile of H x 32 of its own, staged by the kernel phase by phase.
            // compact: Wz, W1, W3, Wmu, W2 mean rows, W2 log-variance rows;  literal: Wz, Wg1, Wh1, Wi1, Wmu, Wg2, Wh2, Ws
            img.assign(tc::chain_tc32_image_floats(c->H, lit), 0.0f);
            put_first_layer(img.data() + 0 * tile, wz, H, 32, 0);
            put_first_layer(img.data() + 1 * tile, wa, H, 32, 0);
            put_first_layer(img.data() + 2 * tile, wb, H, 32, 0);
            if (lit) {
                put_first_layer(img.data() + 3 * tile, wi1, H, 32, 0);
                put_second_layer(img.data() + 4 * tile, wmu, 32, H, 32);
                put_second_layer(img.data() + 5 * tile, wc, 32, H, 32);
                put_second_layer(img.data() + 6 * tile, wh2, 32, H, 32);
                put_first_layer(img.data() + 7 * tile, ws, 32, 32, 0);
            } else {
                put_second_layer(img.data() + 3 * tile, wmu, 32, H, 32);
                put_second_layer(img.data() + 4 * tile, wc, 32, H, 32);
                put_second_layer(img.data() + 5 * tile, wc + 32 * H, 32, H, 32);
            }
        }
        CU_CHECK(c, cudaMemcpy(c->d_chain_image, img.data(), img.size() * sizeof(float), cudaMemcpyHostToDevice));
    }

    ModelDev& m = c->m;
    m.N = c->N; m.D = c->D; m.H = c->H; m.W = c->W;
    const float* b = c->d_blob;
    m.Wxf = b + off[0]; m.Whf = b + off[1]; m.bf = b + off[2]; m.a0 = b + off[3];
    m.Wxb = b + off[4]; m.Whb = b + off[5]; m.bb = b + off[6]; m.b0 = b + off[7];
    m.WzT = c->d_WT; m.bz = b + off[9]; m.Wmu = b + off[10]; m.bmu = b + off[11];
    m.Wsig = b + off[12]; m.bsig = b + off[13]; m.z0 = b + off[14];
    if (c->literal) {
        if (c->use_tc) {
            // I = Wi2 u + bi2 is affine in u, so Wj1 I + bj1 = M u + b' with M = Wj1 Wi2 [H][H] and b' = Wj1 bi2 + bj1:
            // formed here once, in double, from the weights as the tensor cores see them; M is rounded to tf32.
            const size_t N = c->N;
            const float* wj1 = host.data() + off[31];    // [H][N]
            const float* wi2 = host.data() + off[29];    // [N][H]
            const float* bi2 = host.data() + off[30];
            const float* bj1 = host.data() + off[32];
            std::vector<float> mb(H * H + H);
            std::vector<double> acc(H);
            for (size_t i = 0; i < H; ++i) {
                std::fill(acc.begin(), acc.end(), 0.0);
                double bacc = bj1[i];
                for (size_t k = 0; k < N; ++k) {
                    const double w = wj1[i * N + k];
                    const float* row = wi2 + k * H;
                    for (size_t j = 0; j < H; ++j) acc[j] += w * row[j];
                    bacc += w * bi2[k];
                }
                for (size_t j = 0; j < H; ++j) {
                    float f = static_cast<float>(acc[j]);
                    uint32_t u;
                    std::memcpy(&u, &f, 4);
                    u = (u + 0x1000u) & 0xFFFFE000u;
                    std::memcpy(&f, &u, 4);
                    mb[i * H + j] = f;
                }
                mb[H * H + i] = static_cast<float>(bacc);
            }
            CU_CHECK(c, cudaMemcpy(c->d_M, mb.data(), mb.size() * sizeof(float), cudaMemcpyHostToDevice));
        } else {
            // Wj1 [H][N] with rows padded with zeros to ldx floats (rows then start on 32 bytes for any N)
            std::vector<float> wj1p(H * static_cast<size_t>(c->ldx), 0.0f);
            for (size_t i = 0; i < H; ++i)
                std::memcpy(wj1p.data() + i * c->ldx, host.data() + off[31] + i * c->N, sizeof(float) * c->N);
            CU_CHECK(c, cudaMemcpy(c->d_Wj1p, wj1p.data(), wj1p.size() * sizeof(float), cudaMemcpyHostToDevice));
        }
        LiteralDev& l = c->lit;
        l.Wg1T = c->d_WT + H * D; l.bg1 = b + off[16]; l.Wg2 = b + off[17]; l.bg2 = b + off[18];
        l.Wh1T = c->d_WT + 2 * H * D; l.bh1 = b + off[20]; l.Wh2 = b + off[21]; l.bh2 = b + off[22];
        l.Wl = b + off[23]; l.bl = b + off[24]; l.Ws = b + off[25]; l.bs = b + off[26];
        l.Wi1T = c->d_WT + 3 * H * D; l.bi1 = b + off[28];
        l.Wi2 = b + off[29]; l.bi2 = b + off[30];
        l.Wj1 = c->d_Wj1p; l.bj1 = b + off[32]; l.ldn = c->ldx;
        l.Wj2 = b + off[33]; l.bj2 = b + off[34];
        m.W1T = m.b1 = m.W2 = m.b2 = m.W3T = m.b3 = m.W4 = m.b4 = nullptr;
        if (c->use_tc) {
            int rc = make_tile_map(c, &c->map_wi2, l.Wi2, static_cast<uint64_t>(c->N), static_cast<uint64_t>(c->H));
            if (!rc) rc = make_tile_map(c, &c->map_wj2, l.Wj2, static_cast<uint64_t>(c->N), static_cast<uint64_t>(c->H));
            if (rc) return rc;
        }
        c->weights_loaded = true;
        c->proj_stale = true;
        return CUTOFF_OK;
    }
    m.W1T = c->d_WT + H * D; m.b1 = b + off[16]; m.W2 = b + off[17]; m.b2 = b + off[18];
    m.W3T = c->d_WT + 2 * H * D; m.b3 = b + off[20]; m.W4 = b + off[21]; m.b4 = b + off[22];
    if (c->use_tc) {
        const int rc = make_tile_map(c, &c->map_w4, m.W4, 2ull * c->N, static_cast<uint64_t>(c->H));
        if (rc) return rc;
    }
    c->weights_loaded = true;
    c->proj_stale = true;
    return CUTOFF_OK;
}

static int push_common(cutoff_ctx* c, const float* dev_src) {
    k_push<<<1, kPushThreads, 0, c->stream>>>(dev_src, c->d_ring, c->d_state, c->N, c->W);
    c->launches += 1;
    if (c->weights_loaded && !c->proj_stale) launch_projection(c, true);     // else every slot is redone before the next decision
    CU_CHECK(c, cudaGetLastError());
    c->pushes += 1;
    return CUTOFF_OK;
}

int cutoff_push_async(cutoff_ctx* c, const float* runtimes_sec_device) {
    if (!c || !runtimes_sec_device) return CUTOFF_ERR_BAD_ARG;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    return push_common(c, runtimes_sec_device);
}

// Push with a censoring mask: land run-times and mask on the device, replace the censored entries by
// draws from the truncated predictive distribution of the last decision, then push as usual.
static int push_censored(cutoff_ctx* c, const float* runtimes_sec, int on_device, const uint8_t* censored) {
    if (!c->draws_valid) return CUTOFF_ERR_STATE;          // no decision yet whose draws could be used
    if (c->cfg.sample_offset != 0 || (c->cfg.total_samples > 0 && c->cfg.total_samples != c->S))
        return CUTOFF_ERR_UNSUPPORTED;                      // a context that holds only part of the draws
    const cudaMemcpyKind kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    if (!on_device) {
        int finished = 0;
        for (int j = 0; j < c->N; ++j) {
            if (censored[j]) continue;
            if (!(runtimes_sec[j] > 0.0f) || !std::isfinite(runtimes_sec[j])) return CUTOFF_ERR_BAD_VALUE;
            ++finished;
        }
        if (finished == 0) return CUTOFF_ERR_BAD_ARG;
        CU_CHECK(c, cudaStreamSynchronize(c->stream));     // the landing buffers may still be in use
        for (int j = 0; j < c->N; ++j) c->h_stage[j] = censored[j] ? 1.0f : runtimes_sec[j];
        std::memcpy(c->h_mask, censored, c->N);
        CU_CHECK(c, cudaMemcpyAsync(c->d_stage, c->h_stage, sizeof(float) * c->N, kind, c->stream));
        CU_CHECK(c, cudaMemcpyAsync(c->d_mask, c->h_mask, c->N, kind, c->stream));
    } else {
        CU_CHECK(c, cudaMemcpyAsync(c->d_stage, runtimes_sec, sizeof(float) * c->N, kind, c->stream));
        CU_CHECK(c, cudaMemcpyAsync(c->d_mask, censored, c->N, kind, c->stream));
    }
    const NoiseKey key{static_cast<uint32_t>(c->cfg.seed), static_cast<uint32_t>(c->cfg.seed >> 32)};
    k_impute<<<1, kImputeThreads, 0, c->stream>>>(c->d_stage, c->d_mask, c->d_x, c->ldx, c->S, c->N, c->d_state, key);
    c->launches += 1;
    c->draws_valid = false;                                 // one step's draws serve one push
    int rc = push_common(c, c->d_stage);
    if (rc) return rc;
    CU_CHECK(c, cudaMemcpyAsync(c->h_state, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    if (c->h_state->error_flags & (kErrBadValue | kErrNoFinisher)) {
        c->pushes = c->h_state->push_count;
        CU_CHECK(c, cudaMemsetAsync(&c->d_state->error_flags, 0, sizeof(int32_t), c->stream));
        return CUTOFF_ERR_BAD_VALUE;
    }
    return CUTOFF_OK;
}

int cutoff_push(cutoff_ctx* c, const float* runtimes_sec, int on_device, const uint8_t* censored) {
    if (!c || !runtimes_sec) return CUTOFF_ERR_BAD_ARG;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    if (censored) return push_censored(c, runtimes_sec, on_device, censored);
    if (!on_device) {
        for (int j = 0; j < c->N; ++j)
            if (!(runtimes_sec[j] > 0.0f) || !std::isfinite(runtimes_sec[j])) return CUTOFF_ERR_BAD_VALUE;
        CU_CHECK(c, cudaStreamSynchronize(c->stream));       // the landing buffer may still be in use
        std::memcpy(c->h_stage, runtimes_sec, sizeof(float) * c->N);
        CU_CHECK(c, cudaMemcpyAsync(c->d_stage, c->h_stage, sizeof(float) * c->N, cudaMemcpyHostToDevice, c->stream));
        return push_common(c, c->d_stage);
    }
    const int rc = push_common(c, runtimes_sec);
    if (rc) return rc;
    CU_CHECK(c, cudaMemcpyAsync(c->h_state, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    if (c->h_state->error_flags & kErrBadValue) {
        // the kernel left the window untouched; clear the flag and undo the host-side count
        c->pushes = c->h_state->push_count;
        CU_CHECK(c, cudaMemsetAsync(&c->d_state->error_flags, 0, sizeof(int32_t), c->stream));
        return CUTOFF_ERR_BAD_VALUE;
    }
    return CUTOFF_OK;
}

int cutoff_predict_async(cutoff_ctx* c) {
    if (!c) return CUTOFF_ERR_BAD_ARG;
    if (!c->weights_loaded) return CUTOFF_ERR_STATE;
    if (c->pending || c->partial_pending) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    c->pending = true;
    c->pending_warmup = c->pushes < static_cast<uint32_t>(c->W);
    if (c->pending_warmup) {
        // nothing to compute; still read the state so that a bad device push is reported
        CU_CHECK(c, cudaMemcpyAsync(c->h_state, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
        return CUTOFF_OK;
    }
    const int rc = enqueue_decision(c);
    if (rc) c->pending = false;
    return rc;
}

int cutoff_fetch(cutoff_ctx* c, int32_t* c_out) {
    if (!c || !c_out) return CUTOFF_ERR_BAD_ARG;
    if (!c->pending) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    c->pending = false;
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    if (c->h_state->error_flags & kErrBadValue) {
        c->pushes = c->h_state->push_count;
        CU_CHECK(c, cudaMemsetAsync(&c->d_state->error_flags, 0, sizeof(int32_t), c->stream));
        return CUTOFF_ERR_BAD_VALUE;
    }
    if (c->h_state->error_flags & kErrTimeout) return CUTOFF_ERR_TIMEOUT;
    if (c->pending_warmup) {
        *c_out = c->N;
        return CUTOFF_WARMUP;
    }
    const int rc = collect_timing(c);
    if (rc) return rc;
    c->have_result = true;
    c->decided_once = true;
    c->draws_valid = c->n_chunks == 1;
    *c_out = c->h_state->c_star;
    return c->h_state->code == 2 ? CUTOFF_DEGENERATE : CUTOFF_OK;
}

int cutoff_predict(cutoff_ctx* c, int32_t* c_out) {
    if (!c || !c_out) return CUTOFF_ERR_BAD_ARG;
    const int rc = cutoff_predict_async(c);
    if (rc < 0) return rc;
    return cutoff_fetch(c, c_out);
}

// Capture "land the staged run-times, push, decide, read back the state" once; replays need no
// changing argument because the window position, the normaliser and the decision counter live
// in device memory.
static int build_graph(cutoff_ctx* c, bool with_host_copy) {
    refresh_projections(c);                        // not part of the graph: replays only project the vector they push
    const int64_t launches_before = c->launches;
    CU_CHECK(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
    if (with_host_copy) cudaMemcpyAsync(c->d_stage, c->h_stage, sizeof(float) * c->N, cudaMemcpyHostToDevice, c->stream);
    k_push<<<1, kPushThreads, 0, c->stream>>>(c->d_stage, c->d_ring, c->d_state, c->N, c->W);
    c->launches += 1;
    launch_projection(c, true);
    const bool timing = c->timing;
    c->timing = false;
    const int rc = enqueue_decision(c);
    c->timing = timing;
    cudaGraph_t g = nullptr;
    const cudaError_t end = cudaStreamEndCapture(c->stream, &g);
    c->graph_kernels = static_cast<int>(c->launches - launches_before);
    c->launches = launches_before;                 // nothing ran yet
    if (rc != CUTOFF_OK || end != cudaSuccess || !g) {
        if (g) cudaGraphDestroy(g);
        c->last_error = std::string("graph capture failed: ") + cudaGetErrorString(end);
        cudaGetLastError();
        return CUTOFF_ERR_CUDA;
    }
    if (with_host_copy) {
        c->graph = g;
        CU_CHECK(c, cudaGraphInstantiate(&c->graph_exec, c->graph, 0));
    } else {
        c->graph_dev = g;
        CU_CHECK(c, cudaGraphInstantiate(&c->graph_dev_exec, c->graph_dev, 0));
    }
    return CUTOFF_OK;
}

int cutoff_step(cutoff_ctx* c, const float* runtimes_sec, int32_t* c_out) {
    if (!c || !runtimes_sec || !c_out) return CUTOFF_ERR_BAD_ARG;
    if (!c->weights_loaded || c->pending) return CUTOFF_ERR_STATE;
    const bool replay = (c->cfg.flags & CUTOFF_FLAG_GRAPH) && c->decided_once &&
                        c->pushes + 1 >= static_cast<uint32_t>(c->W);
    if (!replay) {
        const int rc = cutoff_push(c, runtimes_sec, 0, nullptr);
        if (rc < 0) return rc;
        return cutoff_predict(c, c_out);
    }
    for (int j = 0; j < c->N; ++j)
        if (!(runtimes_sec[j] > 0.0f) || !std::isfinite(runtimes_sec[j])) return CUTOFF_ERR_BAD_VALUE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    if (!c->graph_exec) {
        CU_CHECK(c, cudaStreamSynchronize(c->stream));
        const int rc = build_graph(c, true);
        if (rc) return rc;
    }
    std::memcpy(c->h_stage, runtimes_sec, sizeof(float) * c->N);     // the stream is idle: every call ends synchronised
    refresh_projections(c);                        // after a restore or new weights; the replay then adds the new vector
    CU_CHECK(c, cudaGraphLaunch(c->graph_exec, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    c->launches += c->graph_kernels;
    c->pushes += 1;
    c->draws_valid = c->n_chunks == 1;
    if (c->h_state->error_flags & kErrTimeout) return CUTOFF_ERR_TIMEOUT;
    c->have_result = true;
    *c_out = c->h_state->c_star;
    return c->h_state->code == 2 ? CUTOFF_DEGENERATE : CUTOFF_OK;
}

int cutoff_step_device(cutoff_ctx* c, const float* runtimes_sec_device, int32_t* c_out) {
    if (!c || !runtimes_sec_device || !c_out) return CUTOFF_ERR_BAD_ARG;
    if (!c->weights_loaded || c->pending) return CUTOFF_ERR_STATE;
    const bool replay = (c->cfg.flags & CUTOFF_FLAG_GRAPH) && c->decided_once &&
                        c->pushes + 1 >= static_cast<uint32_t>(c->W);
    if (!replay) {
        const int rc = cutoff_push(c, runtimes_sec_device, 1, nullptr);
        if (rc < 0) return rc;
        return cutoff_predict(c, c_out);
    }
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    if (!c->graph_dev_exec) {
        CU_CHECK(c, cudaStreamSynchronize(c->stream));
        const int rc = build_graph(c, false);
        if (rc) return rc;
    }
    refresh_projections(c);
    CU_CHECK(c, cudaMemcpyAsync(c->d_stage, runtimes_sec_device, sizeof(float) * c->N, cudaMemcpyDeviceToDevice, c->stream));
    CU_CHECK(c, cudaGraphLaunch(c->graph_dev_exec, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    c->launches += c->graph_kernels;
    if (c->h_state->error_flags & kErrBadValue) {
        // the push kernel left the window untouched, but the decision that followed it ran on the old window and
        // advanced the decision counter: put the counter back, clear the flag, report the bad value
        const uint32_t step_before = c->h_state->step - 1u;
        CU_CHECK(c, cudaMemcpyAsync(&c->d_state->step, &step_before, sizeof(uint32_t), cudaMemcpyHostToDevice, c->stream));
        CU_CHECK(c, cudaMemsetAsync(&c->d_state->error_flags, 0, sizeof(int32_t), c->stream));
        CU_CHECK(c, cudaStreamSynchronize(c->stream));
        c->draws_valid = false;
        return CUTOFF_ERR_BAD_VALUE;
    }
    c->pushes += 1;
    c->draws_valid = c->n_chunks == 1;
    if (c->h_state->error_flags & kErrTimeout) return CUTOFF_ERR_TIMEOUT;
    c->have_result = true;
    *c_out = c->h_state->c_star;
    return c->h_state->code == 2 ? CUTOFF_DEGENERATE : CUTOFF_OK;
}

int cutoff_get_stats(cutoff_ctx* c, float* e_out, float* omega_out) {
    if (!c) return CUTOFF_ERR_BAD_ARG;
    if (!c->have_result) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    if (e_out) CU_CHECK(c, cudaMemcpyAsync(e_out, c->d_E, sizeof(float) * c->N, cudaMemcpyDeviceToHost, c->stream));
    if (omega_out)
        CU_CHECK(c, cudaMemcpyAsync(omega_out, c->d_omega, sizeof(float) * c->N, cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    return CUTOFF_OK;
}

int cutoff_get_order_stat_std(cutoff_ctx* c, float* std_sec) {
    if (!c || !std_sec) return CUTOFF_ERR_BAD_ARG;
    if (!c->have_result || !c->have_std) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaMemcpyAsync(std_sec, c->d_std, sizeof(float) * c->N, cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    return CUTOFF_OK;
}

int cutoff_get_partial_sums(cutoff_ctx* c, double* sums) {
    if (!c || !sums) return CUTOFF_ERR_BAD_ARG;
    if (!c->have_result) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaMemcpyAsync(sums, c->d_sums, sizeof(double) * c->N, cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    return CUTOFF_OK;
}

int cutoff_decide_from_sums(cutoff_ctx* c, const double* sums, int32_t* c_out) {
    if (!c || !sums || !c_out) return CUTOFF_ERR_BAD_ARG;
    if (c->pending) return CUTOFF_ERR_STATE;
    if (c->pushes < static_cast<uint32_t>(c->W)) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaMemcpyAsync(c->d_sums, sums, sizeof(double) * c->N, cudaMemcpyHostToDevice, c->stream));
    const int64_t total = c->cfg.total_samples > 0 ? c->cfg.total_samples : c->S;
    k_decide<<<1, kDecideThreads, 0, c->stream>>>(c->d_sums, c->N, 1.0 / static_cast<double>(total), c->d_state, 0,
                                                  c->d_E, c->d_omega);
    c->launches += 1;
    CU_CHECK(c, cudaMemcpyAsync(c->h_state, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    c->have_result = true;
    *c_out = c->h_state->c_star;
    return c->h_state->code == 2 ? CUTOFF_DEGENERATE : CUTOFF_OK;
}

int cutoff_predict_partial_async(cutoff_ctx* c) {
    if (!c) return CUTOFF_ERR_BAD_ARG;
    if (!c->weights_loaded) return CUTOFF_ERR_STATE;
    if (c->pending || c->partial_pending) return CUTOFF_ERR_STATE;
    if (c->pushes < static_cast<uint32_t>(c->W)) return CUTOFF_WARMUP;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    const int rc = enqueue_decision(c, false);
    if (rc == CUTOFF_OK) c->partial_pending = true;
    return rc;
}

int cutoff_partial_sums_device(cutoff_ctx* c, double** sums_device) {
    if (!c || !sums_device) return CUTOFF_ERR_BAD_ARG;
    *sums_device = c->d_sums;
    return CUTOFF_OK;
}

int cutoff_decide_from_device_sums(cutoff_ctx* c, const double* sums_device, int32_t* c_out) {
    if (!c || !sums_device || !c_out) return CUTOFF_ERR_BAD_ARG;
    if (c->pending) return CUTOFF_ERR_STATE;
    if (c->pushes < static_cast<uint32_t>(c->W)) return CUTOFF_ERR_STATE;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    if (sums_device != c->d_sums)
        CU_CHECK(c, cudaMemcpyAsync(c->d_sums, sums_device, sizeof(double) * c->N, cudaMemcpyDeviceToDevice, c->stream));
    const int64_t total = c->cfg.total_samples > 0 ? c->cfg.total_samples : c->S;
    // the decision counter moves on here if the sums came from cutoff_predict_partial_async (which left it alone)
    k_decide<<<1, kDecideThreads, 0, c->stream>>>(c->d_sums, c->N, 1.0 / static_cast<double>(total), c->d_state,
                                                  c->partial_pending ? 1 : 0, c->d_E, c->d_omega);
    c->launches += 1;
    CU_CHECK(c, cudaMemcpyAsync(c->h_state, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    if (c->h_state->error_flags & kErrBadValue) {
        // a bad asynchronous push came before this decision: as cutoff_fetch reports it
        c->pushes = c->h_state->push_count;
        CU_CHECK(c, cudaMemsetAsync(&c->d_state->error_flags, 0, sizeof(int32_t), c->stream));
        c->partial_pending = false;
        return CUTOFF_ERR_BAD_VALUE;
    }
    if (c->h_state->error_flags & kErrTimeout) return CUTOFF_ERR_TIMEOUT;
    if (c->partial_pending) {
        const int rc = collect_timing(c);
        if (rc) return rc;
        c->partial_pending = false;
        c->decided_once = true;
    }
    c->have_result = true;
    *c_out = c->h_state->c_star;
    return c->h_state->code == 2 ? CUTOFF_DEGENERATE : CUTOFF_OK;
}

int cutoff_measure_pipe_rates(int device, float* rates_out) {
    if (device < 0 || !rates_out) return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    cudaDeviceProp prop;
    CU_CHECK(none, cudaGetDeviceProperties(&prop, device));
    const int sms = prop.multiProcessorCount;
    long long* d_cycles = nullptr;
    float* d_sink = nullptr;
    if (cudaMalloc(&d_cycles, sizeof(long long) * sms) != cudaSuccess || cudaMalloc(&d_sink, sizeof(float)) != cudaSuccess) {
        cudaFree(d_cycles);
        return CUTOFF_ERR_NOMEM;
    }
    std::vector<long long> h(sms);
    int rc = CUTOFF_OK;
    for (int kind = 0; kind < 3 && rc == CUTOFF_OK; ++kind) {
        double best = 0.0;
        for (int rep = 0; rep < 4 && rc == CUTOFF_OK; ++rep) {         // the first repetition warms the clocks up
            if (kind == 0) k_pipe_rate<0><<<sms, kRateThreads>>>(1.25f, d_cycles, d_sink);
            if (kind == 1) k_pipe_rate<1><<<sms, kRateThreads>>>(1.25f, d_cycles, d_sink);
            if (kind == 2) k_pipe_rate<2><<<sms, kRateThreads>>>(1.25f, d_cycles, d_sink);
            if (cudaMemcpy(h.data(), d_cycles, sizeof(long long) * sms, cudaMemcpyDeviceToHost) != cudaSuccess) {
                rc = CUTOFF_ERR_CUDA;
                break;
            }
            long long worst = 1;
            for (long long v : h) worst = v > worst ? v : worst;
            const double warp_instr = static_cast<double>(kRateThreads / 32) * kRateChains * kRateIters;
            const double rate = warp_instr / static_cast<double>(worst);
            if (rep > 0 && rate > best) best = rate;
        }
        rates_out[kind] = static_cast<float>(best);
    }
    cudaFree(d_cycles);
    cudaFree(d_sink);
    return rc;
}

int cutoff_measure_operand_stream(int device, float* gbs_out) {
    if (device < 0 || !gbs_out) return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    cudaDeviceProp prop;
    CU_CHECK(none, cudaGetDeviceProperties(&prop, device));
    const int sms = prop.multiProcessorCount;
    CU_CHECK(none, cudaFuncSetAttribute(k_operand_stream, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(kStreamSmemBytes)));
    constexpr int kCols = 256;
    const int rows_of[2] = {2048, 65536};                // 2 MB that every SM re-reads; 64 MB
    float* d_src = nullptr;
    int* d_err = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaMalloc(&d_src, sizeof(float) * rows_of[1] * kCols) != cudaSuccess) return CUTOFF_ERR_NOMEM;
    int rc = CUTOFF_OK;
    if (cudaMalloc(&d_err, sizeof(int)) != cudaSuccess) rc = CUTOFF_ERR_NOMEM;
    if (rc == CUTOFF_OK && (cudaMemset(d_src, 0, sizeof(float) * rows_of[1] * kCols) != cudaSuccess ||
                            cudaMemset(d_err, 0, sizeof(int)) != cudaSuccess || cudaEventCreate(&e0) != cudaSuccess ||
                            cudaEventCreate(&e1) != cudaSuccess))
        rc = CUTOFF_ERR_CUDA;
    for (int which = 0; which < 2 && rc == CUTOFF_OK; ++which) {
        CUtensorMap map;
        rc = make_tile_map(nullptr, &map, d_src, rows_of[which], kCols);
        if (rc != CUTOFF_OK) break;
        const int iters = static_cast<int>((4096ll << 20) / sms / kStreamStageBytes);    // 4 GB per launch in all
        float best = 0.0f;
        for (int rep = 0; rep < 3; ++rep) {              // the first repetition fills the L2 and warms the clocks up
            cudaEventRecord(e0);
            k_operand_stream<<<sms, 32, kStreamSmemBytes>>>(map, rows_of[which], kCols / 32, iters, d_err);
            cudaEventRecord(e1);
            float ms = 0.0f;
            if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.0f) {
                rc = CUTOFF_ERR_CUDA;
                break;
            }
            const float gbs = static_cast<float>(static_cast<double>(iters) * kStreamStageBytes * sms / (ms * 1e6));
            if (rep > 0 && gbs > best) best = gbs;
        }
        gbs_out[which] = best;
    }
    int h_err = 0;
    if (rc == CUTOFF_OK && cudaMemcpy(&h_err, d_err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) rc = CUTOFF_ERR_CUDA;
    if (rc == CUTOFF_OK && h_err) rc = CUTOFF_ERR_TIMEOUT;
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(d_src);
    cudaFree(d_err);
    return rc;
}

int cutoff_reset(cutoff_ctx* c) {
    if (!c) return CUTOFF_ERR_BAD_ARG;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaMemsetAsync(c->d_state, 0, sizeof(DevState), c->stream));
    CU_CHECK(c, cudaMemsetAsync(c->d_ring, 0, sizeof(float) * c->W * c->N, c->stream));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    c->pushes = 0;
    c->pending = false;
    c->partial_pending = false;
    c->have_result = false;
    c->draws_valid = false;
    c->proj_stale = true;
    return CUTOFF_OK;
}

int cutoff_save_state(cutoff_ctx* c, void* buf, size_t* nbytes) {
    if (!c || !nbytes) return CUTOFF_ERR_BAD_ARG;
    const size_t need = 4 * sizeof(uint32_t) + sizeof(DevState) + sizeof(float) * c->W * c->N;
    if (!buf) { *nbytes = need; return CUTOFF_OK; }
    if (*nbytes < need) return CUTOFF_ERR_BAD_ARG;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    char* p = static_cast<char*>(buf);
    const uint32_t hdr[4] = {0x53465443u /* "CTFS" */, 1u, static_cast<uint32_t>(c->N), static_cast<uint32_t>(c->W)};
    std::memcpy(p, hdr, sizeof(hdr));
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    CU_CHECK(c, cudaMemcpy(p + sizeof(hdr), c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost));
    CU_CHECK(c, cudaMemcpy(p + sizeof(hdr) + sizeof(DevState), c->d_ring, sizeof(float) * c->W * c->N,
                           cudaMemcpyDeviceToHost));
    *nbytes = need;
    return CUTOFF_OK;
}

int cutoff_restore_state(cutoff_ctx* c, const void* buf, size_t nbytes) {
    if (!c || !buf) return CUTOFF_ERR_BAD_ARG;
    const size_t need = 4 * sizeof(uint32_t) + sizeof(DevState) + sizeof(float) * c->W * c->N;
    if (nbytes != need) return CUTOFF_ERR_BAD_ARG;
    const char* p = static_cast<const char*>(buf);
    uint32_t hdr[4];
    std::memcpy(hdr, p, sizeof(hdr));
    if (hdr[0] != 0x53465443u || hdr[1] != 1u || hdr[2] != static_cast<uint32_t>(c->N) ||
        hdr[3] != static_cast<uint32_t>(c->W))
        return CUTOFF_ERR_BAD_ARG;
    DevState s;
    std::memcpy(&s, p + sizeof(hdr), sizeof(s));
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    CU_CHECK(c, cudaMemcpy(c->d_state, &s, sizeof(DevState), cudaMemcpyHostToDevice));
    CU_CHECK(c, cudaMemcpy(c->d_ring, p + sizeof(hdr) + sizeof(DevState), sizeof(float) * c->W * c->N,
                           cudaMemcpyHostToDevice));
    c->pushes = s.push_count;
    c->pending = false;
    c->partial_pending = false;
    c->have_result = false;
    c->draws_valid = false;            // the retained draws belong to a decision on the state that was replaced
    c->proj_stale = true;
    return CUTOFF_OK;
}

int cutoff_set_timing(cutoff_ctx* c, int on) {
    if (!c) return CUTOFF_ERR_BAD_ARG;
    if (on && (c->cfg.flags & CUTOFF_FLAG_GRAPH)) return CUTOFF_ERR_UNSUPPORTED;
    c->timing = on != 0;
    return CUTOFF_OK;
}

int cutoff_get_timing(cutoff_ctx* c, float* ms, int cap) {
    if (!c || !ms || cap < 0) return CUTOFF_ERR_BAD_ARG;
    for (int i = 0; i < kNumStages && i < cap; ++i) ms[i] = c->stage_ms[i];
    return kNumStages;
}

int64_t cutoff_launch_count(cutoff_ctx* c) { return c ? c->launches : 0; }

int cutoff_set_option(cutoff_ctx* c, const char* name, int64_t value) {
    if (!c || !name) return CUTOFF_ERR_BAD_ARG;
    if (c->pending) return CUTOFF_ERR_STATE;
    if (std::strcmp(name, "order_stat_std") == 0) {
        if (value != 0 && value != 1) return CUTOFF_ERR_BAD_ARG;
        if (value && c->cfg.total_samples > 0 && c->cfg.total_samples != c->S) return CUTOFF_ERR_UNSUPPORTED;
        if (c->graph_exec || c->graph_dev_exec) return CUTOFF_ERR_STATE;   // the captured graph has the other sort kernel in it
        c->want_std = value != 0;
        return CUTOFF_OK;
    }
    if (std::strcmp(name, "pair_emission") == 0) {
        if (value != 0 && value != 1) return CUTOFF_ERR_BAD_ARG;
        if (value && (c->literal || !c->use_tc || c->pair_clusters == 0)) return CUTOFF_ERR_UNSUPPORTED;
        if (c->graph_exec || c->graph_dev_exec) return CUTOFF_ERR_STATE;   // the captured graph has the other kernel in it
        c->pair_emission = value != 0;
        return CUTOFF_OK;
    }
    if (std::strcmp(name, "pass_rows") == 0) {
        if (value < 1024 || value > 0x7fffffffll) return CUTOFF_ERR_BAD_ARG;
        if (c->graph_exec || c->graph_dev_exec) return CUTOFF_ERR_STATE;   // the captured graph replays the old split
        plan_chunks(c, static_cast<int>(value));
        c->draws_valid = false;
        return CUTOFF_OK;
    }
    return CUTOFF_ERR_BAD_ARG;
}

// ---- test hooks --------------------------------------------------------------------------------

namespace {
__global__ void k_debug_normals(uint32_t seed_lo, uint32_t seed_hi, uint32_t step, uint32_t stream, uint32_t k0,
                                int64_t count, int nq, int n_elems, float* __restrict__ normals,
                                uint32_t* __restrict__ words) {
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= count * nq) return;
    const int64_t k = idx / nq;
    const int q = static_cast<int>(idx % nq);
    const Philox4 r = philox4x32_10(q, k0 + static_cast<uint32_t>(k), stream, step, seed_lo, seed_hi);
    if (words) {
        uint32_t* w = words + idx * 4;
        w[0] = r.x; w[1] = r.y; w[2] = r.z; w[3] = r.w;
    }
    if (normals) {
        float e[4];
        box_muller(r.x, r.y, e[0], e[1]);
        box_muller(r.z, r.w, e[2], e[3]);
        for (int c = 0; c < 4; ++c)
            if (4 * q + c < n_elems) normals[k * n_elems + 4 * q + c] = e[c];
    }
}
}  // namespace

int cutoff_debug_normals(int device, uint64_t seed, uint32_t step, uint32_t stream, int64_t k0, int64_t count,
                         int32_t n_elems, float* normals_out, uint32_t* words_out) {
    if (device < 0 || k0 < 0 || count < 1 || n_elems < 1 || k0 + count > (1ll << 32)) return CUTOFF_ERR_BAD_ARG;
    if (!normals_out && !words_out) return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    const int nq = (n_elems + 3) / 4;
    float* d_n = nullptr;
    uint32_t* d_w = nullptr;
    int rc = CUTOFF_OK;
    if (normals_out && cudaMalloc(&d_n, sizeof(float) * count * n_elems) != cudaSuccess) rc = CUTOFF_ERR_NOMEM;
    if (!rc && words_out && cudaMalloc(&d_w, sizeof(uint32_t) * count * nq * 4) != cudaSuccess) rc = CUTOFF_ERR_NOMEM;
    if (!rc) {
        const int64_t threads = count * nq;
        k_debug_normals<<<static_cast<unsigned>(ceil_div64(threads, 256)), 256>>>(
            static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32), step, stream, static_cast<uint32_t>(k0),
            count, nq, n_elems, d_n, d_w);
        if (cudaDeviceSynchronize() != cudaSuccess) rc = CUTOFF_ERR_CUDA;
    }
    if (!rc && normals_out &&
        cudaMemcpy(normals_out, d_n, sizeof(float) * count * n_elems, cudaMemcpyDeviceToHost) != cudaSuccess)
        rc = CUTOFF_ERR_CUDA;
    if (!rc && words_out &&
        cudaMemcpy(words_out, d_w, sizeof(uint32_t) * count * nq * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        rc = CUTOFF_ERR_CUDA;
    cudaFree(d_n);
    cudaFree(d_w);
    return rc;
}

int cutoff_debug_samples(cutoff_ctx* c, int64_t k0, int64_t count, float* x_out) {
    if (!c || !x_out || k0 < 0 || count < 1 || k0 + count > c->S) return CUTOFF_ERR_BAD_ARG;
    if (!c->weights_loaded || c->pending) return CUTOFF_ERR_STATE;
    if (c->pushes < static_cast<uint32_t>(c->W)) return CUTOFF_WARMUP;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    c->draws_valid = false;                                 // the sample matrix is about to be overwritten
    launch_encoder(c);
    for (int64_t done = 0; done < count; done += c->chunk_rows) {
        const int n = static_cast<int>(count - done < c->chunk_rows ? count - done : c->chunk_rows);
        const uint32_t base = static_cast<uint32_t>(c->cfg.sample_offset + k0 + done);
        launch_chain(c, base, n);
        launch_emission(c, base, n);
        CU_CHECK(c, cudaMemcpy2DAsync(x_out + done * c->N, sizeof(float) * c->N, c->d_x, sizeof(float) * c->ldx,
                                      sizeof(float) * c->N, n, cudaMemcpyDeviceToHost, c->stream));
        CU_CHECK(c, cudaStreamSynchronize(c->stream));
    }
    CU_CHECK(c, cudaGetLastError());
    return CUTOFF_OK;
}

int cutoff_debug_window(cutoff_ctx* c, float* window_out) {
    if (!c || !window_out) return CUTOFF_ERR_BAD_ARG;
    if (c->pending) return CUTOFF_ERR_STATE;
    if (c->pushes < static_cast<uint32_t>(c->W)) return CUTOFF_WARMUP;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    CU_CHECK(c, cudaStreamSynchronize(c->stream));
    for (int t = 0; t < c->W; ++t) {                       // position t (0 = oldest) sits in slot (pushes + t) mod W
        const size_t slot = (static_cast<size_t>(c->pushes) + t) % c->W;
        CU_CHECK(c, cudaMemcpy(window_out + static_cast<size_t>(t) * c->N, c->d_ring + slot * c->N, sizeof(float) * c->N,
                               cudaMemcpyDeviceToHost));
    }
    return CUTOFF_OK;
}

int cutoff_debug_sort(cutoff_ctx* c, const float* rows, int64_t n_rows, int32_t n, float* keys_out, int32_t* perm_out) {
    if (!c || !rows || !keys_out || !perm_out || n_rows < 1 || n < 1 || n > 4096 || n_rows > (1 << 24))
        return CUTOFF_ERR_BAD_ARG;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    const size_t elems = static_cast<size_t>(n_rows) * n;
    float *d_rows = nullptr, *d_keys = nullptr;
    int* d_perm = nullptr;
    int rc = CUTOFF_OK;
    if (cudaMalloc(&d_rows, elems * 4) != cudaSuccess || cudaMalloc(&d_keys, elems * 4) != cudaSuccess ||
        cudaMalloc(&d_perm, elems * 4) != cudaSuccess)
        rc = CUTOFF_ERR_NOMEM;
    if (!rc && cudaMemcpyAsync(d_rows, rows, elems * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
        rc = CUTOFF_ERR_CUDA;
    if (!rc) {
        const int P = next_pow2(n) < 32 ? 32 : next_pow2(n);
        const int rows_i = static_cast<int>(n_rows);
        const int grid_w = ceil_div(rows_i, kSortWarps) < 4 * c->sm_count ? ceil_div(rows_i, kSortWarps) : 4 * c->sm_count;
        const int grid_c = rows_i < 4 * c->sm_count ? rows_i : 4 * c->sm_count;
        switch (P) {
            case 32: k_debug_sort_warp<1><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            case 64: k_debug_sort_warp<2><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            case 128: k_debug_sort_warp<4><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            case 256: k_debug_sort_warp<8><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            case 512: k_debug_sort_warp<16><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            case 1024: k_debug_sort_warp<32><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            case 2048: k_debug_sort_cta<2><<<grid_c, 64, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm); break;
            default: k_debug_sort_cta<4><<<grid_c, 128, 0, c->stream>>>(d_rows, n, rows_i, d_keys, d_perm);
        }
        c->launches += 1;
        if (cudaMemcpyAsync(keys_out, d_keys, elems * 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
            cudaMemcpyAsync(perm_out, d_perm, elems * 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
            cudaStreamSynchronize(c->stream) != cudaSuccess)
            rc = CUTOFF_ERR_CUDA;
    }
    if (rc == CUTOFF_ERR_CUDA) c->last_error = cudaGetErrorString(cudaGetLastError());
    cudaFree(d_rows); cudaFree(d_keys); cudaFree(d_perm);
    return rc;
}

int cutoff_debug_sort_values(cutoff_ctx* c, const float* rows, int64_t n_rows, int32_t n, float* keys_out) {
    if (!c || !rows || !keys_out || n_rows < 1 || n < 1 || n > 4096 || n_rows > (1 << 24)) return CUTOFF_ERR_BAD_ARG;
    DeviceGuard guard(c->cfg.device);
    CU_CHECK(c, guard.err);
    const size_t elems = static_cast<size_t>(n_rows) * n;
    float *d_rows = nullptr, *d_keys = nullptr;
    int rc = CUTOFF_OK;
    if (cudaMalloc(&d_rows, elems * 4) != cudaSuccess || cudaMalloc(&d_keys, elems * 4) != cudaSuccess) rc = CUTOFF_ERR_NOMEM;
    if (!rc && cudaMemcpyAsync(d_rows, rows, elems * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) rc = CUTOFF_ERR_CUDA;
    if (!rc) {
        const int P = next_pow2(n) < 32 ? 32 : next_pow2(n);
        const int rows_i = static_cast<int>(n_rows);
        const int grid_w = ceil_div(rows_i, kSortWarps) < 4 * c->sm_count ? ceil_div(rows_i, kSortWarps) : 4 * c->sm_count;
        const int grid_c = rows_i < 4 * c->sm_count ? rows_i : 4 * c->sm_count;
        switch (P) {
            case 32: k_debug_sort_values_warp<1><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            case 64: k_debug_sort_values_warp<2><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            case 128: k_debug_sort_values_warp<4><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            case 256: k_debug_sort_values_warp<8><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            case 512: k_debug_sort_values_warp<16><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            case 1024: k_debug_sort_values_warp<32><<<grid_w, kSortWarps * 32, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            case 2048: k_debug_sort_values_cta<2><<<grid_c, 64, 0, c->stream>>>(d_rows, n, rows_i, d_keys); break;
            default: k_debug_sort_values_cta<4><<<grid_c, 128, 0, c->stream>>>(d_rows, n, rows_i, d_keys);
        }
        c->launches += 1;
        if (cudaMemcpyAsync(keys_out, d_keys, elems * 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
            cudaStreamSynchronize(c->stream) != cudaSuccess)
            rc = CUTOFF_ERR_CUDA;
    }
    if (rc == CUTOFF_ERR_CUDA) c->last_error = cudaGetErrorString(cudaGetLastError());
    cudaFree(d_rows); cudaFree(d_keys);
    return rc;
}

// ---- evaluation of cutoff rules on recorded run-times ------------------------------------------------------

int cutoff_eval_trace(int device, const float* trace, int64_t n_steps, int32_t n, int32_t ld, const int32_t* cutoffs,
                      int32_t n_rules, int32_t* best_c, float* best, float* all, float* achieved, float* step_time,
                      int32_t* static_c, void* stream) {
    if (device < 0 || !trace || n_steps < 1 || n_steps > (1ll << 31) - 1 || n < 1 || n > 4096 || ld < n || n_rules < 0 ||
        !best_c || !best || !all || (n_rules > 0 && (!cutoffs || !achieved || !step_time)))
        return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaDeviceProp prop;
    CU_CHECK(none, cudaGetDeviceProperties(&prop, device));
    float* d_sorted = nullptr;         // the sorted rows, kept only when the static cutoff is asked for
    double* d_total = nullptr;
    if (static_c) {
        if (cudaMalloc(&d_sorted, sizeof(float) * static_cast<size_t>(n_steps) * n) != cudaSuccess) return CUTOFF_ERR_NOMEM;
        if (cudaMalloc(&d_total, sizeof(double)) != cudaSuccess) { cudaFree(d_sorted); return CUTOFF_ERR_NOMEM; }
    }
    const int P = next_pow2(n) < 32 ? 32 : next_pow2(n);
    const int cap = 8 * prop.multiProcessorCount;
    const int64_t want_w = ceil_div64(n_steps, kSortWarps);
    const int grid_w = static_cast<int>(want_w < cap ? want_w : cap);
    const int grid_c = static_cast<int>(n_steps < cap ? n_steps : cap);
#define EVAL_ARGS trace, n_steps, n, ld, cutoffs, n_rules, best_c, best, all, achieved, step_time, d_sorted
    switch (P) {
        case 32: k_eval_trace_warp<1><<<grid_w, kSortWarps * 32, 0, s>>>(EVAL_ARGS); break;
        case 64: k_eval_trace_warp<2><<<grid_w, kSortWarps * 32, 0, s>>>(EVAL_ARGS); break;
        case 128: k_eval_trace_warp<4><<<grid_w, kSortWarps * 32, 0, s>>>(EVAL_ARGS); break;
        case 256: k_eval_trace_warp<8><<<grid_w, kSortWarps * 32, 0, s>>>(EVAL_ARGS); break;
        case 512: k_eval_trace_warp<16><<<grid_w, kSortWarps * 32, 0, s>>>(EVAL_ARGS); break;
        case 1024: k_eval_trace_warp<32><<<grid_w, kSortWarps * 32, 0, s>>>(EVAL_ARGS); break;
        case 2048: k_eval_trace_cta<2><<<grid_c, 64, 0, s>>>(EVAL_ARGS); break;
        default: k_eval_trace_cta<4><<<grid_c, 128, 0, s>>>(EVAL_ARGS); break;
    }
#undef EVAL_ARGS
    if (static_c) k_best_static<<<1, kStaticThreads, 0, s>>>(d_sorted, n_steps, n, static_c, d_total);
    const cudaError_t err = cudaStreamSynchronize(s);
    cudaFree(d_sorted);
    cudaFree(d_total);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? CUTOFF_OK : CUTOFF_ERR_CUDA;
}

int cutoff_order_baseline(int device, const float* trace, int64_t n_steps, int32_t n, int32_t ld, int32_t* cutoffs_out,
                          void* stream) {
    if (device < 0 || !trace || n_steps < 1 || n_steps > (1ll << 31) - 1 || n < 1 || ld < n || !cutoffs_out)
        return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* d_work = nullptr;          // [T] sums / means, [T] sums of squares / deviations, [n] normal quantiles
    if (cudaMalloc(&d_work, sizeof(double) * (2 * static_cast<size_t>(n_steps) + n)) != cudaSuccess) return CUTOFF_ERR_NOMEM;
    double* d1 = d_work;
    double* d2 = d_work + n_steps;
    double* dq = d_work + 2 * n_steps;
    k_step_moments<<<static_cast<unsigned>(n_steps), kMomentThreads, 0, s>>>(trace, n_steps, n, ld, d1, d2);
    k_running_moments<<<1, 32, 0, s>>>(n_steps, n, d1, d2);
    k_elfving_quantiles<<<ceil_div(n, 256), 256, 0, s>>>(n, dq);
    k_order_cutoffs<<<static_cast<unsigned>(ceil_div64(n_steps, 8)), 256, 0, s>>>(n_steps, n, d1, d2, dq, cutoffs_out);
    const cudaError_t err = cudaStreamSynchronize(s);
    cudaFree(d_work);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? CUTOFF_OK : CUTOFF_ERR_CUDA;
}

// ---- learning the model: ELBO, gradient, Adam -------------------------------------------------------------------

int64_t cutoff_fit_param_count(int32_t n_workers, int32_t latent_dim, int32_t hidden) {
    if (n_workers < 1 || latent_dim < 1 || hidden < 1) return 0;
    return fit::layout(n_workers, latent_dim, hidden).off[fit::kTensors];
}

int64_t cutoff_fit_workspace_bytes(int32_t n_workers, int32_t latent_dim, int32_t hidden, int32_t lag, int32_t batch) {
    if (n_workers < 1 || latent_dim < 1 || hidden < 1 || lag < 0 || batch < 1) return 0;
    return static_cast<int64_t>(sizeof(float)) * fit::workspace_floats(n_workers, latent_dim, hidden, lag + 1, batch);
}

int cutoff_elbo_grad(int device, int32_t n_workers, int32_t latent_dim, int32_t hidden, int32_t lag, int32_t batch,
                     const float* params, const float* xhat, const float* eps, float* elbo, float* grads, void* workspace,
                     size_t workspace_bytes, void* stream) {
    if (device < 0 || n_workers < 1 || n_workers > 4096 || latent_dim < 1 || latent_dim > 64 || hidden < 1 || hidden > 1024 ||
        lag < 0 || lag > 255 || batch < 1 || batch > 65535 || !params || !xhat || !eps || !elbo || !workspace)
        return CUTOFF_ERR_BAD_ARG;
    if (workspace_bytes < static_cast<size_t>(cutoff_fit_workspace_bytes(n_workers, latent_dim, hidden, lag, batch)))
        return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    fit::elbo_grad(n_workers, latent_dim, hidden, lag + 1, batch, params, xhat, eps, elbo, grads,
                   static_cast<float*>(workspace), static_cast<cudaStream_t>(stream));
    return cudaGetLastError() == cudaSuccess ? CUTOFF_OK : CUTOFF_ERR_CUDA;
}

int cutoff_adam_step(int device, int64_t n, float* params, const float* grads, float* m, float* v, int32_t t, float lr,
                     float beta1, float beta2, float eps, float clip_norm, float grad_scale, float* norm_out, void* workspace,
                     size_t workspace_bytes, void* stream) {
    constexpr int kParts = 256;
    if (device < 0 || n < 1 || !params || !grads || !m || !v || t < 1 || !(lr > 0.f) || !(beta1 >= 0.f && beta1 < 1.f) ||
        !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f) || !(clip_norm > 0.f) || !norm_out || !workspace ||
        workspace_bytes < kParts * sizeof(double))
        return CUTOFF_ERR_BAD_ARG;
    cutoff_ctx* none = nullptr;
    DeviceGuard guard(device);
    CU_CHECK(none, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* partial = static_cast<double*>(workspace);
    const int64_t want = (n + fit::kNormThreads - 1) / fit::kNormThreads;
    const int parts = static_cast<int>(want < kParts ? want : kParts);
    fit::k_sumsq_partial<<<parts, fit::kNormThreads, 0, s>>>(grads, n, grad_scale, partial);
    fit::k_norm_finish<<<1, 32, 0, s>>>(partial, parts, norm_out);
    const float corr1 = 1.f - std::pow(beta1, static_cast<float>(t)), corr2 = 1.f - std::pow(beta2, static_cast<float>(t));
    fit::k_adam<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(params, grads, m, v, n, grad_scale, norm_out, clip_norm, lr,
                                                                      beta1, beta2, eps, corr1, corr2);
    return cudaGetLastError() == cudaSuccess ? CUTOFF_OK : CUTOFF_ERR_CUDA;
}

}  // extern "C"

// ---- allocation-free entry point -------------------------------------------------------------

namespace {
constexpr int kStaticParts = 256;     // partial rows (= most CTAs the sort kernel may use here)
constexpr int kStaticRowsPerWarp = 64;                                                  // rows a warp adds in fp32
constexpr int64_t kStaticBlockRows = static_cast<int64_t>(kStaticParts) * kSortWarps * kStaticRowsPerWarp;   // 131072
static_assert(kStaticParts * CUTOFF_STATIC_MAX_N * sizeof(float) == CUTOFF_STATIC_SCRATCH_BYTES, "scratch size");

// Scratch of cutoff_sorted_row_sums_static: one partial sum row per CTA.  Lives in the library
// image, one copy per GPU.  In host code this name is only a handle for cudaGetSymbolAddress;
// the kernels get the device address found at set-up.
static __device__ __align__(256) float g_static_partial[kStaticParts * CUTOFF_STATIC_MAX_N];

constexpr int kMaxDevices = 64;
float* g_static_partial_addr[kMaxDevices] = {};   // device address per GPU, filled on first use

template <int E>
void launch_static_sort(const float* x, int ldx, int n, int n_rows, int grid, float* partial, cudaStream_t stream) {
    k_sort_sum_warp<E><<<grid, kSortWarps * 32, 0, stream>>>(x, ldx, n, n_rows, partial);
}
}  // namespace

extern "C" int cutoff_sorted_row_sums_static(int device, const float* x, int64_t n_rows, int32_t n, int32_t ldx,
                                             double* sums, void* stream) {
    if (device < 0 || device >= kMaxDevices || !x || !sums || n_rows < 1 || n_rows > CUTOFF_STATIC_MAX_ROWS || n < 1 ||
        ldx < n)
        return CUTOFF_ERR_BAD_ARG;
    if (n > CUTOFF_STATIC_MAX_N) return CUTOFF_ERR_TOO_LARGE;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return CUTOFF_ERR_CUDA;
    if (!g_static_partial_addr[device]) {
        // once per device, with that device current: translate the symbol into a device address
        float* addr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_static_partial) != cudaSuccess || !addr)
            return CUTOFF_ERR_CUDA;
        g_static_partial_addr[device] = addr;
    }
    float* partial = g_static_partial_addr[device];
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int P = next_pow2(n) < 32 ? 32 : next_pow2(n);
    // The rows go through in blocks of kStaticBlockRows: within a block a warp adds at most kStaticRowsPerWarp
    // sorted rows in fp32, then the block's partial rows are added to `sums` in double.  The blocks run one after
    // the other on the stream, so they can share the scratch array.
    for (int64_t r0 = 0; r0 < n_rows; r0 += kStaticBlockRows) {
        const int rows = static_cast<int>(n_rows - r0 < kStaticBlockRows ? n_rows - r0 : kStaticBlockRows);
        const int want = ceil_div(rows, kSortWarps);
        const int grid = want < kStaticParts ? want : kStaticParts;
        const float* xb = x + static_cast<size_t>(r0) * ldx;
        // every CTA of the grid writes its whole partial row (zeros if it had no sample), and the
        // column sum reads exactly `grid` rows: stale contents of the shared array are never read
        switch (P) {
            case 32: launch_static_sort<1>(xb, ldx, n, rows, grid, partial, s); break;
            case 64: launch_static_sort<2>(xb, ldx, n, rows, grid, partial, s); break;
            case 128: launch_static_sort<4>(xb, ldx, n, rows, grid, partial, s); break;
            case 256: launch_static_sort<8>(xb, ldx, n, rows, grid, partial, s); break;
            case 512: launch_static_sort<16>(xb, ldx, n, rows, grid, partial, s); break;
            default: launch_static_sort<32>(xb, ldx, n, rows, grid, partial, s); break;
        }
        k_colsum<<<ceil_div(n, 256), 256, 0, s>>>(partial, grid, n, sums, r0 > 0 ? 1 : 0);
    }
    return cudaGetLastError() == cudaSuccess ? CUTOFF_OK : CUTOFF_ERR_CUDA;
}
