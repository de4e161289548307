/*
 * cutoff.h -- C ABI of the run-time cutoff decision of Cutoff SGD
 * (Teng & Wood, "High Throughput Synchronous Distributed Stochastic Gradient
 * Descent", 2018) for one NVIDIA B200 (sm_100a).
 *
 * The parameter server of Algorithm 1 calls, once per SGD step,
 *      c <- predict_cutoff(q_phi, obs)
 * and then adds the run-times r_w that arrive to obs.  This library is that
 * call: cutoff_predict() is predict_cutoff, cutoff_push() is "obs <- obs U r_w"
 * for one whole step, cutoff_load_weights() supplies q_phi and p_theta.
 *
 * What one decision computes (all of it in CUDA kernels of this library):
 *   1. the last lag+1 pushed vectors, divided by twice the mean of the first
 *      lag+1 pushed vectors (Section 3.1.3, last paragraph);
 *   2. the guide q_phi of Section 3.1.3: forward and backward ReLU RNNs over
 *      that window, then for each of S samples the chain z_t = mu + sigma*eps
 *      with h_out = (tanh-layer(z_{t-1}) + h_left + h_right)/3;
 *   3. for each sample the transition z_{T+1} ~ N(G(z_T), H(z_T)) and the
 *      emission x_{T+1} ~ N(I(z_{T+1}), J(z_{T+1})) (Section 3.1.3 and the
 *      K-sample form of the posterior predictive after Eq. 4);
 *   4. each sample's N run-times sorted ascending, the sorted vectors
 *      averaged over the samples (Section 3.1.1, last paragraph);
 *   5. Omega(c) = c / E[x~_(c)] and c* = argmax_c Omega(c) (Section 3).
 *
 * Model variants: by default transition and emission are one-hidden-layer ReLU
 * MLPs whose heads give a mean and a log-variance; with CUTOFF_FLAG_LITERAL they
 * are the gated transition and the emission networks I, J as Section 3.1.3 prints
 * them.  All noise comes from Philox4x32-10
 * (Salmon et al., SC'11) and the basic Box-Muller transform, addressed by
 * (seed, decision number, stage, sample, element), so results do not depend on
 * how the work is split over threads or GPUs.
 *
 * Conventions
 *   - Every function returns 0 (CUTOFF_OK), a positive informational code, or
 *     a negative error code.  On a negative return no output is written.
 *   - "host" / "device" beside a pointer says where the memory must live.
 *     Caller pointers are borrowed for the duration of the call only.
 *   - A context owns all device memory it allocates and is bound to one
 *     device and one stream.  It is not thread-safe.
 *   - Every entry point makes the context's device current while it runs and
 *     puts the caller's current device back before it returns.
 *   - Nothing here throws, aborts or calls exit().
 */
#ifndef CUTOFF_H_
#define CUTOFF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cutoff_ctx cutoff_ctx;

enum {
    CUTOFF_OK = 0,
    CUTOFF_WARMUP = 1,          /* fewer than lag+1 vectors pushed: c = N (wait for everyone)      */
    CUTOFF_DEGENERATE = 2,      /* no c has a positive expected time: c = N                        */
    CUTOFF_ERR_BAD_ARG = -1,
    CUTOFF_ERR_BAD_BLOB = -2,
    CUTOFF_ERR_BAD_VALUE = -3,  /* a pushed run-time is not finite or not > 0                      */
    CUTOFF_ERR_CUDA = -4,       /* a CUDA call failed; see cutoff_last_error()                     */
    CUTOFF_ERR_UNSUPPORTED = -5,
    CUTOFF_ERR_NOMEM = -6,
    CUTOFF_ERR_STATE = -7,      /* call order: weights not loaded, nothing predicted yet, ...      */
    CUTOFF_ERR_TIMEOUT = -8,    /* a bounded device-side wait gave up (tensor-core pipeline)        */
    CUTOFF_ERR_TOO_LARGE = -9   /* the request exceeds a fixed built-in capacity                    */
};

enum {
    CUTOFF_PRECISION_FP32 = 0,  /* every product in fp32 FMA                                       */
    CUTOFF_PRECISION_TF32 = 1,  /* emission output layer on tensor cores, operands rounded to tf32 */
    CUTOFF_PRECISION_BF16W = 2  /* as TF32, with the output-layer weights first rounded to bf16    */
};

enum {
    CUTOFF_FLAG_GRAPH = 1,      /* replay push+predict as one captured CUDA graph                  */
    CUTOFF_FLAG_LITERAL = 2     /* the generative model exactly as Section 3.1.3 prints it (gated
                                   transition, emission I / J); see cutoff_load_weights            */
};

typedef struct {
    int32_t n_workers;          /* N >= 1                                                          */
    int32_t latent_dim;         /* D in {4, 8, 16, 32}                                             */
    int32_t hidden;             /* H, a multiple of D (and so of 4)                                */
    int32_t lag;                /* the paper's l >= 0; the window holds l+1 vectors                */
    int32_t n_samples;          /* S: samples this context draws per decision (the paper's K)      */
    int32_t precision;          /* CUTOFF_PRECISION_*                                              */
    int32_t device;             /* CUDA device ordinal                                             */
    int32_t flags;              /* CUTOFF_FLAG_*                                                   */
    int64_t sample_offset;      /* index of this context's first sample in the global draw         */
    int64_t total_samples;      /* samples of the whole decision (0 means n_samples); used only to
                                   normalise when several contexts share one decision              */
    void*   stream;             /* cudaStream_t the kernels run on; NULL = the default stream (with
                                   CUTOFF_FLAG_GRAPH: a stream the context creates, because the
                                   default stream cannot be captured)                              */
    uint64_t seed;              /* Philox key                                                      */
} cutoff_config;

/* Create a context: validates cfg, allocates all device memory on cfg->device, and tells that device
 * which of the library's kernels need large shared memory (so contexts on several GPUs can live in one process).
 * out (host) receives the handle.  Errors: BAD_ARG, UNSUPPORTED, NOMEM, CUDA. */
int cutoff_create(cutoff_ctx** out, const cutoff_config* cfg);

/* Release everything the context owns.  NULL is allowed. */
void cutoff_destroy(cutoff_ctx* ctx);

/* Load theta and phi.  blob (host): little-endian header of six uint32
 *   { 0x31465443 ("CTF1"), 1, N, D, H, 0 }
 * followed by fp32 tensors, row-major [outputs x inputs], in this order:
 *   Wxf[HxN] Whf[HxH] bf[H] a0[H]  Wxb[HxN] Whb[HxH] bb[H] b0[H]      (h_left / h_right RNNs)
 *   Wz[HxD] bz[H] Wmu[DxH] bmu[D] Wsig[DxD] bsig[D] z0[D]             (combiner, mu_q, sigma_q)
 *   W1[HxD] b1[H] W2[2DxH] b2[2D]                                     (transition; rows D.. = log-variance)
 *   W3[HxD] b3[H] W4[2NxH] b4[2N]                                     (emission;   rows N.. = log-variance)
 * A context created with CUTOFF_FLAG_LITERAL takes the networks as Section 3.1.3 prints them instead:
 * the header's last word is 1, the guide tensors (first two lines above) are the same, and then follow
 *   Wg1[HxD] bg1[H] Wg2[DxH] bg2[D]     gate      g = MLP_2(z, ReLU, Sigmoid)
 *   Wh1[HxD] bh1[H] Wh2[DxH] bh2[D]     proposal  h = MLP_2(z, ReLU, Identity)
 *   Wl[DxD] bl[D]                       G = (1 - g) * (Wl z + bl) + g * h
 *   Ws[DxD] bs[D]                       H = Softplus(Ws ReLU(G) + bs)            z' = G + H * eps
 *   Wi1[HxD] bi1[H] Wi2[NxH] bi2[N]     I = Wi2 (Wi1 z' + bi1) + bi2             (two affine layers)
 *   Wj1[HxN] bj1[H] Wj2[NxH] bj2[N]     J = Softplus(Wj2 ReLU(Wj1 I + bj1) + bj2)   x = I + J * eps
 * where H and J are standard deviations.  With a tensor-core precision the three products over N
 * (Wi2, Wj1, Wj2) run on the tensor cores with tf32 operands (weights first rounded to bf16 for BF16W).
 * The blob is copied; the caller keeps ownership.  Errors: BAD_ARG, BAD_BLOB (size, magic or
 * dimensions do not match the context, or a value is not finite), CUDA. */
int cutoff_load_weights(cutoff_ctx* ctx, const void* blob, size_t nbytes);

/* Append one step's observed run-times ("obs <- obs U r_w", Algorithm 1).
 * runtimes_sec: N floats, seconds, each finite and > 0; host memory if on_device == 0, device
 * memory on the context's device otherwise (then the check runs on the GPU and a bad value is
 * reported by this call after a stream synchronisation).
 * censored: NULL, or N bytes in the same memory space as runtimes_sec; a non-zero byte marks a worker
 * that was killed at the cutoff, whose run-time is therefore unknown and whose entry of runtimes_sec
 * is ignored (Section 4.2).  Each such worker gets a draw from its own predictive distribution of this
 * step, left-truncated at the largest observed run-time: the first of the S predictive draws of the
 * last decision that exceeds it, scanning cyclically from a pseudo-random start; the threshold itself
 * if none does.  Needs a completed decision since the last push (STATE otherwise), made in a single
 * pass by a context that draws all samples of the decision (UNSUPPORTED otherwise), and at least one
 * worker that finished.  Each decision's draws serve one censored push.
 * The first lag+1 pushes fix the normaliser.  Errors: BAD_ARG, BAD_VALUE, STATE, UNSUPPORTED, CUDA. */
int cutoff_push(cutoff_ctx* ctx, const float* runtimes_sec, int on_device, const uint8_t* censored);

/* As cutoff_push with a device pointer, but only enqueues: no synchronisation, no error report
 * for bad values until the next cutoff_fetch / cutoff_predict (which then returns BAD_VALUE). */
int cutoff_push_async(cutoff_ctx* ctx, const float* runtimes_sec_device);

/* One decision.  c_out (host) receives c* in 1..N.  Blocks until the result is on the host.
 * Returns OK, WARMUP (c = N, nothing computed), DEGENERATE (c = N), or an error.
 * Advances the decision counter that addresses the noise. */
int cutoff_predict(cutoff_ctx* ctx, int32_t* c_out);

/* The same decision split in two: enqueue all kernels on the stream without waiting, then wait
 * and read the result.  cutoff_fetch returns what cutoff_predict would have returned. */
int cutoff_predict_async(cutoff_ctx* ctx);
int cutoff_fetch(cutoff_ctx* ctx, int32_t* c_out);

/* One iteration of the parameter server's loop in a single call: append this step's run-times
 * (host, N floats, as for cutoff_push) and return the cutoff for the next step (as cutoff_predict).
 * With CUTOFF_FLAG_GRAPH the copy, the push and all kernels of the decision are captured into a
 * CUDA graph the first time the window is full and a decision has already run; later calls
 * replay it (no argument changes between replays: window position, normaliser and decision
 * counter live in device memory).  Without the flag it is cutoff_push followed by cutoff_predict.
 * Returns what cutoff_predict returns.  Errors: BAD_ARG, BAD_VALUE, STATE, CUDA, TIMEOUT. */
int cutoff_step(cutoff_ctx* ctx, const float* runtimes_sec, int32_t* c_out);

/* The same with the run-times already on the context's device (N floats): with CUTOFF_FLAG_GRAPH one
 * device-to-device copy into the library's landing buffer, then a replay of the captured push + decision.
 * The values are checked on the GPU: a value that is not finite or not > 0 leaves the window and the
 * decision counter as they were and returns BAD_VALUE after the replay.
 * Errors: BAD_ARG, BAD_VALUE, STATE, CUDA, TIMEOUT. */
int cutoff_step_device(cutoff_ctx* ctx, const float* runtimes_sec_device, int32_t* c_out);

/* Results of the last completed decision.  Either pointer may be NULL.
 * exp_order_stats_sec (host, N floats): E[x~_(j)] in seconds, ascending.
 * omega_per_sec (host, N floats): Omega(c) = c / E[x~_(c)]; -inf where E <= 0.
 * Errors: STATE if no decision has completed, CUDA. */
int cutoff_get_stats(cutoff_ctx* ctx, float* exp_order_stats_sec, float* omega_per_sec);

/* Spread of each order statistic over the samples of the last decision: the standard deviation of
 * x~_(j), in seconds (std_sec, host, N floats) -- the +-2 sigma bands the paper draws around the predicted
 * order statistics (Fig. 3).  Computed only by decisions made after
 * cutoff_set_option(ctx, "order_stat_std", 1) (the sort then also accumulates squares); STATE otherwise. */
int cutoff_get_order_stat_std(cutoff_ctx* ctx, float* std_sec);

/* Sum over this context's samples of the sorted, normalised run-times of the last decision
 * (host, N doubles): the quantity several contexts add up when they share one decision.
 * cutoff_decide_from_sums then finishes a decision from such a total: sums (host, N doubles)
 * over total_samples samples -> c_out, and the stats returned by cutoff_get_stats. */
int cutoff_get_partial_sums(cutoff_ctx* ctx, double* sums);
int cutoff_decide_from_sums(cutoff_ctx* ctx, const double* sums, int32_t* c_out);

/* The same exchange with nothing passing through the host, for several contexts (one per GPU) that share a
 * decision (the K samples of the predictive approximation after Eq. 4 are independent, so they split):
 *   cutoff_predict_partial_async   enqueue this context's part of the decision up to the per-position sums of its
 *                                  sorted samples and return at once; no argmax, the decision counter stays.
 *                                  Returns OK, or WARMUP (fewer than lag+1 vectors: nothing enqueued, c = N).
 *   cutoff_partial_sums_device     *sums_device = the context's own N doubles (device memory; valid until
 *                                  cutoff_destroy) that hold those sums once the enqueued work is done.  They may
 *                                  be all-reduced in place by work enqueued on the context's stream.
 *   cutoff_decide_from_device_sums finish the decision from sums over all total_samples samples
 *                                  (sums_device: device, N doubles; may be the context's own array), advance
 *                                  the decision counter if the sums came from cutoff_predict_partial_async,
 *                                  wait, and return what cutoff_predict returns.
 * Errors: BAD_ARG, STATE (weights missing, a decision already in flight, too few observations), BAD_VALUE (an
 * asynchronous push before it carried a bad value), CUDA, TIMEOUT. */
int cutoff_predict_partial_async(cutoff_ctx* ctx);
int cutoff_partial_sums_device(cutoff_ctx* ctx, double** sums_device);
int cutoff_decide_from_device_sums(cutoff_ctx* ctx, const double* sums_device, int32_t* c_out);

/* Forget all observations and restart the decision counter. */
int cutoff_reset(cutoff_ctx* ctx);

/* Observation state (window, normaliser, counters) as an opaque byte string.
 * save: if buf is NULL, *nbytes receives the size needed; else *nbytes is the capacity on entry
 * and the size written on exit.  restore: the string must come from a context with the same N
 * and lag.  Errors: BAD_ARG, CUDA. */
int cutoff_save_state(cutoff_ctx* ctx, void* buf, size_t* nbytes);
int cutoff_restore_state(cutoff_ctx* ctx, const void* buf, size_t nbytes);

/* Text for a return code; the last CUDA error text of a context. Never NULL. */
const char* cutoff_strerror(int code);
const char* cutoff_last_error(cutoff_ctx* ctx);

/* ---- measurement hooks ---------------------------------------------------------------------
 * With timing on, every stage of a decision is bracketed by CUDA events on the context's stream
 * (not available together with CUTOFF_FLAG_GRAPH).  cutoff_get_timing writes up to cap stage
 * times of the last fetched decision in milliseconds and returns the number of stages;
 * cutoff_stage_name names stage i.  cutoff_launch_count returns the number of kernels this
 * context has launched since it was created. */
int cutoff_set_timing(cutoff_ctx* ctx, int on);
/* cutoff_measure_pipe_rates: the issue rates that bound the sort (Section 3.1.1, last paragraph) and the
 * per-sample chain on this device, measured by a short micro-benchmark (about 10 ms): rates_out (host,
 * 3 floats) = warp-instructions per clock per SM of fp32 min/max, of warp shuffles and of fp32 fused
 * multiply-adds, each from 32 warps per SM running independent chains.  Allocates and frees a few KB of
 * device memory, synchronises the device.  Errors: BAD_ARG, NOMEM, CUDA. */
int cutoff_measure_pipe_rates(int device, float* rates_out);

/* cutoff_measure_operand_stream: the rate, in GB/s over the whole device, at which all SMs together can bring
 * operand tiles from L2 into shared memory with the copies the emission output layer (Section 3.1.3,
 * x ~ N(I(z), J(z))) issues: per K block three tensor-map boxes of 128 rows x 128 bytes into a ring of four
 * stages, one CTA per SM, nothing consuming the data.  gbs_out (host, 2 floats): [0] from a 2 MB matrix that
 * every SM re-reads (the weights' case), [1] from a 64 MB matrix (the hidden vectors' case).  A micro-benchmark
 * of about 1 ms per case; the paper has no counterpart.  Allocates and frees 64 MB of device memory,
 * synchronises the device.  Errors: BAD_ARG, NOMEM, CUDA, TIMEOUT (a copy did not land within its bounded wait). */
int cutoff_measure_operand_stream(int device, float* gbs_out);
int cutoff_get_timing(cutoff_ctx* ctx, float* ms, int cap);
const char* cutoff_stage_name(int i);
int64_t cutoff_launch_count(cutoff_ctx* ctx);

/* Options, by name.  "pass_rows": samples that go through sampling and sorting per pass (>= 1024;
 * clipped to S and to the allocated pass buffers).  "order_stat_std": 1 = also compute the spread
 * of each order statistic (see cutoff_get_order_stat_std), 0 = do not (default); not available to a
 * context that holds only part of a decision's samples (UNSUPPORTED), nor once a graph has been
 * captured (STATE).  "pair_emission": 1 = run the emission output layer (Section 3.1.3, x ~ N(I(z), J(z))) with
 * tensor-core instructions that span two SMs, so that each SM loads only half of every weight tile (compact variant
 * on a tensor-core precision only: UNSUPPORTED otherwise; same results as 0, the default, which is the faster one
 * as measured); not once a graph has been captured (STATE).  Errors: BAD_ARG, STATE, UNSUPPORTED. */
int cutoff_set_option(cutoff_ctx* ctx, const char* name, int64_t value);

/* ---- test hooks ----------------------------------------------------------------------------
 * cutoff_debug_normals: the noise generator alone.  Writes, for samples k0 .. k0+count-1 and
 * elements 0 .. n_elems-1 of the given (seed, step, stream), the standard normals
 * (normals_out, host, count*n_elems floats) and the raw Philox words (words_out, host,
 * count*4*ceil(n_elems/4) uint32); either may be NULL.  device selects the GPU.
 *
 * cutoff_debug_samples: the unsorted predictive draws of the coming decision, in normalised
 * units, for local samples k0 .. k0+count-1 (x_out, host, count*N floats).  Does not advance the
 * decision counter.  Returns WARMUP before lag+1 pushes.
 *
 * cutoff_debug_sort: the library's sorting network applied to caller rows.  rows (host,
 * n_rows*n floats) -> keys_out (host, sorted ascending) and perm_out (host, int32, the original
 * position of each sorted key; equal keys keep their original order). */
int cutoff_debug_normals(int device, uint64_t seed, uint32_t step, uint32_t stream, int64_t k0,
                         int64_t count, int32_t n_elems, float* normals_out, uint32_t* words_out);
int cutoff_debug_samples(cutoff_ctx* ctx, int64_t k0, int64_t count, float* x_out);
/* cutoff_debug_window: the observation window as the encoder will see it, oldest vector first, in
 * seconds (window_out, host, (lag+1)*N floats); imputed entries included.  WARMUP before lag+1 pushes. */
int cutoff_debug_window(cutoff_ctx* ctx, float* window_out);
int cutoff_debug_sort(cutoff_ctx* ctx, const float* rows, int64_t n_rows, int32_t n,
                      float* keys_out, int32_t* perm_out);
/* cutoff_debug_sort_values: the same networks in the instantiation the decision itself runs (plain
 * fp32 keys, rows padded with +infinity), the sorted rows returned instead of summed (Section 3.1.1,
 * last paragraph: "sort").  rows (host, n_rows*n floats, any finite values, +-0 and +infinity
 * included) -> keys_out (host, n_rows*n floats, each row ascending).  n <= 4096. */
int cutoff_debug_sort_values(cutoff_ctx* ctx, const float* rows, int64_t n_rows, int32_t n, float* keys_out);

/* ---- evaluation of cutoff rules on recorded run-times --------------------------------------------
 * The quantities of the paper's Fig. 2 (Section 4.1), per SGD step t of a recorded trace of worker run-times:
 * with x~(t) the observed run-times of the step in ascending order (Section 3: Omega(c) = c / x~_(c)),
 *   best[t], best_c[t]   the ground-truth maximum max_c Omega(c) and the cutoff that attains it (largest c on a tie)
 *   all[t]               N / x~_(N): the throughput of waiting for all workers
 *   achieved[m*T + t]    Omega(c) for the cutoff c = cutoffs[m*T + t] that rule m chose for the step (clipped to 1..N)
 *   step_time[m*T + t]   x~_(c): how long the step lasts under that cutoff, in seconds
 *   *static_c            the one cutoff that maximises sum_t c / x~_(c)(t) over the whole trace (a static cutoff,
 *                        as in Chen et al. 2016, cited in Section 1); NULL = not wanted
 * trace: device, n_steps x ld floats, row t = the N run-times of step t (all finite, > 0), n <= 4096, ld >= n.
 * cutoffs: device, n_rules x n_steps int32 (NULL if n_rules = 0).  All outputs are device arrays of n_steps
 * (best_c int32; best, all float), n_rules*n_steps (achieved, step_time) or one element (static_c).
 * The call waits for its kernels.  Errors: BAD_ARG, NOMEM, CUDA.
 *
 * cutoff_order_baseline: the "order" rule of Fig. 4.  For step t > 0 the expected order statistics of n iid
 * normal run-times by Elfving's formula (Section 3.1.1, in its standard form
 * mu + sigma * Phi^-1((j - pi/8) / (n - pi/4 + 1))), with mu and sigma the mean and (population) deviation of
 * every run-time of steps 0 .. t-1, and cutoffs_out[t] = argmax_c c / E[x~_(c)] over positive expectations (largest
 * c on a tie, n if none); cutoffs_out[0] = n.  cutoffs_out: device, n_steps int32.  Waits.  Errors as above. */
int cutoff_eval_trace(int device, const float* trace, int64_t n_steps, int32_t n, int32_t ld, const int32_t* cutoffs,
                      int32_t n_rules, int32_t* best_c, float* best, float* all, float* achieved, float* step_time,
                      int32_t* static_c, void* stream);
int cutoff_order_baseline(int device, const float* trace, int64_t n_steps, int32_t n, int32_t ld, int32_t* cutoffs_out,
                          void* stream);

/* ---- learning the model -----------------------------------------------------------------------------
 * Section 3.1.3 fits the generative model p_theta and the guide q_phi together by stochastic gradient ascent on
 *     ELBO = E_q [ log p_theta(x_{T-l:T}, z_{T-l:T}) - log q_phi(z_{T-l:T} | x_{T-l:T}) ],
 * Section 4.1 names the optimiser: Adam with gradient clipping.  These calls are one training step's arithmetic for
 * the compact networks, in fp32, on device buffers of the caller (the noise is an input: draw it as you like).
 *
 * The parameter vector is the tensors of the weight blob, in its order (Wxf Whf bf a0 Wxb Whb bb b0 Wz bz Wmu bmu
 * Wsig bsig z0 W1 b1 W2 b2 W3 b3 W4 b4), back to back without the header: cutoff_fit_param_count floats.
 *
 * cutoff_elbo_grad: the one-sample reparameterised ELBO of each of `batch` windows -- z_t = mu_t + sigma_t eps_t,
 * sum over the window's steps of log p(x_t | z_t) + log p(z_t | z_{t-1}) - log q(z_t | ...) with the densities of the
 * mean / log-variance heads and the guide of Section 3.1.3; the latent before the window is z0, the RNNs start from
 * a0 and b0 -- and the gradient of their SUM with respect to every parameter.
 *   params  device, cutoff_fit_param_count floats
 *   xhat    device, batch x (lag+1) x n_workers floats: normalised run-times (divided by twice the mean of the first
 *           window, Section 3.1.3 last paragraph), oldest vector of a window first
 *   eps     device, batch x (lag+1) x latent_dim floats: the standard-normal draws of the guide
 *   elbo    device, batch floats, overwritten
 *   grads   device, cutoff_fit_param_count floats, overwritten; NULL = forward pass only
 *   workspace  device, at least cutoff_fit_workspace_bytes(...) bytes, contents undefined afterwards
 * Only enqueues work on `stream`.  Every reduction runs in a fixed order: results are reproducible bit for bit.
 *
 * cutoff_adam_step: g = grad_scale * grads (e.g. -1/batch to minimise the negative mean ELBO); if ||g|| over all n
 * entries exceeds clip_norm, g is scaled by clip_norm / ||g||; then Adam's step number t (1, 2, ...):
 * m = beta1 m + (1-beta1) g, v = beta2 v + (1-beta2) g^2, params -= lr (m / (1-beta1^t)) / (sqrt(v / (1-beta2^t)) + eps).
 * params, m, v: device, n floats, updated in place (m and v start at zero); norm_out: device, one float, receives ||g||
 * before clipping; workspace: device, at least 2048 bytes.  Only enqueues.  Errors of both: BAD_ARG, CUDA. */
int64_t cutoff_fit_param_count(int32_t n_workers, int32_t latent_dim, int32_t hidden);
int64_t cutoff_fit_workspace_bytes(int32_t n_workers, int32_t latent_dim, int32_t hidden, int32_t lag, int32_t batch);
int cutoff_elbo_grad(int device, int32_t n_workers, int32_t latent_dim, int32_t hidden, int32_t lag, int32_t batch,
                     const float* params, const float* xhat, const float* eps, float* elbo, float* grads, void* workspace,
                     size_t workspace_bytes, void* stream);
int cutoff_adam_step(int device, int64_t n, float* params, const float* grads, float* m, float* v, int32_t t, float lr,
                     float beta1, float beta2, float eps, float clip_norm, float grad_scale, float* norm_out, void* workspace,
                     size_t workspace_bytes, void* stream);

/* ---- allocation-free entry point ---------------------------------------------------------------
 * The paper has no counterpart for this call.  It serves programs that may not allocate device
 * memory at the time they need order statistics: a server that handed all of the GPU's memory to
 * its own pool at start-up (a late cudaMalloc there fails or fragments the pool), a control loop
 * that cannot afford the device-wide synchronisation an allocation may imply, or code under a
 * "nothing is allocated after initialisation" rule.  Such a caller already holds its predictive
 * samples and only wants them sorted and summed.
 *
 * cutoff_sorted_row_sums_static sorts the first n entries of each of n_rows rows ascending and adds
 * the sorted rows position by position:   sums[j] = sum over rows of (j-th smallest entry of the row).
 * Dividing by n_rows gives the Monte-Carlo expected order statistics of Section 3.1.1.
 *   device    CUDA device ordinal (0..63) that owns x, sums and stream
 *   x         device, n_rows x ldx floats, row-major; entries beyond n in a row are ignored
 *   n_rows    1 .. CUTOFF_STATIC_MAX_ROWS;   n  1 .. CUTOFF_STATIC_MAX_N;   ldx >= n
 *   sums      device, n doubles, overwritten
 * Accuracy: the rows go through in blocks of 131072; inside a block a warp adds at most 64 sorted rows in
 * single precision, everything above that is added in double, so the error of a sum does not grow with
 * n_rows beyond that of 64 single-precision additions (about 4e-6 relative to the largest partial sum).
 *   stream    cudaStream_t to run on (NULL = default stream); the call only enqueues work
 * The call performs no cudaMalloc, cudaFree or other allocating routine.  Its only scratch is a
 * fixed array of CUTOFF_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that
 * loads the library holds that much memory until the process exits.  n above the limit returns
 * CUTOFF_ERR_TOO_LARGE and does nothing; n_rows above CUTOFF_STATIC_MAX_ROWS returns BAD_ARG.
 * The first call on a device looks up the array's device address (a one-time set-up step that
 * loads the library's code on that device); make that first call before starting any stream
 * capture.  All calls on a device share the one array, and it keeps what the last call left in
 * it: each call overwrites every scratch row it later reads, so nothing needs clearing, but two
 * calls whose work overlaps on the GPU (different streams, or different host threads) race on it.
 * Issue them on one stream, or order them with events.  Not thread-safe with respect to its
 * first call on a device.  Errors: BAD_ARG, TOO_LARGE, CUDA. */
#define CUTOFF_STATIC_MAX_N 1024
#define CUTOFF_STATIC_MAX_ROWS (1 << 24)
#define CUTOFF_STATIC_SCRATCH_BYTES (256 * 1024 * 4)
int cutoff_sorted_row_sums_static(int device, const float* x, int64_t n_rows, int32_t n, int32_t ldx,
                                  double* sums, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CUTOFF_H_ */
