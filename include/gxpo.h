/*
 * gxpo.h -- C ABI of the GXPO active-phase parameter update for NVIDIA B200 (sm_100a).
 *
 * GXPO (Gradient Extrapolation-Based Policy Optimization) replaces one optimizer
 * step of a GRPO trainer by: two fast probe optimizer steps, a per-coordinate
 * geometric extrapolation of the observed two-step displacement to a virtual
 * K-step point, a partial move towards it, one corrective optimizer step with the
 * gradient taken at the repositioned point, and a rolling z-score gate on the norm
 * of that gradient which permanently falls back to the single-pass step
 * (Algorithm 1 of the paper).  This library is the parameter-space part of that
 * step.  The three backward passes stay with the caller: gradients come in as
 * device buffers.
 *
 * Conventions
 *   - Every pointer inside gxpo_tensor is a DEVICE pointer owned by the caller; the
 *     library never allocates, frees or keeps parameter memory.  Pointers passed to
 *     the *_host entry points are HOST pointers (see there).
 *   - theta, work, m, v are float32.  Gradients are float32 or bfloat16, one dtype
 *     per context.  Arithmetic is float32; the norm is accumulated in float64.
 *   - Every call returns a gxpo_status; nothing throws, aborts or traps.  The text
 *     of the last failure is available from gxpo_last_error().
 *   - Sweeps are asynchronous on the cudaStream_t passed as `stream` (void*, may be
 *     NULL for the legacy default stream).  Only gxpo_gate_update and
 *     gxpo_state_export wait for the device.
 *   - Vector (128/256-bit) access is used for a tensor when all of its bound
 *     pointers are 32-byte aligned; otherwise that tensor takes a slower scalar
 *     path with identical results.  Any n >= 0 is accepted; n == 0 is a no-op.
 *   - The calls of one context share its small device scratch (partial sums, counters):
 *     issue them on one stream, or order the streams yourself, so that no two of its
 *     kernels run at the same time.
 *   - A context is not thread-safe; use one per host thread or lock around it.
 *   - One GPU per context: the device current at gxpo_create.
 */
#ifndef GXPO_H
#define GXPO_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gxpo_ctx gxpo_ctx; /* opaque, library-owned */

typedef enum {
    GXPO_OK = 0,
    GXPO_ERR_INVALID_ARG = 1, /* null pointer, negative size, K < 2, alpha outside [0,1], ... */
    GXPO_ERR_ALIGNMENT = 2,   /* a pointer is not aligned to its element size */
    GXPO_ERR_STATE = 3,       /* call out of order for Algorithm 1, or nothing bound */
    GXPO_ERR_CUDA = 4,        /* a CUDA runtime call failed; see gxpo_last_error */
    GXPO_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (only the shared-memory
                                 staged sweeps wait on anything; the register-staged kernels
                                 and all reductions are wait-free).  An active step reports it
                                 from the gate update that ends the step; a fallback step, which
                                 has no gate update, from the next gxpo_probe_step /
                                 gxpo_probe_step_deferred / gxpo_gate_peek / gxpo_gate_last /
                                 gxpo_state_export on the context, once */
    GXPO_ERR_NONFINITE = 6    /* ||g_slow|| was not finite; the gate was tripped */
} gxpo_status;

enum { GXPO_OPT_GD = 0, GXPO_OPT_ADAMW = 1 };  /* base optimizer, "OptimStep" in Algorithm 1 */
enum { GXPO_F32 = 0, GXPO_BF16 = 1 };          /* gradient dtype */

/* Where the intermediate points live (the paper is silent; both keep theta^t alive
 * until the extrapolation, as Algorithm 1 needs):
 *   PINGPONG : probe 0 writes theta^{t,1} into `work`, probe 1 updates `work` in
 *              place, extrapolate writes theta-tilde into `theta`, the slow step
 *              updates `theta` in place.  The caller's backward pass 2 reads `work`,
 *              backward pass 3 reads `theta`.  26+26+16+26 bytes per parameter.
 *   SNAPSHOT : probe 0 copies theta^t into `work` and writes theta^{t,1} into
 *              `theta`; every later point is written into `theta`, so a model that
 *              aliases `theta` never has to be re-pointed.  30+26+16+26 bytes. */
enum { GXPO_PLACE_PINGPONG = 0, GXPO_PLACE_SNAPSHOT = 1 };

/* Base optimizer.  GD: theta <- theta - lr g (the paper's surrogate, Sec. 2.1).
 * AdamW (the paper's experiments; decoupled decay, bias-corrected, constant lr):
 *   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
 *   theta <- theta (1 - lr wd) - lr (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps).
 * The step count t advances on EVERY optimizer step, probes included (Sec. 2.3). */
typedef struct {
    int kind; /* GXPO_OPT_GD or GXPO_OPT_ADAMW */
    /* Doubles, as trainers hold them: the float32 constants the kernels use (beta,
     * 1-beta, 1-lr*wd, lr/(1-beta1^t), 1/sqrt(1-beta2^t)) are each formed in double
     * and rounded once, so beta2 = 0.999 gives 1-beta2 = float(0.001), not
     * 1 - float(0.999). */
    double lr, beta1, beta2, eps, weight_decay;
} gxpo_opt_cfg;

/* Hyper-parameters of Algorithm 1 ("Require" line) and of the adaptive rule.
 *   K >= 2 virtual depth, alpha in [0,1] move fraction, delta >= 0 active-set
 *   threshold (|g0_i| > delta, strict).  den_eps: 0 = the literal scale factor of
 *   Eq. (scale_factor); > 0 = coordinates with |1 + r_i| <= den_eps keep scale 1.
 *   tau, gate_eps, window: Eq. (z_score).  min_history: the z-score is evaluated
 *   once the buffer holds at least this many norms (Algorithm 1: 2).  std_ddof: 0
 *   population, 1 sample standard deviation. */
typedef struct {
    int K;
    float alpha, delta, den_eps;
    double tau, gate_eps;
    int window, min_history, std_ddof;
    int placement; /* GXPO_PLACE_* */
} gxpo_cfg;

/* One parameter tensor.  `work` has the same length as `theta`; it may be NULL when the
 * caller only ever takes steps that keep no point there (see gxpo_bind_model_weights:
 * bfloat16-only probe points; fallback steps), and calls that need it then return
 * GXPO_ERR_STATE.  m and v may be NULL for GXPO_OPT_GD.  g0/g1/g_slow are read-only inputs of the context's
 * gradient dtype; g_slow may alias g0 or g1 (both are dead once gxpo_extrapolate
 * has run).  No other buffers may overlap. */
typedef struct {
    float* theta;
    float* work;
    float* m;
    float* v;
    const void* g0;
    const void* g1;
    const void* g_slow;
    long long n;
} gxpo_tensor;

/* What the gate saw at the end of an active step (Eq. (z_score)). z, mu, sigma are
 * NaN while the buffer is still warming up. */
typedef struct {
    int active;        /* 1 if the NEXT step is still an active step (t < s_star) */
    int tripped;       /* 1 if this update set s_star */
    long long t;       /* index of the next training step */
    long long s_star;  /* first fallback step, -1 while unset */
    double norm, z, mu, sigma;
} gxpo_gate_result;

/* Fill cfg/opt with the values the paper's experiments state (K=5, alpha=0.5,
 * delta=1e-8, tau=0.5, lr=1e-7) and this library's documented choices for what the
 * paper leaves open (AdamW betas 0.9/0.999, eps 1e-8, weight decay 0.01; window 20,
 * gate_eps 1e-8, min_history 2, population std, den_eps 0, PINGPONG). */
void gxpo_default_cfg(gxpo_cfg* cfg, gxpo_opt_cfg* opt);

/* Create a context on the current device.  Allocates a few KB of device scratch
 * (partial sums, gate ring buffer) and one pinned result slot.
 * Errors: INVALID_ARG for bad hyper-parameters, CUDA if allocation fails. */
gxpo_status gxpo_create(const gxpo_cfg* cfg, const gxpo_opt_cfg* opt, int grad_dtype,
                        gxpo_ctx** out);
void gxpo_destroy(gxpo_ctx* ctx);

/* Bind a tensor list (count == 1 is the flat-buffer case).  Copies the descriptors
 * and builds the chunk table on the device; the list itself is not kept.  May be
 * called again between steps to re-bind.  Before it overwrites an earlier table it waits
 * for this context's own outstanding work (the last gate update, the last fallback
 * sweep) and for nothing else: other streams of the process keep running, and no device
 * memory is freed or allocated unless the new list needs a larger table than any before.
 * Errors: INVALID_ARG (null list entry fields, n < 0, count < 0, m/v missing for
 * AdamW), ALIGNMENT (pointer not aligned to its element size), STATE (mid-step). */
gxpo_status gxpo_bind(gxpo_ctx* ctx, const gxpo_tensor* list, int count);

/* Optional bfloat16 copies of the live parameters, for trainers whose model runs its
 * forward and backward passes on bfloat16 weights while this library keeps the float32
 * masters (the paper trains in bf16).  weights_bf16[i] is a DEVICE buffer of the i-th
 * bound tensor's length (or NULL for none); count must equal the bound count.  Every
 * sweep that produces a point a backward pass is taken at -- the first probe step
 * (theta^{t,1}), the extrapolation (theta-tilde), the slow step and the fallback step
 * (theta^{t+1}) -- then also stores that point rounded to nearest-even bfloat16, which
 * saves the caller a separate cast sweep (read 4 + write 2 bytes per parameter) before
 * each backward pass.  The second probe step's point is never needed and not stored.
 * bf16_only says which float32 points are NOT stored beside their copies:
 *   GXPO_BF16_BESIDE            every point is stored in float32 and as a copy.
 *   GXPO_BF16_ONLY_THETA1       gxpo_probe_step_deferred writes ONLY the bfloat16 copy of
 *                               theta^{t,1} (gxpo_probe_extrapolate recomputes the float32
 *                               value anyway); `work` is left untouched.
 *   GXPO_BF16_ONLY_PROBE_POINTS in addition gxpo_probe_extrapolate writes ONLY the bfloat16
 *                               copy of theta-tilde: theta^t stays in `theta`, m and v stay as
 *                               they were, and gxpo_slow_step redoes both probe steps and the
 *                               extrapolation in registers (the same functions on the same
 *                               bits, hence the float32 theta-tilde whose rounding the third
 *                               backward pass saw) before its own step.  16 + 18 + 32 = 66
 *                               bytes per parameter including the three copies, and `work`
 *                               is never touched: tensors may be bound with work == NULL,
 *                               20 instead of 24 bytes per parameter resident.  The step must
 *                               then be gxpo_probe_step_deferred, gxpo_probe_extrapolate,
 *                               gxpo_slow_step under gxpo_set_gradients_persist(ctx, 1), with
 *                               AdamW, diagnostics off and g_slow in a buffer of its own;
 *                               anything else returns GXPO_ERR_STATE before the step starts.
 * Both ONLY modes need PINGPONG placement and a buffer for every non-empty tensor.
 * Results (theta, m, v, the copies) are bit-identical across the three modes.
 * Pass weights_bf16 = NULL to unbind.  gxpo_bind drops the binding.  Only legal between
 * steps; waits for this context's own outstanding work, like gxpo_bind. */
enum { GXPO_BF16_BESIDE = 0, GXPO_BF16_ONLY_THETA1 = 1, GXPO_BF16_ONLY_PROBE_POINTS = 2 };
gxpo_status gxpo_bind_model_weights(gxpo_ctx* ctx, void* const* weights_bf16, int count,
                                    int bf16_only);

/* Algorithm 1, "first/second fast optimizer step" (which = 0, 1) and the fallback
 * phase's single step (which = -1).
 *   which =  0: theta^{t,1} <- OptimStep(theta^t, g0)      state: IDLE   -> PROBED0
 *               illegal once the gate has tripped (t >= s_star).
 *   which =  1: theta^{t,2} <- OptimStep(theta^{t,1}, g1)  state: PROBED0 -> PROBED1
 *   which = -1: theta^{t+1} <- OptimStep(theta^t, g0) in place in `theta`, the
 *               single-pass step Algorithm 1 takes when t >= s_star; legal between
 *               steps at any time (a caller may also warm up with it); advances t.
 * Errors: STATE when called out of order or in the wrong phase. */
gxpo_status gxpo_probe_step(gxpo_ctx* ctx, int which, void* stream);

/* Algorithm 1, active set through reposition (Eqs. (retention), (scale_factor),
 * (k_step_position), (blend_step)): per coordinate
 *   scale = S_K(r)/S_2(r) with r = g1/g0 if |g0| > delta, else 1
 *   theta-tilde = theta^t + alpha (theta^{t,2} - theta^t) scale      -> `theta`
 * state: PROBED1 -> EXTRAPOLATED. */
gxpo_status gxpo_extrapolate(gxpo_ctx* ctx, void* stream);

/* gxpo_probe_step(ctx, 1) and gxpo_extrapolate in ONE sweep: Algorithm 1 takes no
 * backward pass at theta^{t,2}, so that point never has to reach memory.  Same
 * per-coordinate arithmetic, bit-identical theta-tilde, m and v; 32 instead of
 * 26 + 16 bytes per parameter.  state: PROBED0 (or PROBED0_DEFERRED, see
 * gxpo_probe_step_deferred) -> EXTRAPOLATED. */
gxpo_status gxpo_probe_extrapolate(gxpo_ctx* ctx, void* stream);

/* The first fast step for callers that will take the second one with
 * gxpo_probe_extrapolate: theta^{t,1} is written exactly as by gxpo_probe_step(ctx, 0)
 * (the caller's second backward pass needs it), but m and v are NOT written; they stay
 * at their start-of-step values until gxpo_probe_extrapolate replays this step in
 * registers (same function, same bits, hence the same theta^{t,1}), takes the second
 * step and writes m and v once.  Results are bit-identical to the other call sequences;
 * the active step moves 18 + 28 + 26 = 72 instead of 26 + 32 + 26 = 84 bytes per
 * parameter.  The optimizer step count advances as usual.  Until gxpo_probe_extrapolate
 * has run, m and v in memory are one step behind and g0 must stay intact.
 * state: IDLE -> PROBED0_DEFERRED; from there only gxpo_probe_extrapolate is legal. */
gxpo_status gxpo_probe_step_deferred(gxpo_ctx* ctx, void* stream);

/* A promise about the caller's gradient buffers, off by default: on != 0 says that g0 and
 * g1 still hold this step's gradients while gxpo_slow_step's sweep runs (nothing reuses
 * them between the backward passes, and g_slow has a buffer of its own), and that device
 * scalars given to gxpo_set_grad_scale for them keep their values until then as well.  After
 * gxpo_probe_step_deferred, gxpo_probe_extrapolate may then leave m and v unwritten once
 * more, and the slow step's sweep replays both probe steps' moment updates in registers from
 * g0 and g1 before it takes its own step: 18 + 20 + 30 = 68 instead of 72 bytes per
 * parameter, bit-identical theta, m and v.  The library uses this where it pays (AdamW on
 * lists of at least 8 chunks of 32768 parameters per SM, with diagnostics off and
 * gxpo_tune's variant 0 or 3) and never when some tensor's g_slow pointer equals its g0 or
 * g1 pointer; elsewhere the promise changes nothing.  Between gxpo_probe_extrapolate and
 * gxpo_slow_step m and v in memory are then two steps behind; a caller who breaks the
 * promise gets wrong moments, not an error.
 * Paper: no counterpart (Algorithm 1 does not say where the optimizer state lives between
 * its three steps).  Errors: STATE mid-step. */
gxpo_status gxpo_set_gradients_persist(gxpo_ctx* ctx, int on);

/* Algorithm 1, "slow correction": theta^{t+1} <- OptimStep(theta-tilde, g_slow), in
 * place in `theta`, and sum(g_slow^2) accumulated in the same sweep (float64,
 * deterministic for a fixed launch shape).  state: EXTRAPOLATED -> SLOW_DONE. */
gxpo_status gxpo_slow_step(gxpo_ctx* ctx, void* stream);

/* Adaptive rule (Eq. (z_score); Algorithm 1 after the slow correction), evaluated
 * by a device kernel: ||g_slow||, mu and sigma of the stored norms, Z, Z >= tau =>
 * s_star = t + 1; the norm is pushed either way; t advances.  Waits for `stream`
 * (the kernel writes its 72-byte record straight into pinned host memory, which the host
 * polls: no copy and no event in between).  `out` may be NULL.  state: SLOW_DONE -> IDLE.
 * Returns NONFINITE (after completing the update and tripping the gate) when the
 * norm is Inf/NaN -- that rule is this library's, not the paper's. */
gxpo_status gxpo_gate_update(gxpo_ctx* ctx, void* stream, gxpo_gate_result* out);

/* The same update without the wait: the gate kernel (which delivers its record itself) is only
 * enqueued on `stream`, and the call returns at once, so the host can go on issuing work
 * (the next rollouts, the next backward pass) while the step drains.  The outcome is
 * collected by whichever call needs it first: gxpo_gate_last, gxpo_gate_peek, the next
 * gxpo_probe_step(ctx, 0) / gxpo_probe_step_deferred (they must know whether the gate
 * has tripped), gxpo_backward_passes, gxpo_state_export -- each waits for the record
 * if it is still in flight.  state: SLOW_DONE -> IDLE. */
gxpo_status gxpo_gate_update_async(gxpo_ctx* ctx, void* stream);

/* Outcome of the most recent gate update (waits for it if it is still in flight).
 * Returns NONFINITE, like gxpo_gate_update, when that update saw a non-finite norm;
 * STATE when no update has run yet.  `out` may be NULL. */
gxpo_status gxpo_gate_last(gxpo_ctx* ctx, gxpo_gate_result* out);

/* Sharded parameter sets (one process per GPU, each holding a slice of every
 * tensor or a subset of the list): the only cross-shard quantity of the whole
 * update is sum(g_slow^2).  Point the context at a caller-owned DEVICE double;
 * gxpo_slow_step then writes this shard's sum there and gxpo_gate_update reads
 * the norm from it, so the caller can sum it across ranks in between (one 8-byte
 * all-reduce on the same stream).  NULL restores the internal scalar.  With the
 * same reduced value on every rank the gates flip together. */
gxpo_status gxpo_set_sumsq_buffer(gxpo_ctx* ctx, double* sumsq_dev);

/* Gradient scaling and global-norm clipping (the paper's training recipe clips at 1.0;
 * it is the trainer's step, not part of Algorithm 1).  A scale is a DEVICE float that
 * every sweep multiplies into gradient `which` (0 = g0, 1 = g1, 2 = g_slow) as it loads
 * it: the optimizer steps and the retention ratio see the scaled gradient, while
 * ||g_slow|| for the gate is taken of the gradient as given.  NULL = no scaling.
 * Only legal between steps. */
gxpo_status gxpo_set_grad_scale(gxpo_ctx* ctx, int which, const float* scale_dev);

/* Clip gradient `which` by its global norm over the bound list: one pass over that
 * gradient computes ||g||, a device-side step turns it into min(1, max_norm / (||g|| + 1e-6))
 * (the usual trainers' convention), and the sweeps of THIS training step scale the
 * gradient by it as they load it -- the gradient buffer itself is not rewritten, so
 * clipping costs one read of g instead of a read plus a read-modify-write.  Call it
 * right before the sweep that consumes the gradient (which = 0 before the first probe
 * or fallback step, 1 before the second probe, 2 before the slow step); the coefficient
 * expires at the end of the step.  Asynchronous on `stream`.
 * Errors: STATE at any other point of the call order, INVALID_ARG for max_norm <= 0. */
gxpo_status gxpo_clip_grad_norm(gxpo_ctx* ctx, int which, double max_norm, void* stream);

/* Per-step diagnostics of the active phase: the quantities the paper's appendix
 * tabulates ("Active-phase GXPO diagnostics").  Off by default.  When on, the sums are
 * gathered inside the extrapolation sweep (gxpo_extrapolate or gxpo_probe_extrapolate) at
 * no extra memory traffic; only <g0, g_slow> needs g0 once more: the slow step's sweep
 * reads it along (+2 bytes per parameter for bfloat16 gradients) where that sweep runs
 * shared-memory staged (AdamW on long lists), otherwise one more pass over the two
 * gradient buffers follows the slow step (+4 bytes per parameter).  It is skipped
 * (cos = NaN) when some tensor's g_slow shares g0's buffer.
 *   g0_norm, g1_norm, gslow_norm : Euclidean norms over all coordinates
 *   cos_g0_gslow                 : <g0, g_slow> / (||g0|| ||g_slow||)
 *   ratio_mean, ratio_std        : mean and population standard deviation of the
 *                                  retention ratio r_i = g1_i / g0_i (Eq. (retention))
 *                                  over the active coordinates
 *   scale_mean                   : mean of scale_i (Eq. (scale_factor)); inactive
 *                                  coordinates count with scale 1
 *   disp_ratio                   : ||theta^{t,K} - theta^t|| / ||theta^{t,2} - theta^t||
 *   inactive_frac                : 1 - |A_t| / n
 * A coordinate whose ratio or scale is not a finite float32 is "irregular": it is
 * counted in n_irregular and left out of the ratio, scale and displacement figures.
 * Accuracy: the counts are exact; the sums are float64 sums of float32 partial sums over
 * 8 consecutive coordinates, so a figure built from non-negative terms (the norms,
 * disp_ratio) is within 3e-7 relative of the exact one, and a term whose square is under
 * float32's normal range (|x| < 1e-19) may be lost; groups whose float32 partial sum
 * would exceed 1e30 are summed in float64 throughout.
 * With a caller-owned sum-of-squares buffer (gxpo_set_sumsq_buffer) gslow_norm and the
 * cosine use whatever that buffer holds; everything else is this context's share. */
typedef struct {
    double g0_norm, g1_norm, gslow_norm, cos_g0_gslow, ratio_mean, ratio_std, scale_mean,
           disp_ratio, inactive_frac;
    long long n, n_active, n_irregular;
} gxpo_diagnostics;

/* Switch the diagnostics on or off; only legal between steps. */
gxpo_status gxpo_enable_diagnostics(gxpo_ctx* ctx, int on);

/* Diagnostics of the last completed active step.  Legal between steps, after an active
 * step that ran with diagnostics on has gone through gxpo_gate_update.  Waits for
 * `stream` (one small read-back).  Errors: STATE otherwise. */
gxpo_status gxpo_get_diagnostics(gxpo_ctx* ctx, void* stream, gxpo_diagnostics* out);

/* Host-side view of the gate; no device work (it only waits if a gxpo_gate_update_async
 * record has not arrived yet). */
gxpo_status gxpo_gate_peek(const gxpo_ctx* ctx, int* active, long long* s_star, long long* t);

/* Optimizer step count so far (3 per active step, 1 per fallback step). */
long long gxpo_optimizer_steps(const gxpo_ctx* ctx);

/* Backward passes spent so far: 3 s + (t - s) with s = min(s_star, t) (Sec. 2.3). */
long long gxpo_backward_passes(const gxpo_ctx* ctx);

/* Checkpointing of the small state (gate ring buffer, t, s_star, optimizer step
 * count).  Call with buf == NULL to get the size in *len.  theta/m/v are the
 * caller's tensors and are checkpointed by the caller.  Only legal between steps. */
gxpo_status gxpo_state_export(gxpo_ctx* ctx, void* buf, size_t* len);
gxpo_status gxpo_state_import(gxpo_ctx* ctx, const void* buf, size_t len);

/* One whole training step of Algorithm 1 for parameters and optimizer state that
 * live in HOST memory (offloaded optimizer state).  All pointers in `list` are HOST
 * pointers (pinned memory makes the copies asynchronous); `work` is ignored.  The
 * three gradients are supplied up front, so this entry point fits callers that
 * replay stored gradients or whose loss has a closed-form gradient; it streams
 * pieces of each tensor through device staging buffers owned by the context
 * (allocated on first use, `staging_elems` parameters per piece), runs the same
 * kernels on them, and writes theta, m, v back.  If the gate is active it runs an
 * active step including gxpo_gate_update, otherwise a fallback step with g0.
 * Does not need gxpo_bind.  Waits for completion. */
gxpo_status gxpo_step_host(gxpo_ctx* ctx, const gxpo_tensor* list, int count,
                           long long staging_elems, void* stream, gxpo_gate_result* out);

/* Launch-shape knobs, for benchmarking: resident CTAs per SM (0 = default), the
 * memory-access variant (0 = default: 256-bit loads; on lists of at least 32 chunks per SM
 * the fused sweep and the AdamW sweeps that write m and v back are fed by a producer thread
 * that stages whole tiles in shared memory with bulk asynchronous copies; 1 = 128-bit
 * loads, register staging everywhere; 2 = 256-bit loads, register staging everywhere;
 * 3 = like 0 for lists of any length) and the
 * number of 2048-element tiles a CTA takes per round-robin turn (0 = default: 16, or
 * 8 / 4 for lists of only a few thousand 32768-element chunks; else 1, 2, 4, 8 or 16).  Element-wise results are identical across all settings; only the
 * summation order of the norm changes. */
gxpo_status gxpo_tune(gxpo_ctx* ctx, int ctas_per_sm, int variant, int unit_tiles);

/* The slow correction for callers that must not allocate.  (The paper has no
 * counterpart to this entry point: it is the same update as gxpo_slow_step, packaged
 * differently.)
 *
 * Who needs it: a trainer that has handed all device memory to its own pool, or that
 * runs with the GPU nearly full (a 7.6e9-parameter list occupies 167 of 180 GB), cannot
 * rely on gxpo_create's cudaMalloc succeeding; code that runs inside another library's
 * callback, or under a policy that forbids allocation after start-up, may not call it at
 * all.  This function needs no context and calls no cudaMalloc, cudaFree or any other
 * allocating routine: its reduction scratch is an array built into the library image
 * (about 512 KB, resident on every GPU that loads the library until the process exits).
 *
 * What it does, for ONE flat buffer of n parameters, in place:
 *     theta <- OptimStep(theta, g_slow)   (m, v updated for AdamW; may be NULL for GD)
 *     *sumsq_dev <- sum(g_slow^2)         (float64; take the square root for the norm)
 * theta, m, v, g_slow and sumsq_dev are DEVICE pointers owned by the caller; g_slow has
 * dtype `grad_dtype`.  `t_opt` is the optimizer's step count INCLUDING this step (the
 * third step of the first active step has t_opt = 3); it only matters for AdamW's bias
 * correction.  The work is enqueued on `stream` and not waited for.
 *
 * Limits and sharing:
 *   - n <= GXPO_NOALLOC_MAX_PARAMS; larger n is rejected with GXPO_ERR_INVALID_ARG and a
 *     message saying so.  Split a larger buffer and add the sums.
 *   - The partial sums are taken per 32768-parameter chunk and added in chunk order, so
 *     the result depends only on the data, not on the launch shape.  It can differ from
 *     gxpo_slow_step's sum in the last bits (different grouping).
 *   - All calls on one GPU share the one scratch array, whatever the stream or thread.
 *     Calls that overlap on the GPU race on it and give wrong sums: order them (same
 *     stream, or events).  Each call resets the part of the scratch that must start at
 *     zero, so the previous call's contents never leak into the next.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress) with that device current; make that first call outside any
 *     stream capture.
 * Errors: a status code as everywhere else; if `errbuf` is not NULL, a description of
 * the failure is written there (at most errbuf_len bytes, NUL-terminated). */
#define GXPO_NOALLOC_MAX_PARAMS 2147483648LL
gxpo_status gxpo_slow_step_noalloc(float* theta, float* m, float* v, const void* g_slow,
                                   long long n, int grad_dtype, const gxpo_opt_cfg* opt,
                                   long long t_opt, double* sumsq_dev, void* stream,
                                   char* errbuf, size_t errbuf_len);

/* Exercises the bounded wait of the bulk-copy variant end to end: a one-thread kernel waits
 * on a barrier that nothing completes, gives up after a few thousand polls and raises the
 * device error word, which this call reads back and clears.  Returns GXPO_ERR_TIMEOUT when
 * that happened -- the expected outcome -- and GXPO_OK otherwise.  The context stays
 * usable.  Only legal between steps; waits for `stream`. */
gxpo_status gxpo_selftest_bounded_wait(gxpo_ctx* ctx, void* stream);

/* Host-side fault injection for tests of the error path: sets the device error word on
 * `stream` exactly as a bounded wait that gave up would, without running any waiting
 * kernel.  The step in flight (or the next one) then reports GXPO_ERR_TIMEOUT where the
 * description of that status says.  The context stays usable. */
gxpo_status gxpo_selftest_inject_timeout(gxpo_ctx* ctx, void* stream);

/* Number of kernels this context has launched so far. */
long long gxpo_launch_count(const gxpo_ctx* ctx);

/* What the most recent sweep call of this context launched: which kernel function the
 * library's dispatch chose for the bound list (it depends on the optimizer, the list's
 * length, gxpo_tune, the gradients-persist promise, diagnostics), its grid, and the bytes
 * per parameter that sweep has to move -- every operand counted once, bfloat16 copies and
 * replayed gradients included.  A benchmark reads its roofline's byte count and kernel
 * name from here instead of repeating the dispatch rules.  extra_launches counts further
 * kernels the same call launched (the separate <g0, g_slow> pass of the diagnostics, whose
 * bytes are included; the clipping coefficient kernel).
 * Paper: no counterpart.  Errors: STATE before the first sweep. */
typedef struct {
    char kernel[48];              /* e.g. "step_kernel", "step_bulk_kernel", "fused_bulk_light_kernel" */
    int staged;                   /* 1: operands staged in shared memory by bulk asynchronous copies */
    int grid;                     /* CTAs launched (0 where the call does not record it) */
    int bytes_read_per_param;
    int bytes_written_per_param;
    int extra_launches;
    int valid;
} gxpo_sweep_info;
gxpo_status gxpo_last_sweep(const gxpo_ctx* ctx, gxpo_sweep_info* out);

const char* gxpo_last_error(const gxpo_ctx* ctx);
const char* gxpo_status_string(gxpo_status s);

/* ---- Surrogate harness (the paper's diagonal-quadratic sanity check, Corollary 1):
 *      f(theta) = sum_i a_i theta_i^2 / 2 - b_i theta_i.  Not part of the update; it
 *      stands in for the caller's backward pass in tests and benchmarks. ---------- */

/* g <- a * theta - b, float32, rounded after the product and after the difference. */
gxpo_status gxpo_quad_grad(const float* theta, const float* a, const float* b, float* g,
                           long long n, void* stream);

/* One whole active step with plain GD on the surrogate in a single sweep: the three
 * gradients are recomputed in registers.  theta is updated in place; sum(g_slow^2)
 * is written to *sumsq_dev (device pointer to one double).  16 bytes per parameter.
 * `scratch_dev` is gxpo_quad_scratch_bytes() of device memory that the caller
 * zeroes once before the first call and then leaves alone. */
gxpo_status gxpo_quad_active_step(float* theta, const float* a, const float* b, long long n,
                                  float lr, int K, float alpha, float delta, float den_eps,
                                  double* sumsq_dev, void* scratch_dev, void* stream);
size_t gxpo_quad_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* GXPO_H */
