// Host side of the GXPO library: context, argument checks, the call-order state
// machine of Algorithm 1, chunk tables and kernel launches.  C ABI in include/gxpo.h.
#include "gxpo.h"
#include "gxpo_kernels.cuh"
#include "gxpo_bulk.cuh"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>
#include <new>
#include <vector>

using namespace gxpo;

namespace {

constexpr int kDefaultCtasStep = 2;    // measured best for the 14R/12W sweep
constexpr int kDefaultCtasStepLight = 3;  // 14R/4W (deferred first probe): read-heavy, wants more loads in flight
constexpr int kDefaultCtasExtrap = 4;  // the extrapolation needs more warps to cover its arithmetic
constexpr int kDefaultCtasFused = 3;   // register-staged fused sweep (its 118-120 registers allow 2)
constexpr int kDefaultCtasBulk = 1;    // bulk-copy staged fused sweep: one ring per SM (two measure the same)

enum Phase { IDLE = 0, PROBED0 = 1, PROBED1 = 2, EXTRAPOLATED = 3, SLOW_DONE = 4, PROBED0_DEFERRED = 5 };

struct Staging {                       // device pieces for gxpo_step_host
    long long elems = 0;
    int slots = 0;
    float* theta[3] = {nullptr, nullptr, nullptr};
    float* work[3] = {nullptr, nullptr, nullptr};
    float* m[3] = {nullptr, nullptr, nullptr};
    float* v[3] = {nullptr, nullptr, nullptr};
    void* g[3][3] = {{nullptr, nullptr, nullptr}, {nullptr, nullptr, nullptr}, {nullptr, nullptr, nullptr}};
    cudaStream_t stream[3] = {nullptr, nullptr, nullptr};
    cudaEvent_t done[3] = {nullptr, nullptr, nullptr};
    double* piece_sumsq = nullptr;     // device accumulator across pieces
};

}  // namespace

struct gxpo_ctx {
    gxpo_cfg cfg;
    gxpo_opt_cfg opt;
    int grad_dtype;
    int device;
    int sm_count;
    int ctas_per_sm;                   // 0 = default
    int variant;                       // 0 = default, 1 = 128-bit, 2 = 256-bit register staging, 3 = 256-bit + bulk-copy staged fused sweep
    int* d_err;                        // device error word (bounded waits)
    int timeout_seen;
    int unit_shift;                    // work unit = kChunk >> unit_shift elements; -1 = choose per launch
    Phase phase;
    // bound list
    TensorDesc* d_descs;
    ChunkRef* d_chunks;
    long long num_chunks;
    int num_tensors;
    int bound;
    std::vector<TensorDesc>* h_descs;  // host copy of the bound descriptors
    int only_bf16_theta1;              // GXPO_BF16_ONLY_*: 1 = the deferred first probe writes the bfloat16 copy only;
                                       // 2 = so does the fused sweep (theta-tilde), and the slow step recomputes it
    int work_missing;                  // some tensor was bound with work == NULL
    FusedParams lag_fused;             // mode 2: the fused sweep's parameters, for the recomputing slow step
    long long total_params;
    // reductions and gate
    double* d_partials;
    unsigned* d_ticket;
    double* d_sumsq;
    double* user_sumsq;                // caller-owned replacement for d_sumsq, or null
    GateState* d_gate;
    double* d_ring;
    GateResult* h_result;              // pinned and mapped: the gate kernel writes it directly
    GateResult* h_result_dev;          // the same memory as the device addresses it
    unsigned long long gate_seq;       // sequence number of the last gate update launched
    cudaEvent_t gate_done;             // recorded after the gate kernel
    int gate_pending;                  // a gate update is in flight (gxpo_gate_update_async)
    int have_gate;
    gxpo_gate_result last_gate;
    // per-step diagnostics (off by default)
    // gradient scaling: per gradient a device scalar (caller's, or clip[] below), or null
    const float* gscale[3];            // what the sweeps use
    const float* user_gscale[3];       // what gxpo_set_grad_scale gave (restored when a clip expires)
    float* d_clip;                     // [3] clipping coefficients written by gxpo_clip_grad_norm
    double* d_gnorm;                   // [3] sum of squares, then [3] norms, of the clipped gradients
    int diag_on;
    int diag_ready;                    // 1 once an active step with diagnostics has completed
    int gslow_aliased;                 // some tensor's g_slow shares g0's buffer: no <g0, g_slow>
    int gslow_shares_probe;            // some tensor's g_slow shares g0's or g1's buffer
    int grads_persist;                 // the caller promised that g0 and g1 outlive the slow step's sweep
    int state_lag;                     // this step's fused sweep left m and v unwritten: the slow step replays (1),
                                       // or recomputes theta-tilde as well (2)
    double* d_diag;                    // kDiagN sums + <g0, g_slow>
    double* d_diag_partials;           // kDiagN x kMaxGrid
    DiagResult* d_diag_result;
    DiagResult* h_diag_result;         // pinned
    // host mirror
    long long t, s_star, t_opt;
    long long launches;
    gxpo_sweep_info last_sweep;        // what the most recent sweep launched (gxpo_last_sweep)
    int wb_any;                        // some tensor has a bfloat16 model-weight copy bound
    // waiting for this context's own work only (re-binding, checkpointing)
    cudaStream_t copy_stream;          // non-blocking; table uploads and state copies
    cudaEvent_t idle_event;            // recorded after work that no gate update follows
    int idle_marked;
    long long desc_cap, chunk_cap;     // capacity of d_descs / d_chunks (entries); tables only grow
    // device error word after a fallback step (no gate kernel runs there to collect it)
    int* h_err;                        // pinned
    cudaEvent_t err_done;
    int err_pending;
    long long err_step;
    const void* occ_key[32];           // resident CTAs per SM, per kernel (cache)
    int occ_val[32];
    int occ_n;
    Staging stg;
    char err[512];
};

namespace {

gxpo_status fail(gxpo_ctx* c, gxpo_status s, const char* fmt, ...) {
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof(c->err), fmt, ap);
        va_end(ap);
    }
    return s;
}

#define CUDA_TRY(c, call)                                                                 \
    do {                                                                                  \
        cudaError_t e_ = (call);                                                          \
        if (e_ != cudaSuccess)                                                            \
            return fail((c), GXPO_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

bool finite_f(float x) { return std::isfinite(x); }

// Remember that `s` carries work of this context which no gate update will follow (a fallback
// step, a clipping pass between steps), so that wait_idle can wait for exactly that work.
gxpo_status mark_idle_work(gxpo_ctx* c, cudaStream_t s) {
    CUDA_TRY(c, cudaEventRecord(c->idle_event, s));
    c->idle_marked = 1;
    return GXPO_OK;
}

// Describe the sweep just launched: kernel function, launch shape and the bytes per parameter
// it has to move.  bench and tests read this instead of re-deriving the dispatch.
void note_sweep(gxpo_ctx* c, const char* kernel, int staged, int grid, int rd, int wr) {
    gxpo_sweep_info& i = c->last_sweep;
    std::snprintf(i.kernel, sizeof(i.kernel), "%s", kernel);
    i.staged = staged;
    i.grid = grid;
    i.bytes_read_per_param = rd;
    i.bytes_written_per_param = wr;
    i.extra_launches = 0;
    i.valid = 1;
}

gxpo_status check_cfg(gxpo_ctx* c, const gxpo_cfg* g, const gxpo_opt_cfg* o, int grad_dtype) {
    if (g->K < 2 || g->K > 4096) return fail(c, GXPO_ERR_INVALID_ARG, "K must be in [2, 4096], got %d", g->K);
    if (!(g->alpha >= 0.0f && g->alpha <= 1.0f)) return fail(c, GXPO_ERR_INVALID_ARG, "alpha must be in [0, 1]");
    if (!(g->delta >= 0.0f) || !finite_f(g->delta)) return fail(c, GXPO_ERR_INVALID_ARG, "delta must be finite and >= 0");
    if (!(g->den_eps >= 0.0f) || !finite_f(g->den_eps)) return fail(c, GXPO_ERR_INVALID_ARG, "den_eps must be finite and >= 0");
    if (std::isnan(g->tau)) return fail(c, GXPO_ERR_INVALID_ARG, "tau is NaN");
    if (!(g->gate_eps >= 0.0)) return fail(c, GXPO_ERR_INVALID_ARG, "gate_eps must be >= 0");
    if (g->window < 1 || g->window > (1 << 20)) return fail(c, GXPO_ERR_INVALID_ARG, "window must be in [1, 2^20]");
    if (g->min_history < 1) return fail(c, GXPO_ERR_INVALID_ARG, "min_history must be >= 1");
    if (g->std_ddof < 0 || g->std_ddof > 1) return fail(c, GXPO_ERR_INVALID_ARG, "std_ddof must be 0 or 1");
    if (g->placement != GXPO_PLACE_PINGPONG && g->placement != GXPO_PLACE_SNAPSHOT)
        return fail(c, GXPO_ERR_INVALID_ARG, "unknown placement %d", g->placement);
    if (o->kind != GXPO_OPT_GD && o->kind != GXPO_OPT_ADAMW) return fail(c, GXPO_ERR_INVALID_ARG, "unknown optimizer kind %d", o->kind);
    if (!std::isfinite(o->lr)) return fail(c, GXPO_ERR_INVALID_ARG, "lr is not finite");
    if (o->kind == GXPO_OPT_ADAMW) {
        if (!(o->beta1 >= 0.0 && o->beta1 < 1.0) || !(o->beta2 >= 0.0 && o->beta2 < 1.0))
            return fail(c, GXPO_ERR_INVALID_ARG, "betas must be in [0, 1)");
        if (!(o->eps >= 0.0) || !std::isfinite(o->eps)) return fail(c, GXPO_ERR_INVALID_ARG, "eps must be finite and >= 0");
        if (!std::isfinite(o->weight_decay)) return fail(c, GXPO_ERR_INVALID_ARG, "weight_decay is not finite");
    }
    if (grad_dtype != GXPO_F32 && grad_dtype != GXPO_BF16) return fail(c, GXPO_ERR_INVALID_ARG, "unknown gradient dtype %d", grad_dtype);
    return GXPO_OK;
}

// Persistent grid: CTAs per SM (tuned or default) clamped to what is actually resident
// for this kernel, times the SM count.  Work is dealt round-robin, so a grid that is
// only partly resident would leave a tail wave running alone.
int grid_for(gxpo_ctx* c, const void* kernel, long long units, int default_per_sm) {
    int per_sm = c->ctas_per_sm > 0 ? c->ctas_per_sm : default_per_sm;
    int resident = 0;
    for (int i = 0; i < c->occ_n; ++i)
        if (c->occ_key[i] == kernel) resident = c->occ_val[i];
    if (resident == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kThreads, 0) != cudaSuccess || resident < 1)
            resident = 1;
        if (c->occ_n < 32) { c->occ_key[c->occ_n] = kernel; c->occ_val[c->occ_n] = resident; c->occ_n += 1; }
    }
    if (per_sm > resident) per_sm = resident;
    long long g = (long long)c->sm_count * per_sm;
    if (g > kMaxGrid) g = kMaxGrid;
    if (g > units) g = units;
    if (g < 1) g = 1;
    return (int)g;
}

// Work unit for one launch.  Whole chunks (16 tiles) have the least per-unit overhead
// and are right for lists of billions of parameters; a list of only a few thousand
// chunks is dealt in quarter or half chunks so that every CTA still gets tens of units
// and the last wave is short.
int unit_shift_for(const gxpo_ctx* c, long long num_chunks) {
    if (c->unit_shift >= 0) return c->unit_shift;
    const long long want = 32LL * c->sm_count * kDefaultCtasStep;
    int sh = 0;
    while (sh < 2 && (num_chunks << sh) < want) ++sh;
    return sh;
}

// (x, x) as one 64-bit word, for the two-lane instructions
unsigned long long pair_of(float x) {
    unsigned u;
    std::memcpy(&u, &x, sizeof(u));
    return ((unsigned long long)u << 32) | u;
}
void fill_step_pairs(StepParams& p) {
    p.beta1_2 = pair_of(p.beta1); p.beta2_2 = pair_of(p.beta2); p.omb1_2 = pair_of(p.omb1); p.omb2_2 = pair_of(p.omb2);
    p.eps_2 = pair_of(p.eps); p.inv_sqrt_bc2_2 = pair_of(p.inv_sqrt_bc2); p.step_2 = pair_of(p.step_size);
    p.decay_2 = pair_of(p.decay); p.neg_lr_2 = pair_of(-p.lr);
}

StepParams make_step_params(gxpo_ctx* c, int which_grad, int in_sel, int out_sel, int snapshot,
                            int want_norm) {
    StepParams p;
    std::memset(&p, 0, sizeof(p));
    p.which_grad = which_grad;
    p.in_sel = in_sel;
    p.out_sel = out_sel;
    p.snapshot = snapshot;
    p.want_norm = want_norm;
    p.write_state = 1;
    p.emit = which_grad != 1;          // no backward pass is taken at theta^{t,2}
    p.gscale = c->gscale[which_grad];
    const gxpo_opt_cfg& o = c->opt;
    p.lr = (float)o.lr;
    if (o.kind == GXPO_OPT_ADAMW) {
        // constants are formed in double from the double hyper-parameters, rounded once
        const double t = (double)c->t_opt;   // already incremented for this step
        const double b1 = o.beta1, b2 = o.beta2, lr = o.lr;
        p.beta1 = (float)b1;
        p.beta2 = (float)b2;
        p.omb1 = (float)(1.0 - b1);
        p.omb2 = (float)(1.0 - b2);
        p.eps = (float)o.eps;
        p.decay = (float)(1.0 - lr * o.weight_decay);
        p.step_size = (float)(lr / (1.0 - std::pow(b1, t)));
        p.inv_sqrt_bc2 = (float)(1.0 / std::sqrt(1.0 - std::pow(b2, t)));
    }
    fill_step_pairs(p);
    return p;
}

// Bytes per parameter a sweep has to move (algorithmic: every operand once).
int grad_bytes(const gxpo_ctx* c) { return c->grad_dtype == GXPO_BF16 ? 2 : 4; }
void note_step(gxpo_ctx* c, const StepParams& p, bool list, bool staged, int grid, bool dot) {
    const bool adamw = c->opt.kind == GXPO_OPT_ADAMW;
    const int G = grad_bytes(c);
    const int rd = 4 + (adamw ? 8 : 0) + G + (p.replay ? 2 * G : 0) + (dot ? G : 0);
    const int wr = (p.skip_out ? 0 : 4) + ((adamw && p.write_state) ? 8 : 0) + (p.snapshot ? 4 : 0) +
                   ((p.emit && list && c->wb_any) ? 2 : 0);
    note_sweep(c, staged ? "step_bulk_kernel" : "step_kernel", staged ? 1 : 0, grid, rd, wr);
}
void note_fused(gxpo_ctx* c, const FusedParams& p, bool list, bool defer, const char* kernel, bool staged, int grid) {
    const bool adamw = c->opt.kind == GXPO_OPT_ADAMW;
    const int G = grad_bytes(c);
    const int rd = (defer ? 4 : 8) + (adamw ? 8 : 0) + 2 * G;
    const int wr = (p.step.skip_out ? 0 : 4) + ((adamw && p.step.write_state) ? 8 : 0) + ((list && c->wb_any) ? 2 : 0);
    note_sweep(c, kernel, staged ? 1 : 0, grid, rd, wr);
}

typedef void (*StepFn)(const TensorDesc*, const ChunkRef*, long long, TensorDesc, StepParams, int,
                       double*, unsigned*, double*);
typedef void (*ExtrapFn)(const TensorDesc*, const ChunkRef*, long long, TensorDesc, ExtrapParams, int,
                         double*, unsigned*, double*);
typedef void (*FusedFn)(const TensorDesc*, const ChunkRef*, long long, TensorDesc, FusedParams, int,
                        double*, unsigned*, double*);

StepFn pick_step(bool adamw, bool bf16, int variant) {
    if (variant != 1) variant = 2;
    if (variant == 1) {
        if (adamw) return bf16 ? step_kernel<true, uint16_t, 4> : step_kernel<true, float, 4>;
        return bf16 ? step_kernel<false, uint16_t, 4> : step_kernel<false, float, 4>;
    }
    if (adamw) return bf16 ? step_kernel<true, uint16_t, 8> : step_kernel<true, float, 8>;
    return bf16 ? step_kernel<false, uint16_t, 8> : step_kernel<false, float, 8>;
}
// With diagnostics the sweeps use the 256-bit access variant only.
ExtrapFn pick_extrap(bool bf16, int variant, bool diag) {
    if (variant != 1) variant = 2;
    if (diag) return bf16 ? extrap_kernel<uint16_t, 8, true> : extrap_kernel<float, 8, true>;
    if (variant == 1) return bf16 ? extrap_kernel<uint16_t, 4, false> : extrap_kernel<float, 4, false>;
    return bf16 ? extrap_kernel<uint16_t, 8, false> : extrap_kernel<float, 8, false>;
}
template <bool DEFER, bool DIAG>
FusedFn pick_fused_t(bool adamw, bool bf16, int variant) {
    if (variant == 1 && !DIAG) {
        if (adamw) return bf16 ? fused_kernel<true, uint16_t, 4, DEFER, false> : fused_kernel<true, float, 4, DEFER, false>;
        return bf16 ? fused_kernel<false, uint16_t, 4, DEFER, false> : fused_kernel<false, float, 4, DEFER, false>;
    }
    if (adamw) return bf16 ? fused_kernel<true, uint16_t, 8, DEFER, DIAG> : fused_kernel<true, float, 8, DEFER, DIAG>;
    return bf16 ? fused_kernel<false, uint16_t, 8, DEFER, DIAG> : fused_kernel<false, float, 8, DEFER, DIAG>;
}
FusedFn pick_fused(bool adamw, bool bf16, int variant, bool defer, bool diag) {
    if (diag) return defer ? pick_fused_t<true, true>(adamw, bf16, variant) : pick_fused_t<false, true>(adamw, bf16, variant);
    return defer ? pick_fused_t<true, false>(adamw, bf16, variant) : pick_fused_t<false, false>(adamw, bf16, variant);
}

// The bulk-copy staged AdamW sweep: one CTA per SM, whole chunks.
typedef void (*StepBulkFn)(const TensorDesc*, const ChunkRef*, long long, TensorDesc, StepParams, int, double*,
                           unsigned*, double*, int*, double*, double*);

// Work unit of a staged sweep: whole chunks on long lists; half or quarter chunks (still whole
// stages) when whole chunks would give a CTA fewer than 32 turns, so that the last round of
// the round-robin leaves few CTAs idle.
int bulk_unit_shift(const gxpo_ctx* c, long long num_chunks, long long grid) {
    if (c->unit_shift >= 0) return c->unit_shift < 2 ? c->unit_shift : 2;
    int sh = 0;
    while (sh < 2 && (num_chunks << sh) < 32 * grid) ++sh;
    return sh;
}
template <typename G>
gxpo_status launch_step_bulk_t(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                               long long num_chunks, const TensorDesc& flat, const StepParams& p, double* sumsq,
                               double* dot_out) {
    StepBulkFn fn;
    int smem;
#define GXPO_STEP_MODE(M) { fn = step_bulk_kernel<true, G, M>; smem = (int)StepLayout<true, G, M>::kTotal; }
    switch ((dot_out ? kStepDot : 0) | (p.replay ? kStepReplay : 0)) {
        case 0: GXPO_STEP_MODE(0) break;
        case kStepDot: GXPO_STEP_MODE(kStepDot) break;
        default: GXPO_STEP_MODE(kStepReplay) break;       // replay never comes with diagnostics
    }
#undef GXPO_STEP_MODE
    int resident = 0;
    for (int i = 0; i < c->occ_n; ++i)
        if (c->occ_key[i] == (const void*)fn) resident = c->occ_val[i];
    if (resident == 0) {
        CUDA_TRY(c, cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, (const void*)fn, kBulkThreads, (size_t)smem) != cudaSuccess || resident < 1)
            resident = 1;
        if (c->occ_n < 32) { c->occ_key[c->occ_n] = (const void*)fn; c->occ_val[c->occ_n] = resident; c->occ_n += 1; }
    }
    int per_sm = c->ctas_per_sm > 0 ? c->ctas_per_sm : kDefaultCtasBulk;
    if (per_sm > resident) per_sm = resident;
    long long g = (long long)c->sm_count * per_sm;
    const int ush = bulk_unit_shift(c, num_chunks, g);
    if (g > (num_chunks << ush)) g = num_chunks << ush;
    // the diagnostics' partial-sum array is idle between the extrapolation sweep and the next step
    fn<<<(int)g, kBulkThreads, smem, s>>>(descs, chunks, num_chunks, flat, p, ush, c->d_partials, c->d_ticket, sumsq, c->d_err,
                                          c->d_diag_partials, dot_out);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    note_step(c, p, chunks != nullptr, true, (int)g, dot_out != nullptr);
    return GXPO_OK;
}
gxpo_status launch_step_bulk(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                             long long num_chunks, const TensorDesc& flat, const StepParams& p, double* sumsq,
                             double* dot_out) {
    return c->grad_dtype == GXPO_BF16 ? launch_step_bulk_t<uint16_t>(c, s, descs, chunks, num_chunks, flat, p, sumsq, dot_out)
                                      : launch_step_bulk_t<float>(c, s, descs, chunks, num_chunks, flat, p, sumsq, dot_out);
}

// The slow step that recomputes theta-tilde (bfloat16-only probe points): one CTA per SM.
typedef void (*SlowRecomputeFn)(const TensorDesc*, const ChunkRef*, long long, TensorDesc, FusedParams, StepParams, int,
                                double*, unsigned*, double*, int*);
gxpo_status launch_slow_recompute(gxpo_ctx* c, cudaStream_t s, const StepParams& p, double* sumsq) {
    if (c->num_chunks <= 0) {
        CUDA_TRY(c, cudaMemsetAsync(sumsq, 0, sizeof(double), s));
        return GXPO_OK;
    }
    const bool bf16 = c->grad_dtype == GXPO_BF16;
    // one CTA per SM with the replaying sweep's ring; two CTAs with the smaller ring on request (gxpo_tune)
    const bool two = c->ctas_per_sm == 2;
    SlowRecomputeFn fn = bf16 ? (two ? slow_recompute_bulk_kernel<uint16_t, 1> : slow_recompute_bulk_kernel<uint16_t, 0>)
                              : (two ? slow_recompute_bulk_kernel<float, 1> : slow_recompute_bulk_kernel<float, 0>);
    const int smem = bf16 ? (two ? (int)RecomputeLayout<uint16_t, 1>::kTotal : (int)RecomputeLayout<uint16_t, 0>::kTotal)
                          : (two ? (int)RecomputeLayout<float, 1>::kTotal : (int)RecomputeLayout<float, 0>::kTotal);
    int resident = 0;
    for (int i = 0; i < c->occ_n; ++i)
        if (c->occ_key[i] == (const void*)fn) resident = c->occ_val[i];
    if (resident == 0) {
        CUDA_TRY(c, cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, (const void*)fn, kBulkThreads, (size_t)smem) != cudaSuccess || resident < 1)
            resident = 1;
        if (c->occ_n < 32) { c->occ_key[c->occ_n] = (const void*)fn; c->occ_val[c->occ_n] = resident; c->occ_n += 1; }
    }
    int per_sm = two ? 2 : 1;
    if (per_sm > resident) per_sm = resident;
    long long g = (long long)c->sm_count * per_sm;
    const int ush = bulk_unit_shift(c, c->num_chunks, g);
    if (g > (c->num_chunks << ush)) g = c->num_chunks << ush;
    const TensorDesc none = {};
    fn<<<(int)g, kBulkThreads, smem, s>>>(c->d_descs, c->d_chunks, c->num_chunks, none, c->lag_fused, p, ush, c->d_partials,
                                          c->d_ticket, sumsq, c->d_err);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    const int G = grad_bytes(c);
    note_sweep(c, "slow_recompute_bulk_kernel", 1, (int)g, 12 + 3 * G, 12 + ((p.emit && c->wb_any) ? 2 : 0));
    return GXPO_OK;
}

// AdamW sweeps that write m and v back run bulk-copy staged on long lists (default) or
// always (variant 3); the read-heavy deferred probe and plain GD stay register-staged.
bool step_runs_staged(const gxpo_ctx* c, const StepParams& p, long long num_chunks) {
    return c->opt.kind == GXPO_OPT_ADAMW && p.write_state &&
           ((c->variant == 0 && num_chunks >= 32LL * c->sm_count) || c->variant == 3);
}

// Launch one OptimStep sweep over either the bound list (chunks != null) or one
// flat piece described by `flat`.
// dot_out (only honoured when the sweep runs staged, see step_runs_staged; want_norm must be
// set): also leave <g0, g> there.
gxpo_status launch_step(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                        long long num_chunks, const TensorDesc& flat, const StepParams& p,
                        double* sumsq, double* dot_out = nullptr) {
    if (num_chunks <= 0) {
        if (p.want_norm) CUDA_TRY(c, cudaMemsetAsync(sumsq, 0, sizeof(double), s));
        return GXPO_OK;
    }
    const bool adamw = c->opt.kind == GXPO_OPT_ADAMW;
    if (p.replay || step_runs_staged(c, p, num_chunks))      // only the staged kernel can replay
        return launch_step_bulk(c, s, descs, chunks, num_chunks, flat, p, sumsq, dot_out);
    StepFn fn = pick_step(adamw, c->grad_dtype == GXPO_BF16, c->variant);
    const int ush = unit_shift_for(c, num_chunks);
    const int grid = grid_for(c, (const void*)fn, num_chunks << ush,
                              (adamw && !p.write_state) ? kDefaultCtasStepLight : kDefaultCtasStep);
    fn<<<grid, kThreads, 0, s>>>(descs, chunks, num_chunks, flat, p, ush, c->d_partials, c->d_ticket, sumsq);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    note_step(c, p, chunks != nullptr, false, grid, false);
    return GXPO_OK;
}

gxpo_status launch_extrap(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                          long long num_chunks, const TensorDesc& flat, const ExtrapParams& p, bool diag) {
    if (num_chunks <= 0) {
        if (diag) CUDA_TRY(c, cudaMemsetAsync(c->d_diag, 0, (kDiagN + 1) * sizeof(double), s));
        return GXPO_OK;
    }
    ExtrapFn fn = pick_extrap(c->grad_dtype == GXPO_BF16, c->variant, diag);
    const int ush = unit_shift_for(c, num_chunks);
    const int grid = grid_for(c, (const void*)fn, num_chunks << ush, kDefaultCtasExtrap);
    fn<<<grid, kThreads, 0, s>>>(descs, chunks, num_chunks, flat, p, ush, c->d_diag_partials, c->d_ticket, c->d_diag);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    note_sweep(c, "extrap_kernel", 0, grid, 8 + 2 * grad_bytes(c), 4 + ((chunks && c->wb_any) ? 2 : 0));
    return GXPO_OK;
}

// The bulk-copy staged variant of the fused sweep: one CTA per SM, whole chunks.
typedef void (*BulkFn)(const TensorDesc*, const ChunkRef*, long long, TensorDesc, FusedParams, int, int*, double*,
                       unsigned*, double*);
template <bool ADAMW, typename G, bool DEFER>
gxpo_status launch_bulk_t(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                          long long num_chunks, const TensorDesc& flat, const FusedParams& p, bool diag) {
    BulkFn fn = diag ? fused_bulk_kernel<ADAMW, G, DEFER, true> : fused_bulk_kernel<ADAMW, G, DEFER, false>;
    int smem = (int)BulkLayout<ADAMW, G, DEFER>::kTotal;
    int want_per_sm = kDefaultCtasBulk;
    const char* name = "fused_bulk_kernel";
    if constexpr (ADAMW && DEFER) {
        if (!p.step.write_state && !diag) {   // m and v stay unwritten: the latency-bound shape, two CTAs per SM
            fn = fused_bulk_light_kernel<G>;                      // (with diagnostics it would not fit the registers)
            smem = (int)BulkLayout<true, G, true, true>::kTotal;
            want_per_sm = 2;
            name = "fused_bulk_light_kernel";
        }
    }
    // first launch of this instantiation in this context: allow the ring's shared memory and
    // find out how many CTAs fit; remembered in the occupancy cache afterwards
    int resident = 0;
    for (int i = 0; i < c->occ_n; ++i)
        if (c->occ_key[i] == (const void*)fn) resident = c->occ_val[i];
    if (resident == 0) {
        CUDA_TRY(c, cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, (const void*)fn, kBulkThreads, (size_t)smem) != cudaSuccess || resident < 1)
            resident = 1;
        if (c->occ_n < 32) { c->occ_key[c->occ_n] = (const void*)fn; c->occ_val[c->occ_n] = resident; c->occ_n += 1; }
    }
    int per_sm = c->ctas_per_sm > 0 ? c->ctas_per_sm : want_per_sm;
    if (per_sm > resident) per_sm = resident;
    long long g = (long long)c->sm_count * per_sm;
    const int ush = bulk_unit_shift(c, num_chunks, g);
    if (g > (num_chunks << ush)) g = num_chunks << ush;
    fn<<<(int)g, kBulkThreads, smem, s>>>(descs, chunks, num_chunks, flat, p, ush, c->d_err, c->d_diag_partials,
                                          c->d_ticket, c->d_diag);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    note_fused(c, p, chunks != nullptr, DEFER, name, true, (int)g);
    return GXPO_OK;
}
gxpo_status launch_fused_bulk(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                              long long num_chunks, const TensorDesc& flat, const FusedParams& p, bool defer,
                              bool diag) {
    const bool adamw = c->opt.kind == GXPO_OPT_ADAMW, bf16 = c->grad_dtype == GXPO_BF16;
#define GXPO_BULK(A, G) (defer ? launch_bulk_t<A, G, true>(c, s, descs, chunks, num_chunks, flat, p, diag) \
                               : launch_bulk_t<A, G, false>(c, s, descs, chunks, num_chunks, flat, p, diag))
    if (adamw) return bf16 ? GXPO_BULK(true, uint16_t) : GXPO_BULK(true, float);
    return bf16 ? GXPO_BULK(false, uint16_t) : GXPO_BULK(false, float);
#undef GXPO_BULK
}

gxpo_status launch_fused(gxpo_ctx* c, cudaStream_t s, const TensorDesc* descs, const ChunkRef* chunks,
                         long long num_chunks, const TensorDesc& flat, const FusedParams& p, bool defer,
                         bool diag) {
    if (num_chunks <= 0) {
        if (diag) CUDA_TRY(c, cudaMemsetAsync(c->d_diag, 0, (kDiagN + 1) * sizeof(double), s));
        return GXPO_OK;
    }
    // default (0): the bulk-copy staged kernel for lists long enough to keep every SM's ring
    // busy (it deals whole chunks, one CTA per SM), register staging for short lists; 3
    // forces bulk staging, 1 and 2 force register staging.
    // A sweep that leaves m and v unwritten (see gxpo_probe_extrapolate) has its own staged shape, which
    // pays from far shorter lists on; the caller has checked that.
    const bool long_list = num_chunks >= 32LL * c->sm_count;
    const bool light = c->opt.kind == GXPO_OPT_ADAMW && defer && !p.step.write_state;
    if ((c->variant == 0 && (long_list || light)) || c->variant == 3)
        return launch_fused_bulk(c, s, descs, chunks, num_chunks, flat, p, defer, diag);
    FusedFn fn = pick_fused(c->opt.kind == GXPO_OPT_ADAMW, c->grad_dtype == GXPO_BF16, c->variant == 1 ? 1 : 2, defer, diag);
    const int ush = unit_shift_for(c, num_chunks);
    const int grid = grid_for(c, (const void*)fn, num_chunks << ush, kDefaultCtasFused);
    fn<<<grid, kThreads, 0, s>>>(descs, chunks, num_chunks, flat, p, ush, c->d_diag_partials, c->d_ticket, c->d_diag);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    note_fused(c, p, chunks != nullptr, defer, "fused_kernel", false, grid);
    return GXPO_OK;
}

ExtrapParams make_extrap_params(const gxpo_ctx* c, int placement) {
    ExtrapParams p;
    p.K = c->cfg.K;
    p.alpha = c->cfg.alpha;
    p.delta = c->cfg.delta;
    p.den_eps = c->cfg.den_eps;
    p.alpha_2 = pair_of(p.alpha); p.one_2 = pair_of(1.0f); p.neg_one_2 = pair_of(-1.0f);
    p.gscale0 = c->gscale[0];
    p.gscale1 = c->gscale[1];
    if (placement == GXPO_PLACE_PINGPONG) { p.theta2_sel = 1; p.theta0_sel = 0; }
    else { p.theta2_sel = 0; p.theta0_sel = 1; }
    return p;
}

bool gate_active(const gxpo_ctx* c) { return c->s_star < 0 || c->t < c->s_star; }

// A clipping coefficient belongs to the step it was computed in.
void expire_clips(gxpo_ctx* c) {
    for (int k = 0; k < 3; ++k) c->gscale[k] = c->user_gscale[k];
}

// Enqueue the gate kernel and its read-back; the host learns the outcome in finish_gate.
// t advances by one whatever the outcome, so the host mirror moves on at once.
gxpo_status launch_gate(gxpo_ctx* c, cudaStream_t s, const double* sumsq) {
    c->gate_seq += 1;
    gate_kernel<<<1, 32, 0, s>>>(c->d_gate, c->d_ring, sumsq, c->t, c->cfg.tau, c->cfg.gate_eps,
                                 c->cfg.window, c->cfg.min_history, c->cfg.std_ddof, c->d_err, c->h_result_dev, c->gate_seq);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    CUDA_TRY(c, cudaEventRecord(c->gate_done, s));
    c->gate_pending = 1;
    c->t += 1;
    return GXPO_OK;
}

// Wait for a pending gate read-back (if any) and fold it into the host mirror.
gxpo_status finish_gate(gxpo_ctx* c) {
    if (!c->gate_pending) return GXPO_OK;
    // Poll the record's sequence number in host memory (the kernel writes it last); after a
    // bounded number of polls fall back to waiting on the event, which also surfaces a failed launch.
    volatile unsigned long long* seq = &c->h_result->seq;
    bool seen = false;
    for (int spin = 0; spin < (1 << 22); ++spin) {
        if (*seq == c->gate_seq) { seen = true; break; }
#if defined(__x86_64__) || defined(__i386__)
        __builtin_ia32_pause();
#endif
    }
    if (!seen) {
        CUDA_TRY(c, cudaEventSynchronize(c->gate_done));
        if (*seq != c->gate_seq) return fail(c, GXPO_ERR_CUDA, "the gate kernel finished without delivering its result");
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    c->gate_pending = 0;
    const GateResult r = *c->h_result;
    c->s_star = r.s_star;
    if (r.dev_error) c->timeout_seen = 1;
    gxpo_gate_result& o = c->last_gate;
    o.active = r.active; o.tripped = r.tripped; o.t = r.t; o.s_star = r.s_star;
    o.norm = r.norm; o.z = r.z; o.mu = r.mu; o.sigma = r.sigma;
    c->have_gate = 1;
    return GXPO_OK;
}

// A fallback step runs no gate kernel, so nothing collects the device error word a bounded
// wait may have raised in its staged sweep.  The sweep is therefore followed by a 4-byte
// read-back of the word (and its reset); the next call that looks at the context's state
// folds it in here and reports the incomplete step once.
gxpo_status enqueue_error_readback(gxpo_ctx* c, cudaStream_t s, long long step) {
    CUDA_TRY(c, cudaMemcpyAsync(c->h_err, c->d_err, sizeof(int), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(c, cudaMemsetAsync(c->d_err, 0, sizeof(int), s));
    CUDA_TRY(c, cudaEventRecord(c->err_done, s));
    c->err_pending = 1;
    c->err_step = step;
    return GXPO_OK;
}
gxpo_status collect_fallback_error(gxpo_ctx* c) {
    if (!c->err_pending) return GXPO_OK;
    CUDA_TRY(c, cudaEventSynchronize(c->err_done));
    c->err_pending = 0;
    if (*c->h_err) {
        *c->h_err = 0;
        return fail(c, GXPO_ERR_TIMEOUT, "a bounded device-side wait gave up during fallback step %lld: its outputs are incomplete", c->err_step);
    }
    return GXPO_OK;
}

// Wait until everything this context has enqueued so far is complete -- its own work only, not
// the device: a pending gate read-back, then whatever followed the last gate update.
gxpo_status wait_idle(gxpo_ctx* c) {
    gxpo_status st = finish_gate(c);
    if (st != GXPO_OK) return st;
    if (c->idle_marked) {
        CUDA_TRY(c, cudaEventSynchronize(c->idle_event));
        c->idle_marked = 0;
    }
    return GXPO_OK;
}

gxpo_status gate_outcome(gxpo_ctx* c, gxpo_gate_result* out) {
    if (out) *out = c->last_gate;
    if (c->timeout_seen) {
        c->timeout_seen = 0;
        return fail(c, GXPO_ERR_TIMEOUT, "a bounded device-side wait gave up during step %lld: its outputs are incomplete", c->last_gate.t - 1);
    }
    if (!std::isfinite(c->last_gate.norm))
        return fail(c, GXPO_ERR_NONFINITE, "||g_slow|| is not finite at step %lld; gate tripped", c->last_gate.t - 1);
    return GXPO_OK;
}

gxpo_status run_gate(gxpo_ctx* c, cudaStream_t s, const double* sumsq, gxpo_gate_result* out) {
    gxpo_status st = launch_gate(c, s, sumsq);
    if (st == GXPO_OK) st = finish_gate(c);
    if (st != GXPO_OK) return st;
    return gate_outcome(c, out);
}

void free_staging(gxpo_ctx* c) {
    Staging& st = c->stg;
    for (int i = 0; i < 3; ++i) {
        cudaFree(st.theta[i]); cudaFree(st.work[i]); cudaFree(st.m[i]); cudaFree(st.v[i]);
        for (int k = 0; k < 3; ++k) cudaFree(st.g[i][k]);
        if (st.stream[i]) cudaStreamDestroy(st.stream[i]);
        if (st.done[i]) cudaEventDestroy(st.done[i]);
    }
    cudaFree(st.piece_sumsq);
    st = Staging();
}

gxpo_status ensure_staging(gxpo_ctx* c, long long elems) {
    Staging& st = c->stg;
    if (st.elems >= elems && st.slots > 0) return GXPO_OK;
    free_staging(c);
    const size_t gsz = (c->grad_dtype == GXPO_BF16) ? 2 : 4;
    const bool adamw = c->opt.kind == GXPO_OPT_ADAMW;
    for (int i = 0; i < 2; ++i) {
        CUDA_TRY(c, cudaMalloc(&st.theta[i], elems * sizeof(float)));
        CUDA_TRY(c, cudaMalloc(&st.work[i], elems * sizeof(float)));
        if (adamw) {
            CUDA_TRY(c, cudaMalloc(&st.m[i], elems * sizeof(float)));
            CUDA_TRY(c, cudaMalloc(&st.v[i], elems * sizeof(float)));
        }
        for (int k = 0; k < 3; ++k) CUDA_TRY(c, cudaMalloc(&st.g[i][k], elems * gsz));
        CUDA_TRY(c, cudaStreamCreateWithFlags(&st.stream[i], cudaStreamNonBlocking));
        CUDA_TRY(c, cudaEventCreateWithFlags(&st.done[i], cudaEventDisableTiming));
    }
    CUDA_TRY(c, cudaMalloc(&st.piece_sumsq, 2 * sizeof(double)));
    st.elems = elems;
    st.slots = 2;
    return GXPO_OK;
}

__global__ void accumulate_kernel(double* total, const double* piece) {
    if (threadIdx.x == 0 && blockIdx.x == 0) *total = __dadd_rn(*total, *piece);
}

}  // namespace

extern "C" {

void gxpo_default_cfg(gxpo_cfg* cfg, gxpo_opt_cfg* opt) {
    if (cfg) {
        cfg->K = 5;
        cfg->alpha = 0.5f;
        cfg->delta = 1e-8f;
        cfg->den_eps = 0.0f;
        cfg->tau = 0.5;
        cfg->gate_eps = 1e-8;
        cfg->window = 20;
        cfg->min_history = 2;
        cfg->std_ddof = 0;
        cfg->placement = GXPO_PLACE_PINGPONG;
    }
    if (opt) {
        opt->kind = GXPO_OPT_ADAMW;
        opt->lr = 1e-7;
        opt->beta1 = 0.9;
        opt->beta2 = 0.999;
        opt->eps = 1e-8;
        opt->weight_decay = 0.01;
    }
}

gxpo_status gxpo_create(const gxpo_cfg* cfg, const gxpo_opt_cfg* opt, int grad_dtype, gxpo_ctx** out) {
    if (!cfg || !opt || !out) return GXPO_ERR_INVALID_ARG;
    *out = nullptr;
    gxpo_status s = check_cfg(nullptr, cfg, opt, grad_dtype);
    if (s != GXPO_OK) return s;
    gxpo_ctx* c = new (std::nothrow) gxpo_ctx();
    if (!c) return GXPO_ERR_INVALID_ARG;
    std::memset(static_cast<void*>(c), 0, sizeof(*c));
    new (&c->stg) Staging();
    c->cfg = *cfg;
    c->opt = *opt;
    c->grad_dtype = grad_dtype;
    c->variant = 0;
    c->unit_shift = -1;
    c->s_star = -1;
    c->phase = IDLE;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_partials, kMaxGrid * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_ticket, sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_sumsq, sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_err, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->d_err, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_gate, sizeof(GateState));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_ring, (size_t)cfg->window * sizeof(double));
    if (e == cudaSuccess) e = cudaHostAlloc(&c->h_result, sizeof(GateResult), cudaHostAllocMapped);
    if (e == cudaSuccess) std::memset(c->h_result, 0, sizeof(GateResult));
    if (e == cudaSuccess) e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->h_result_dev), c->h_result, 0);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->gate_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->idle_event, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->err_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaMallocHost(&c->h_err, sizeof(int));
    if (e == cudaSuccess) *c->h_err = 0;
    if (e == cudaSuccess) e = cudaMalloc(&c->d_clip, 3 * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_gnorm, 6 * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_diag, (kDiagN + 1) * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_diag_partials, (size_t)kDiagN * kMaxGrid * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_diag_result, sizeof(DiagResult));
    if (e == cudaSuccess) e = cudaMallocHost(&c->h_diag_result, sizeof(DiagResult));
    if (e == cudaSuccess) e = cudaMemset(c->d_diag, 0, (kDiagN + 1) * sizeof(double));
    if (e == cudaSuccess) e = cudaMemset(c->d_ticket, 0, sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMemset(c->d_sumsq, 0, sizeof(double));
    if (e == cudaSuccess) e = cudaMemset(c->d_ring, 0, (size_t)cfg->window * sizeof(double));
    if (e == cudaSuccess) {
        GateState g0;
        g0.head = 0; g0.count = 0; g0.s_star = -1;
        e = cudaMemcpy(c->d_gate, &g0, sizeof(g0), cudaMemcpyHostToDevice);
    }
    if (e != cudaSuccess) {
        gxpo_destroy(c);
        return GXPO_ERR_CUDA;
    }
    *out = c;
    return GXPO_OK;
}

void gxpo_destroy(gxpo_ctx* c) {
    if (!c) return;
    free_staging(c);
    cudaFree(c->d_descs);
    cudaFree(c->d_chunks);
    cudaFree(c->d_partials);
    cudaFree(c->d_ticket);
    cudaFree(c->d_sumsq);
    cudaFree(c->d_err);
    cudaFree(c->d_gate);
    cudaFree(c->d_ring);
    if (c->h_result) cudaFreeHost(c->h_result);
    if (c->gate_done) cudaEventDestroy(c->gate_done);
    if (c->idle_event) cudaEventDestroy(c->idle_event);
    if (c->err_done) cudaEventDestroy(c->err_done);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    if (c->h_err) cudaFreeHost(c->h_err);
    delete c->h_descs;
    cudaFree(c->d_clip);
    cudaFree(c->d_gnorm);
    cudaFree(c->d_diag);
    cudaFree(c->d_diag_partials);
    cudaFree(c->d_diag_result);
    if (c->h_diag_result) cudaFreeHost(c->h_diag_result);
    delete c;
}

static gxpo_status check_tensor(gxpo_ctx* c, const gxpo_tensor& t, int i, bool need_work) {
    if (t.n < 0) return fail(c, GXPO_ERR_INVALID_ARG, "tensor %d: n < 0", i);
    if (t.n > (long long)kChunk * 0xFFFFFFFFLL) return fail(c, GXPO_ERR_INVALID_ARG, "tensor %d: n too large", i);
    if (t.n == 0) return GXPO_OK;
    if (!t.theta || !t.g0 || !t.g1 || !t.g_slow || (need_work && !t.work))
        return fail(c, GXPO_ERR_INVALID_ARG, "tensor %d: null theta/work/gradient pointer", i);
    if (c->opt.kind == GXPO_OPT_ADAMW && (!t.m || !t.v))
        return fail(c, GXPO_ERR_INVALID_ARG, "tensor %d: AdamW needs m and v", i);
    const uintptr_t gmask = (c->grad_dtype == GXPO_BF16) ? 1u : 3u;
    if ((((uintptr_t)t.theta) & 3u) || (((uintptr_t)t.work) & 3u) || (((uintptr_t)t.m) & 3u) ||
        (((uintptr_t)t.v) & 3u) || (((uintptr_t)t.g0) & gmask) || (((uintptr_t)t.g1) & gmask) ||
        (((uintptr_t)t.g_slow) & gmask))
        return fail(c, GXPO_ERR_ALIGNMENT, "tensor %d: a pointer is not aligned to its element size", i);
    return GXPO_OK;
}

gxpo_status gxpo_bind(gxpo_ctx* c, const gxpo_tensor* list, int count) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (count < 0 || (count > 0 && !list)) return fail(c, GXPO_ERR_INVALID_ARG, "bad list/count");
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "gxpo_bind in the middle of a step");
    std::vector<TensorDesc> descs((size_t)count);
    std::vector<ChunkRef> chunks;
    long long total = 0;
    int aliased = 0, shares_probe = 0, work_missing = 0;
    for (int i = 0; i < count; ++i) {
        gxpo_status s = check_tensor(c, list[i], i, false);
        if (s != GXPO_OK) return s;
        if (list[i].n > 0 && !list[i].work) work_missing = 1;
        TensorDesc& d = descs[(size_t)i];
        d.theta = list[i].theta; d.work = list[i].work; d.m = list[i].m; d.v = list[i].v;
        d.g[0] = list[i].g0; d.g[1] = list[i].g1; d.g[2] = list[i].g_slow;
        d.n = list[i].n;
        total += d.n;
        if (d.n > 0 && d.g[2] == d.g[0]) aliased = 1;
        if (d.n > 0 && (d.g[2] == d.g[0] || d.g[2] == d.g[1])) shares_probe = 1;
    }
    chunks.reserve((size_t)(total / kChunk + count));
    for (int i = 0; i < count; ++i) {
        const long long nc = (descs[(size_t)i].n + kChunk - 1) / kChunk;
        for (long long k = 0; k < nc; ++k) chunks.push_back(ChunkRef{(unsigned)i, (unsigned)k});
    }
    // The old tables may still be read by this context's last sweeps: wait for those (this
    // context's work only; other streams of the process keep running), then overwrite the
    // tables in place.  They are reallocated only when the new list needs more room.
    { gxpo_status ws = wait_idle(c); if (ws != GXPO_OK) return ws; }
    c->num_chunks = 0; c->num_tensors = 0; c->total_params = 0; c->bound = 0;
    if ((long long)descs.size() > c->desc_cap) {
        cudaFree(c->d_descs); c->d_descs = nullptr; c->desc_cap = 0;
        CUDA_TRY(c, cudaMalloc(&c->d_descs, descs.size() * sizeof(TensorDesc)));
        c->desc_cap = (long long)descs.size();
    }
    if ((long long)chunks.size() > c->chunk_cap) {
        cudaFree(c->d_chunks); c->d_chunks = nullptr; c->chunk_cap = 0;
        CUDA_TRY(c, cudaMalloc(&c->d_chunks, chunks.size() * sizeof(ChunkRef)));
        c->chunk_cap = (long long)chunks.size();
    }
    if (count > 0)
        CUDA_TRY(c, cudaMemcpyAsync(c->d_descs, descs.data(), descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice, c->copy_stream));
    if (!chunks.empty())
        CUDA_TRY(c, cudaMemcpyAsync(c->d_chunks, chunks.data(), chunks.size() * sizeof(ChunkRef), cudaMemcpyHostToDevice, c->copy_stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->copy_stream));
    c->num_chunks = (long long)chunks.size();
    c->num_tensors = count;
    c->total_params = total;
    c->gslow_aliased = aliased;
    c->gslow_shares_probe = shares_probe;
    c->state_lag = 0;
    c->diag_ready = 0;
    c->only_bf16_theta1 = 0;
    c->work_missing = work_missing;
    c->wb_any = 0;
    if (!c->h_descs) c->h_descs = new (std::nothrow) std::vector<TensorDesc>();
    if (!c->h_descs) return fail(c, GXPO_ERR_INVALID_ARG, "out of host memory");
    *c->h_descs = descs;
    c->bound = 1;
    return GXPO_OK;
}

gxpo_status gxpo_bind_model_weights(gxpo_ctx* c, void* const* weights_bf16, int count, int only_bf16_theta1) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (!c->bound || !c->h_descs) return fail(c, GXPO_ERR_STATE, "nothing bound: call gxpo_bind first");
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "model weights can only be bound between steps");
    std::vector<TensorDesc>& descs = *c->h_descs;
    if (weights_bf16 && count != (int)descs.size())
        return fail(c, GXPO_ERR_INVALID_ARG, "count %d does not match the %d bound tensors", count, (int)descs.size());
    bool all = weights_bf16 != nullptr;
    for (size_t i = 0; i < descs.size(); ++i) {
        void* w = weights_bf16 ? weights_bf16[i] : nullptr;
        if (((uintptr_t)w) & 1u) return fail(c, GXPO_ERR_ALIGNMENT, "tensor %d: bfloat16 pointer is not 2-byte aligned", (int)i);
        if (!w && descs[i].n > 0) all = false;
    }
    if (only_bf16_theta1 < 0 || only_bf16_theta1 > 2)
        return fail(c, GXPO_ERR_INVALID_ARG, "bf16_only must be GXPO_BF16_BESIDE (0), GXPO_BF16_ONLY_THETA1 (1) or GXPO_BF16_ONLY_PROBE_POINTS (2)");
    if (only_bf16_theta1 && (!all || c->cfg.placement != GXPO_PLACE_PINGPONG))
        return fail(c, GXPO_ERR_INVALID_ARG, "bfloat16-only points need a bfloat16 buffer for every tensor and PINGPONG placement");
    if (only_bf16_theta1 == 2 && c->opt.kind != GXPO_OPT_ADAMW)
        return fail(c, GXPO_ERR_INVALID_ARG, "GXPO_BF16_ONLY_PROBE_POINTS is built for AdamW only");
    int any = 0;
    for (size_t i = 0; i < descs.size(); ++i) {
        descs[i].wb = static_cast<uint16_t*>(weights_bf16 ? weights_bf16[i] : nullptr);
        if (descs[i].wb && descs[i].n > 0) any = 1;
    }
    { gxpo_status ws = wait_idle(c); if (ws != GXPO_OK) return ws; }
    if (!descs.empty()) {
        CUDA_TRY(c, cudaMemcpyAsync(c->d_descs, descs.data(), descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice, c->copy_stream));
        CUDA_TRY(c, cudaStreamSynchronize(c->copy_stream));
    }
    c->wb_any = any;
    c->only_bf16_theta1 = only_bf16_theta1;
    return GXPO_OK;
}

gxpo_status gxpo_probe_step(gxpo_ctx* c, int which, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (which < -1 || which > 1) return fail(c, GXPO_ERR_INVALID_ARG, "which must be -1, 0 or 1");
    if (!c->bound) return fail(c, GXPO_ERR_STATE, "nothing bound: call gxpo_bind first");
    cudaStream_t s = (cudaStream_t)stream;
    const TensorDesc none = {};
    const int place = c->cfg.placement;
    if (which == -1) {
        if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "fallback step in the middle of an active step");
        { gxpo_status fe = collect_fallback_error(c); if (fe != GXPO_OK) return fe; }
        c->t_opt += 1;
        StepParams p = make_step_params(c, 0, 0, 0, 0, 0);
        gxpo_status st = launch_step(c, s, c->d_descs, c->d_chunks, c->num_chunks, none, p, c->d_sumsq);
        if (st != GXPO_OK) { c->t_opt -= 1; return st; }
        // only the staged sweep waits on anything; it alone can raise the error word
        if (c->num_chunks > 0 && step_runs_staged(c, p, c->num_chunks)) {
            st = enqueue_error_readback(c, s, c->t);
            if (st != GXPO_OK) return st;
        }
        st = mark_idle_work(c, s);
        if (st != GXPO_OK) return st;
        c->t += 1;
        expire_clips(c);
        return GXPO_OK;
    }
    if (c->work_missing) return fail(c, GXPO_ERR_STATE, "this call keeps a point in `work`, which was bound as NULL");
    if (which == 0) {
        if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "probe step 0 must start a step");
        { gxpo_status fe = collect_fallback_error(c); if (fe != GXPO_OK) return fe; }
        { gxpo_status fg = finish_gate(c); if (fg != GXPO_OK) return fg; }
        if (!gate_active(c)) return fail(c, GXPO_ERR_STATE, "gate has tripped (s*=%lld, t=%lld): only fallback steps are legal", c->s_star, c->t);
        c->t_opt += 1;
        StepParams p = (place == GXPO_PLACE_PINGPONG) ? make_step_params(c, 0, 0, 1, 0, 0)
                                                      : make_step_params(c, 0, 0, 0, 1, 0);
        gxpo_status st = launch_step(c, s, c->d_descs, c->d_chunks, c->num_chunks, none, p, c->d_sumsq);
        if (st != GXPO_OK) { c->t_opt -= 1; return st; }
        c->phase = PROBED0;
        return GXPO_OK;
    }
    if (c->phase == PROBED0_DEFERRED)
        return fail(c, GXPO_ERR_STATE, "after gxpo_probe_step_deferred only gxpo_probe_extrapolate can take the second probe step");
    if (c->phase != PROBED0) return fail(c, GXPO_ERR_STATE, "probe step 1 must follow probe step 0");
    c->t_opt += 1;
    StepParams p = (place == GXPO_PLACE_PINGPONG) ? make_step_params(c, 1, 1, 1, 0, 0)
                                                  : make_step_params(c, 1, 0, 0, 0, 0);
    gxpo_status st = launch_step(c, s, c->d_descs, c->d_chunks, c->num_chunks, none, p, c->d_sumsq);
    if (st != GXPO_OK) { c->t_opt -= 1; return st; }
    c->phase = PROBED1;
    return GXPO_OK;
}

// theta-tilde as bfloat16 only: theta^t has to survive in `theta` and m, v have to stay put until
// the slow step, which recomputes theta-tilde from g0 and g1 -- that is the deferred flow under
// the gradients-persist promise, and nothing else.  Checked before the step starts.
static gxpo_status check_only16(gxpo_ctx* c) {
    if (!c->grads_persist || c->gslow_shares_probe)
        return fail(c, GXPO_ERR_STATE, "GXPO_BF16_ONLY_PROBE_POINTS needs gxpo_set_gradients_persist(ctx, 1) and a g_slow buffer apart from g0 and g1: the slow step recomputes theta-tilde from them");
    if (c->diag_on) return fail(c, GXPO_ERR_STATE, "GXPO_BF16_ONLY_PROBE_POINTS does not go with diagnostics");
    if (c->variant == 1 || c->variant == 2)
        return fail(c, GXPO_ERR_STATE, "GXPO_BF16_ONLY_PROBE_POINTS runs in the shared-memory staged sweeps only (gxpo_tune variant 0 or 3)");
    return GXPO_OK;
}

gxpo_status gxpo_probe_step_deferred(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (!c->bound) return fail(c, GXPO_ERR_STATE, "nothing bound: call gxpo_bind first");
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "probe step 0 must start a step");
    if (c->only_bf16_theta1 == 2) { gxpo_status os = check_only16(c); if (os != GXPO_OK) return os; }
    if (c->work_missing && !c->only_bf16_theta1)
        return fail(c, GXPO_ERR_STATE, "theta^{t,1} goes to `work`, which was bound as NULL (bind bfloat16 copies with GXPO_BF16_ONLY_THETA1 or GXPO_BF16_ONLY_PROBE_POINTS)");
    { gxpo_status fe = collect_fallback_error(c); if (fe != GXPO_OK) return fe; }
    { gxpo_status fg = finish_gate(c); if (fg != GXPO_OK) return fg; }
    if (!gate_active(c)) return fail(c, GXPO_ERR_STATE, "gate has tripped (s*=%lld, t=%lld): only fallback steps are legal", c->s_star, c->t);
    const TensorDesc none = {};
    c->t_opt += 1;
    StepParams p = (c->cfg.placement == GXPO_PLACE_PINGPONG) ? make_step_params(c, 0, 0, 1, 0, 0)
                                                             : make_step_params(c, 0, 0, 0, 1, 0);
    p.write_state = 0;
    p.skip_out = c->only_bf16_theta1 ? 1 : 0;
    gxpo_status st = launch_step(c, (cudaStream_t)stream, c->d_descs, c->d_chunks, c->num_chunks, none, p, c->d_sumsq);
    if (st != GXPO_OK) { c->t_opt -= 1; return st; }
    c->phase = PROBED0_DEFERRED;
    return GXPO_OK;
}

gxpo_status gxpo_extrapolate(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != PROBED1) return fail(c, GXPO_ERR_STATE, "extrapolate must follow probe step 1");
    const TensorDesc none = {};
    gxpo_status st = launch_extrap(c, (cudaStream_t)stream, c->d_descs, c->d_chunks, c->num_chunks, none,
                                   make_extrap_params(c, c->cfg.placement), c->diag_on != 0);
    if (st != GXPO_OK) return st;
    c->phase = EXTRAPOLATED;
    return GXPO_OK;
}

gxpo_status gxpo_probe_extrapolate(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != PROBED0 && c->phase != PROBED0_DEFERRED)
        return fail(c, GXPO_ERR_STATE, "fused probe+extrapolate must follow probe step 0");
    if (c->work_missing && c->only_bf16_theta1 != 2 && c->cfg.placement != GXPO_PLACE_PINGPONG)
        return fail(c, GXPO_ERR_STATE, "this placement keeps theta^t in `work`, which was bound as NULL");
    const TensorDesc none = {};
    const int place = c->cfg.placement;
    const bool defer = c->phase == PROBED0_DEFERRED;
    const bool only16 = c->only_bf16_theta1 == 2;      // theta-tilde as bfloat16 only
    if (only16) {
        if (!defer) return fail(c, GXPO_ERR_STATE, "GXPO_BF16_ONLY_PROBE_POINTS: take the first probe step with gxpo_probe_step_deferred");
        gxpo_status os = check_only16(c);
        if (os != GXPO_OK) return os;
    }
    FusedParams p;
    p.step0 = make_step_params(c, 0, 0, 0, 0, 0);       // constants of the first probe step (replayed when deferred)
    c->t_opt += 1;
    p.step = (place == GXPO_PLACE_PINGPONG) ? make_step_params(c, 1, 1, 1, 0, 0) : make_step_params(c, 1, 0, 0, 0, 0);
    p.ex = make_extrap_params(c, place);
    // With the caller's promise that g0 and g1 outlive the slow step's sweep, m and v can stay
    // unwritten once more: the slow step's staged sweep replays both moment updates from g0
    // and g1 (8 bytes of writes saved here, 4 bytes of reads added there).  Both sweeps then
    // run staged.  Never when g_slow lands in g0's or g1's buffer, and not with diagnostics on
    // (their arithmetic, not the state writes, then bounds this sweep).
    // Measured: the pair of staged sweeps (20 + 30 B/param) beats the register-staged pair (28 + 26) from
    // about 6 chunks per SM on (flat 40M parameters: 0.478 against 0.491 ms per step; 20M: 0.284 against 0.278).
    const bool lag = defer && c->grads_persist && !c->gslow_shares_probe && c->opt.kind == GXPO_OPT_ADAMW &&
                     !c->diag_on &&
                     (c->variant == 3 || (c->variant == 0 && c->num_chunks >= 8LL * c->sm_count));
    if (lag || only16) p.step.write_state = 0;
    gxpo_status st;
    if (only16) {
        p.step.skip_out = 1;
        c->lag_fused = p;
        st = c->num_chunks > 0 ? launch_fused_bulk(c, (cudaStream_t)stream, c->d_descs, c->d_chunks, c->num_chunks, none, p, true, false)
                               : GXPO_OK;
    } else {
        st = launch_fused(c, (cudaStream_t)stream, c->d_descs, c->d_chunks, c->num_chunks, none, p, defer, c->diag_on != 0);
    }
    if (st != GXPO_OK) { c->t_opt -= 1; return st; }
    c->state_lag = only16 ? 2 : (lag ? 1 : 0);
    c->phase = EXTRAPOLATED;
    return GXPO_OK;
}

gxpo_status gxpo_slow_step(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != EXTRAPOLATED) return fail(c, GXPO_ERR_STATE, "slow step must follow extrapolate");
    const TensorDesc none = {};
    c->t_opt += 1;
    StepParams p = make_step_params(c, 2, 0, 0, 0, 1);
    // diagnostics: <g0, g_slow> rides along in the staged sweep (one more read of g0);
    // otherwise it is a pass of its own over both gradients
    if (c->state_lag == 2) {
        gxpo_status st2 = launch_slow_recompute(c, (cudaStream_t)stream, p, c->user_sumsq ? c->user_sumsq : c->d_sumsq);
        if (st2 != GXPO_OK) { c->t_opt -= 1; return st2; }
        c->state_lag = 0;
        c->phase = SLOW_DONE;
        return GXPO_OK;
    }
    if (c->state_lag) {
        p.replay = 1;
        p.gscale_r0 = c->gscale[0];
        p.gscale_r1 = c->gscale[1];
    }
    const bool want_dot = c->diag_on && !c->gslow_aliased && c->num_chunks > 0;
    const bool dot_inside = want_dot && !p.replay && step_runs_staged(c, p, c->num_chunks);
    gxpo_status st = launch_step(c, (cudaStream_t)stream, c->d_descs, c->d_chunks, c->num_chunks, none, p,
                                 c->user_sumsq ? c->user_sumsq : c->d_sumsq, dot_inside ? c->d_diag + kDiagN : nullptr);
    if (st != GXPO_OK) { c->t_opt -= 1; return st; }
    c->state_lag = 0;
    if (want_dot && !dot_inside) {
        const bool bf16 = c->grad_dtype == GXPO_BF16;
        long long g = (long long)c->sm_count * 4;        // what fits at 64 registers: 32 warps per SM, one chunk each at a time
        if (g * (kThreads / 32) > c->num_chunks) g = (c->num_chunks + kThreads / 32 - 1) / (kThreads / 32);
        if (bf16) dot_kernel<uint16_t><<<(int)g, kThreads, 0, (cudaStream_t)stream>>>(c->d_descs, c->d_chunks, c->num_chunks, 0, 2, c->d_partials, c->d_ticket, c->d_diag + kDiagN);
        else      dot_kernel<float><<<(int)g, kThreads, 0, (cudaStream_t)stream>>>(c->d_descs, c->d_chunks, c->num_chunks, 0, 2, c->d_partials, c->d_ticket, c->d_diag + kDiagN);
        c->launches += 1;
        CUDA_TRY(c, cudaGetLastError());
        c->last_sweep.bytes_read_per_param += 2 * grad_bytes(c);   // the extra pass reads g0 and g_slow
        c->last_sweep.extra_launches = 1;
    }
    c->phase = SLOW_DONE;
    return GXPO_OK;
}

gxpo_status gxpo_gate_update(gxpo_ctx* c, void* stream, gxpo_gate_result* out) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != SLOW_DONE) return fail(c, GXPO_ERR_STATE, "gate update must follow the slow step");
    c->phase = IDLE;
    c->diag_ready = c->diag_on;
    expire_clips(c);
    return run_gate(c, (cudaStream_t)stream, c->user_sumsq ? c->user_sumsq : c->d_sumsq, out);
}

gxpo_status gxpo_gate_update_async(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != SLOW_DONE) return fail(c, GXPO_ERR_STATE, "gate update must follow the slow step");
    gxpo_status st = finish_gate(c);
    if (st != GXPO_OK) return st;
    c->phase = IDLE;
    c->diag_ready = c->diag_on;
    expire_clips(c);
    return launch_gate(c, (cudaStream_t)stream, c->user_sumsq ? c->user_sumsq : c->d_sumsq);
}

gxpo_status gxpo_gate_last(gxpo_ctx* c, gxpo_gate_result* out) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    { gxpo_status fe = collect_fallback_error(c); if (fe != GXPO_OK) return fe; }
    gxpo_status st = finish_gate(c);
    if (st != GXPO_OK) return st;
    if (!c->have_gate) return fail(c, GXPO_ERR_STATE, "no gate update has run yet");
    return gate_outcome(c, out);
}

gxpo_status gxpo_set_sumsq_buffer(gxpo_ctx* c, double* sumsq_dev) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase == SLOW_DONE) return fail(c, GXPO_ERR_STATE, "a norm is pending: call gxpo_gate_update first");
    if (((uintptr_t)sumsq_dev) & 7u) return fail(c, GXPO_ERR_ALIGNMENT, "sumsq buffer must be 8-byte aligned");
    c->user_sumsq = sumsq_dev;
    return GXPO_OK;
}

gxpo_status gxpo_set_grad_scale(gxpo_ctx* c, int which, const float* scale_dev) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (which < 0 || which > 2) return fail(c, GXPO_ERR_INVALID_ARG, "which must be 0 (g0), 1 (g1) or 2 (g_slow)");
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "gradient scales can only be changed between steps");
    if (((uintptr_t)scale_dev) & 3u) return fail(c, GXPO_ERR_ALIGNMENT, "scale pointer must be 4-byte aligned");
    c->gscale[which] = scale_dev;
    c->user_gscale[which] = scale_dev;
    return GXPO_OK;
}

gxpo_status gxpo_clip_grad_norm(gxpo_ctx* c, int which, double max_norm, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (which < 0 || which > 2) return fail(c, GXPO_ERR_INVALID_ARG, "which must be 0 (g0), 1 (g1) or 2 (g_slow)");
    if (!(max_norm > 0.0) || !std::isfinite(max_norm)) return fail(c, GXPO_ERR_INVALID_ARG, "max_norm must be finite and > 0");
    if (!c->bound) return fail(c, GXPO_ERR_STATE, "nothing bound: call gxpo_bind first");
    // legal exactly where the sweep that consumes this gradient is the next one to run
    const bool ok = (which == 0 && c->phase == IDLE) ||
                    (which == 1 && (c->phase == PROBED0 || c->phase == PROBED0_DEFERRED)) ||
                    (which == 2 && c->phase == EXTRAPOLATED);
    if (!ok) return fail(c, GXPO_ERR_STATE, "clip the gradient right before the sweep that consumes it");
    cudaStream_t s = (cudaStream_t)stream;
    if (c->num_chunks > 0) {
        long long g = (long long)c->sm_count * 4;        // what fits at 64 registers: 32 warps per SM, one chunk each at a time
        if (g * (kThreads / 32) > c->num_chunks) g = (c->num_chunks + kThreads / 32 - 1) / (kThreads / 32);
        if (c->grad_dtype == GXPO_BF16)
            dot_kernel<uint16_t><<<(int)g, kThreads, 0, s>>>(c->d_descs, c->d_chunks, c->num_chunks, which, which, c->d_partials, c->d_ticket, c->d_gnorm + which);
        else
            dot_kernel<float><<<(int)g, kThreads, 0, s>>>(c->d_descs, c->d_chunks, c->num_chunks, which, which, c->d_partials, c->d_ticket, c->d_gnorm + which);
        c->launches += 1;
        CUDA_TRY(c, cudaGetLastError());
    } else {
        CUDA_TRY(c, cudaMemsetAsync(c->d_gnorm + which, 0, sizeof(double), s));
    }
    clip_coef_kernel<<<1, 32, 0, s>>>(c->d_gnorm + which, max_norm, c->d_clip + which, c->d_gnorm + 3 + which);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    note_sweep(c, "dot_kernel", 0, 0, grad_bytes(c), 0);
    c->last_sweep.extra_launches = 1;                       // the coefficient kernel
    if (c->phase == IDLE) { gxpo_status ms = mark_idle_work(c, s); if (ms != GXPO_OK) return ms; }
    c->gscale[which] = c->d_clip + which;
    return GXPO_OK;
}

gxpo_status gxpo_enable_diagnostics(gxpo_ctx* c, int on) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "diagnostics can only be switched between steps");
    c->diag_on = on ? 1 : 0;
    c->diag_ready = 0;
    return GXPO_OK;
}

gxpo_status gxpo_set_gradients_persist(gxpo_ctx* c, int on) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "the promise can only be changed between steps");
    c->grads_persist = on ? 1 : 0;
    return GXPO_OK;
}

gxpo_status gxpo_get_diagnostics(gxpo_ctx* c, void* stream, gxpo_diagnostics* out) {
    if (!c || !out) return GXPO_ERR_INVALID_ARG;
    if (c->phase != IDLE || !c->diag_ready)
        return fail(c, GXPO_ERR_STATE, "no diagnostics: enable them, then complete an active step through gxpo_gate_update");
    cudaStream_t s = (cudaStream_t)stream;
    diag_finalize_kernel<<<1, 32, 0, s>>>(c->d_diag, c->user_sumsq ? c->user_sumsq : c->d_sumsq, c->total_params,
                                          c->gslow_aliased ? 0 : 1, c->d_diag_result);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    CUDA_TRY(c, cudaMemcpyAsync(c->h_diag_result, c->d_diag_result, sizeof(DiagResult), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(c, cudaStreamSynchronize(s));
    const DiagResult r = *c->h_diag_result;
    out->g0_norm = r.g0_norm; out->g1_norm = r.g1_norm; out->gslow_norm = r.gslow_norm;
    out->cos_g0_gslow = r.cos_g0_gslow; out->ratio_mean = r.ratio_mean; out->ratio_std = r.ratio_std;
    out->scale_mean = r.scale_mean; out->disp_ratio = r.disp_ratio; out->inactive_frac = r.inactive_frac;
    out->n = r.n; out->n_active = r.n_active; out->n_irregular = r.n_irregular;
    return GXPO_OK;
}

gxpo_status gxpo_selftest_bounded_wait(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "self-test in the middle of a step");
    cudaStream_t s = (cudaStream_t)stream;
    bounded_wait_probe_kernel<<<1, 32, 0, s>>>(4096u, c->d_err);
    c->launches += 1;
    CUDA_TRY(c, cudaGetLastError());
    int err = 0;
    CUDA_TRY(c, cudaMemcpyAsync(&err, c->d_err, sizeof(int), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(c, cudaStreamSynchronize(s));
    CUDA_TRY(c, cudaMemsetAsync(c->d_err, 0, sizeof(int), s));
    CUDA_TRY(c, cudaStreamSynchronize(s));
    if (err) return fail(c, GXPO_ERR_TIMEOUT, "self-test: the wait on a barrier nobody completes gave up, as it must");
    return GXPO_OK;
}

gxpo_status gxpo_selftest_inject_timeout(gxpo_ctx* c, void* stream) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    CUDA_TRY(c, cudaMemsetAsync(c->d_err, 1, sizeof(int), s));      // any non-zero word means "a wait gave up"
    return GXPO_OK;
}

gxpo_status gxpo_last_sweep(const gxpo_ctx* c, gxpo_sweep_info* out) {
    if (!c || !out) return GXPO_ERR_INVALID_ARG;
    if (!c->last_sweep.valid) return fail(const_cast<gxpo_ctx*>(c), GXPO_ERR_STATE, "no sweep has been launched yet");
    *out = c->last_sweep;
    return GXPO_OK;
}

gxpo_status gxpo_gate_peek(const gxpo_ctx* c, int* active, long long* s_star, long long* t) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    { gxpo_status fe = collect_fallback_error(const_cast<gxpo_ctx*>(c)); if (fe != GXPO_OK) return fe; }
    { gxpo_status fg = finish_gate(const_cast<gxpo_ctx*>(c)); if (fg != GXPO_OK) return fg; }
    if (active) *active = gate_active(c) ? 1 : 0;
    if (s_star) *s_star = c->s_star;
    if (t) *t = c->t;
    return GXPO_OK;
}

long long gxpo_optimizer_steps(const gxpo_ctx* c) { return c ? c->t_opt : -1; }

long long gxpo_backward_passes(const gxpo_ctx* c) {
    if (!c) return -1;
    if (finish_gate(const_cast<gxpo_ctx*>(c)) != GXPO_OK) return -1;
    const long long s = (c->s_star < 0 || c->s_star > c->t) ? c->t : c->s_star;
    return 3 * s + (c->t - s);
}

long long gxpo_launch_count(const gxpo_ctx* c) { return c ? c->launches : -1; }

const char* gxpo_last_error(const gxpo_ctx* c) { return c ? c->err : "null context"; }

const char* gxpo_status_string(gxpo_status s) {
    switch (s) {
        case GXPO_OK: return "ok";
        case GXPO_ERR_INVALID_ARG: return "invalid argument";
        case GXPO_ERR_ALIGNMENT: return "misaligned pointer";
        case GXPO_ERR_STATE: return "call out of order";
        case GXPO_ERR_CUDA: return "CUDA error";
        case GXPO_ERR_TIMEOUT: return "device-side wait timed out";
        case GXPO_ERR_NONFINITE: return "non-finite gradient norm";
    }
    return "unknown status";
}

gxpo_status gxpo_tune(gxpo_ctx* c, int ctas_per_sm, int variant, int unit_tiles) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (ctas_per_sm < 0 || ctas_per_sm > 16) return fail(c, GXPO_ERR_INVALID_ARG, "ctas_per_sm must be in [0, 16]");
    if (variant < 0 || variant > 3) return fail(c, GXPO_ERR_INVALID_ARG, "variant must be 0, 1, 2 or 3");
    int ush = -1;
    const bool auto_unit = unit_tiles == 0;
    if (auto_unit) ush = 0;
    for (int k = 0; k <= 4; ++k) if (unit_tiles == (kTilesPerChunk >> k)) ush = k;
    if (ush < 0) return fail(c, GXPO_ERR_INVALID_ARG, "unit_tiles must be 0, 1, 2, 4, 8 or 16");
    c->ctas_per_sm = ctas_per_sm;
    c->variant = variant;
    c->unit_shift = auto_unit ? -1 : ush;
    return GXPO_OK;
}

// ---- small-state checkpoint -------------------------------------------------
namespace {
struct StateHeader {
    unsigned magic, version;
    int window, head, count, pad;
    long long t, s_star, t_opt;
};
constexpr unsigned kMagic = 0x4F505847u;   // "GXPO"
}  // namespace

gxpo_status gxpo_state_export(gxpo_ctx* c, void* buf, size_t* len) {
    if (!c || !len) return GXPO_ERR_INVALID_ARG;
    const size_t need = sizeof(StateHeader) + (size_t)c->cfg.window * sizeof(double);
    if (!buf) { *len = need; return GXPO_OK; }
    if (*len < need) { *len = need; return fail(c, GXPO_ERR_INVALID_ARG, "buffer too small: need %zu bytes", need); }
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "state export in the middle of a step");
    { gxpo_status fe = collect_fallback_error(c); if (fe != GXPO_OK) return fe; }
    { gxpo_status ws = wait_idle(c); if (ws != GXPO_OK) return ws; }
    GateState g;
    CUDA_TRY(c, cudaMemcpyAsync(&g, c->d_gate, sizeof(g), cudaMemcpyDeviceToHost, c->copy_stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->copy_stream));
    StateHeader h;
    std::memset(&h, 0, sizeof(h));
    h.magic = kMagic; h.version = 1; h.window = c->cfg.window; h.head = g.head; h.count = g.count;
    h.t = c->t; h.s_star = c->s_star; h.t_opt = c->t_opt;
    std::memcpy(buf, &h, sizeof(h));
    CUDA_TRY(c, cudaMemcpyAsync(static_cast<char*>(buf) + sizeof(h), c->d_ring, (size_t)c->cfg.window * sizeof(double), cudaMemcpyDeviceToHost, c->copy_stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->copy_stream));
    *len = need;
    return GXPO_OK;
}

gxpo_status gxpo_state_import(gxpo_ctx* c, const void* buf, size_t len) {
    if (!c || !buf) return GXPO_ERR_INVALID_ARG;
    const size_t need = sizeof(StateHeader) + (size_t)c->cfg.window * sizeof(double);
    if (len < need) return fail(c, GXPO_ERR_INVALID_ARG, "state blob too short");
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "state import in the middle of a step");
    { gxpo_status fg = finish_gate(c); if (fg != GXPO_OK) return fg; }
    StateHeader h;
    std::memcpy(&h, buf, sizeof(h));
    if (h.magic != kMagic || h.version != 1) return fail(c, GXPO_ERR_INVALID_ARG, "not a GXPO state blob");
    if (h.window != c->cfg.window) return fail(c, GXPO_ERR_INVALID_ARG, "window mismatch: blob %d, context %d", h.window, c->cfg.window);
    if (h.head < 0 || h.head >= h.window || h.count < 0 || h.count > h.window || h.t < 0 || h.t_opt < 0 || h.s_star < -1)
        return fail(c, GXPO_ERR_INVALID_ARG, "corrupt state blob");
    { gxpo_status ws = wait_idle(c); if (ws != GXPO_OK) return ws; }
    GateState g;
    g.head = h.head; g.count = h.count; g.s_star = h.s_star;
    CUDA_TRY(c, cudaMemcpyAsync(c->d_gate, &g, sizeof(g), cudaMemcpyHostToDevice, c->copy_stream));
    CUDA_TRY(c, cudaMemcpyAsync(c->d_ring, static_cast<const char*>(buf) + sizeof(h), (size_t)c->cfg.window * sizeof(double), cudaMemcpyHostToDevice, c->copy_stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->copy_stream));
    c->t = h.t; c->s_star = h.s_star; c->t_opt = h.t_opt;
    return GXPO_OK;
}

// ---- host-resident parameters ------------------------------------------------
gxpo_status gxpo_step_host(gxpo_ctx* c, const gxpo_tensor* list, int count, long long staging_elems,
                           void* stream, gxpo_gate_result* out) {
    if (!c) return GXPO_ERR_INVALID_ARG;
    if (count < 0 || (count > 0 && !list)) return fail(c, GXPO_ERR_INVALID_ARG, "bad list/count");
    if (c->phase != IDLE) return fail(c, GXPO_ERR_STATE, "host step in the middle of a device step");
    { gxpo_status fg = finish_gate(c); if (fg != GXPO_OK) return fg; }
    if (staging_elems <= 0) staging_elems = 1LL << 24;
    staging_elems = (staging_elems + kChunk - 1) / kChunk * kChunk;
    for (int i = 0; i < count; ++i) {
        gxpo_status s = check_tensor(c, list[i], i, false);
        if (s != GXPO_OK) return s;
    }
    gxpo_status s0 = ensure_staging(c, staging_elems);
    if (s0 != GXPO_OK) return s0;
    Staging& st = c->stg;
    cudaStream_t user = (cudaStream_t)stream;
    const bool adamw = c->opt.kind == GXPO_OPT_ADAMW;
    const bool active = gate_active(c);
    const size_t gsz = (c->grad_dtype == GXPO_BF16) ? 2 : 4;
    CUDA_TRY(c, cudaStreamSynchronize(user));
    CUDA_TRY(c, cudaMemsetAsync(st.piece_sumsq, 0, 2 * sizeof(double), st.stream[0]));
    CUDA_TRY(c, cudaStreamSynchronize(st.stream[0]));
    const long long t_opt0 = c->t_opt;
    int piece = 0;
    for (int i = 0; i < count; ++i) {
        const gxpo_tensor& T = list[i];
        for (long long off = 0; off < T.n; off += staging_elems, ++piece) {
            const long long len = (T.n - off < staging_elems) ? (T.n - off) : staging_elems;
            const int k = piece & 1;
            cudaStream_t s = st.stream[k];
            // the slot is free once its previous piece has been copied back (same stream)
            const size_t fb = (size_t)len * sizeof(float);
            CUDA_TRY(c, cudaMemcpyAsync(st.theta[k], T.theta + off, fb, cudaMemcpyHostToDevice, s));
            if (adamw) {
                CUDA_TRY(c, cudaMemcpyAsync(st.m[k], T.m + off, fb, cudaMemcpyHostToDevice, s));
                CUDA_TRY(c, cudaMemcpyAsync(st.v[k], T.v + off, fb, cudaMemcpyHostToDevice, s));
            }
            CUDA_TRY(c, cudaMemcpyAsync(st.g[k][0], static_cast<const char*>(T.g0) + off * gsz, len * gsz, cudaMemcpyHostToDevice, s));
            if (active) {
                CUDA_TRY(c, cudaMemcpyAsync(st.g[k][1], static_cast<const char*>(T.g1) + off * gsz, len * gsz, cudaMemcpyHostToDevice, s));
                CUDA_TRY(c, cudaMemcpyAsync(st.g[k][2], static_cast<const char*>(T.g_slow) + off * gsz, len * gsz, cudaMemcpyHostToDevice, s));
            }
            TensorDesc d;
            d.wb = nullptr;
            d.theta = st.theta[k]; d.work = st.work[k]; d.m = st.m[k]; d.v = st.v[k];
            d.g[0] = st.g[k][0]; d.g[1] = st.g[k][1]; d.g[2] = st.g[k][2];
            d.n = len;
            const long long nch = (len + kChunk - 1) / kChunk;
            gxpo_status rs;
            if (active) {
                // the kernels of a piece run back to back on the slot's stream; the
                // norm's scratch is shared, which is safe because both slots' kernels
                // are serialised through the `done` events below
                if (piece > 0) CUDA_TRY(c, cudaStreamWaitEvent(s, st.done[k ^ 1], 0));
                c->t_opt = t_opt0 + 1;
                rs = launch_step(c, s, nullptr, nullptr, nch, d, make_step_params(c, 0, 0, 1, 0, 0), c->d_sumsq);
                if (rs != GXPO_OK) return rs;
                c->t_opt = t_opt0 + 2;
                FusedParams fp;
                fp.step0 = make_step_params(c, 0, 0, 0, 0, 0);
                fp.step = make_step_params(c, 1, 1, 1, 0, 0);
                fp.ex = make_extrap_params(c, GXPO_PLACE_PINGPONG);
                rs = launch_fused(c, s, nullptr, nullptr, nch, d, fp, false, false);
                if (rs != GXPO_OK) return rs;
                c->t_opt = t_opt0 + 3;
                rs = launch_step(c, s, nullptr, nullptr, nch, d, make_step_params(c, 2, 0, 0, 0, 1), st.piece_sumsq + 1);
                if (rs != GXPO_OK) return rs;
                accumulate_kernel<<<1, 32, 0, s>>>(st.piece_sumsq, st.piece_sumsq + 1);
                c->launches += 1;
                CUDA_TRY(c, cudaEventRecord(st.done[k], s));
            } else {
                c->t_opt = t_opt0 + 1;
                rs = launch_step(c, s, nullptr, nullptr, nch, d, make_step_params(c, 0, 0, 0, 0, 0), c->d_sumsq);
                if (rs != GXPO_OK) return rs;
            }
            CUDA_TRY(c, cudaMemcpyAsync(T.theta + off, st.theta[k], fb, cudaMemcpyDeviceToHost, s));
            if (adamw) {
                CUDA_TRY(c, cudaMemcpyAsync(T.m + off, st.m[k], fb, cudaMemcpyDeviceToHost, s));
                CUDA_TRY(c, cudaMemcpyAsync(T.v + off, st.v[k], fb, cudaMemcpyDeviceToHost, s));
            }
        }
    }
    CUDA_TRY(c, cudaStreamSynchronize(st.stream[0]));
    CUDA_TRY(c, cudaStreamSynchronize(st.stream[1]));
    if (active) {
        c->t_opt = t_opt0 + 3;
        return run_gate(c, st.stream[0], st.piece_sumsq, out);
    }
    c->t_opt = t_opt0 + 1;
    c->t += 1;
    if (out) {
        out->active = 0; out->tripped = 0; out->t = c->t; out->s_star = c->s_star;
        out->norm = out->z = out->mu = out->sigma = std::nan("");
    }
    // no gate kernel ran: collect the error word of the staged sweeps here
    { gxpo_status es = enqueue_error_readback(c, st.stream[0], c->t - 1); if (es != GXPO_OK) return es; }
    return collect_fallback_error(c);
}

// ---- surrogate harness ---------------------------------------------------------
gxpo_status gxpo_quad_grad(const float* theta, const float* a, const float* b, float* g, long long n, void* stream) {
    if (n < 0 || (n > 0 && (!theta || !a || !b || !g))) return GXPO_ERR_INVALID_ARG;
    if (n == 0) return GXPO_OK;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long long want = (n / 8 + kThreads - 1) / kThreads;
    long long grid = (long long)sms * 8;
    if (grid > want) grid = want < 1 ? 1 : want;
    quad_grad_kernel<<<(int)grid, kThreads, 0, (cudaStream_t)stream>>>(theta, a, b, g, n);
    return cudaGetLastError() == cudaSuccess ? GXPO_OK : GXPO_ERR_CUDA;
}

size_t gxpo_quad_scratch_bytes(void) { return kMaxGrid * sizeof(double) + 64; }

gxpo_status gxpo_quad_active_step(float* theta, const float* a, const float* b, long long n, float lr, int K,
                                  float alpha, float delta, float den_eps, double* sumsq_dev,
                                  void* scratch_dev, void* stream) {
    if (n < 0 || K < 2 || !sumsq_dev || !scratch_dev || (n > 0 && (!theta || !a || !b))) return GXPO_ERR_INVALID_ARG;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long long want = (n / 8 + kThreads - 1) / kThreads;
    long long grid = (long long)sms * 8;
    if (grid > want) grid = want < 1 ? 1 : want;
    if (grid > kMaxGrid) grid = kMaxGrid;
    QuadParams q;
    q.lr = lr; q.alpha = alpha; q.delta = delta; q.den_eps = den_eps; q.K = K;
    double* partials = static_cast<double*>(scratch_dev);
    unsigned* ticket = reinterpret_cast<unsigned*>(static_cast<char*>(scratch_dev) + kMaxGrid * sizeof(double));
    quad_active_kernel<<<(int)grid, kThreads, 0, (cudaStream_t)stream>>>(theta, a, b, n, q, partials, ticket, sumsq_dev);
    return cudaGetLastError() == cudaSuccess ? GXPO_OK : GXPO_ERR_CUDA;
}

}  // extern "C"

// ---- allocation-free slow step ----------------------------------------------------
// Everything this entry point needs lives in this file: the scratch array, the variant
// of the OptimStep sweep that writes one partial sum per chunk into it, the per-device
// set-up that turns the array's name into a device address, and the entry point.
namespace {

constexpr long long kNoAllocMaxChunks = GXPO_NOALLOC_MAX_PARAMS / kChunk;   // 65536
constexpr size_t kNoAllocPartialBytes = (size_t)kNoAllocMaxChunks * sizeof(double);
constexpr int kNoAllocMaxDevices = 64;

// One float64 partial per 32768-element chunk (512 KB), then the ticket counter in a
// 256-byte cell of its own.  Held by every device that loads the library, until exit.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocPartialBytes + 256];

// The OptimStep sweep over one flat buffer with sum(g^2) reduced per chunk: each chunk's
// partial lands in its own slot and the last CTA to finish adds the slots in index
// order, so the sum depends on n alone and not on how many CTAs ran.
template <bool ADAMW, typename G>
__global__ void __launch_bounds__(kThreads)
step_flat_perchunk_kernel(TensorDesc d, long long num_chunks, StepParams p, double* partials,
                          unsigned* ticket, double* sumsq_out) {
    __shared__ double red[8];
    for (long long c = blockIdx.x; c < num_chunks; c += gridDim.x) {
        const long long off = c * kChunk;
        const long long rem = d.n - off;
        const int len = rem < kChunk ? (int)rem : kChunk;
        float* th = d.theta + off;
        float* m = ADAMW ? d.m + off : nullptr;
        float* v = ADAMW ? d.v + off : nullptr;
        const G* g = reinterpret_cast<const G*>(d.g[2]) + off;
        const bool vec = aligned32(th) && aligned32(g) && (!ADAMW || (aligned32(m) && aligned32(v)));
        double acc = 0.0;
        if (vec) step_chunk_vec<ADAMW, G, 8>(th, th, nullptr, m, v, g, len, p, 1.0f, acc);
        else     step_chunk_scalar<ADAMW, G>(th, th, nullptr, m, v, g, len, p, 1.0f, acc);
        const double tot = block_sum(acc, red);
        if (threadIdx.x == 0) partials[c] = tot;
    }
    __shared__ bool is_last;
    if (threadIdx.x == 0) {
        __threadfence();
        is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (is_last) {
        __threadfence();
        double s = 0.0;
        for (long long i = threadIdx.x; i < num_chunks; i += kThreads) s += __ldcg(partials + i);
        s = block_sum(s, red);
        if (threadIdx.x == 0) {
            *sumsq_out = s;
            *ticket = 0u;
        }
    }
}

struct NoAllocDevice {
    bool ready;
    unsigned char* scratch;    // device address of g_noalloc_scratch on this device
    int sm_count;
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;

gxpo_status noalloc_fail(char* buf, size_t len, gxpo_status s, const char* fmt, ...) {
    if (buf && len > 0) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, len, fmt, ap);
        va_end(ap);
    }
    return s;
}

}  // namespace

extern "C" gxpo_status gxpo_slow_step_noalloc(float* theta, float* m, float* v, const void* g_slow,
                                              long long n, int grad_dtype, const gxpo_opt_cfg* opt,
                                              long long t_opt, double* sumsq_dev, void* stream,
                                              char* errbuf, size_t errbuf_len) {
    if (errbuf && errbuf_len > 0) errbuf[0] = '\0';
    if (!opt || !sumsq_dev) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "opt and sumsq_dev must not be null");
    if (grad_dtype != GXPO_F32 && grad_dtype != GXPO_BF16) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "unknown gradient dtype %d", grad_dtype);
    if (opt->kind != GXPO_OPT_GD && opt->kind != GXPO_OPT_ADAMW) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "unknown optimizer kind %d", opt->kind);
    const bool adamw = opt->kind == GXPO_OPT_ADAMW;
    if (!std::isfinite(opt->lr)) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "lr is not finite");
    if (adamw) {
        if (!(opt->beta1 >= 0.0 && opt->beta1 < 1.0) || !(opt->beta2 >= 0.0 && opt->beta2 < 1.0))
            return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "betas must be in [0, 1)");
        if (!(opt->eps >= 0.0) || !std::isfinite(opt->eps) || !std::isfinite(opt->weight_decay))
            return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "eps must be finite and >= 0, weight_decay finite");
        if (t_opt < 1) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "t_opt counts this step and must be >= 1, got %lld", t_opt);
    }
    if (n < 0) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "n < 0");
    if (n > GXPO_NOALLOC_MAX_PARAMS)
        return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG,
                            "n = %lld exceeds GXPO_NOALLOC_MAX_PARAMS = %lld (the built-in scratch holds one partial sum per %d parameters); "
                            "split the buffer and add the sums, or use a context", n, (long long)GXPO_NOALLOC_MAX_PARAMS, kChunk);
    if (((uintptr_t)sumsq_dev) & 7u) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_ALIGNMENT, "sumsq_dev must be 8-byte aligned");
    if (n > 0) {
        if (!theta || !g_slow || (adamw && (!m || !v)))
            return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "null theta/m/v/g_slow pointer");
        const uintptr_t gmask = (grad_dtype == GXPO_BF16) ? 1u : 3u;
        if ((((uintptr_t)theta) & 3u) || (((uintptr_t)m) & 3u) || (((uintptr_t)v) & 3u) || (((uintptr_t)g_slow) & gmask))
            return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_ALIGNMENT, "a pointer is not aligned to its element size");
    }
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;

    // Per-device set-up, first call on each device: in host code the array's name is only
    // a handle, so ask the runtime for its address on the current device and keep it.
    int dev = -1;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kNoAllocMaxDevices) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_INVALID_ARG, "device ordinal %d out of range", dev);
    NoAllocDevice nd;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_dev[dev].ready) {
            void* ptr = nullptr;
            e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
            if (e != cudaSuccess || !ptr)
                return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_CUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            int sms = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess || sms < 1)
                return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_CUDA, "cudaDeviceGetAttribute failed: %s", cudaGetErrorString(e));
            g_noalloc_dev[dev].scratch = static_cast<unsigned char*>(ptr);
            g_noalloc_dev[dev].sm_count = sms;
            g_noalloc_dev[dev].ready = true;
        }
        nd = g_noalloc_dev[dev];
    }
    double* partials = reinterpret_cast<double*>(nd.scratch);
    unsigned* ticket = reinterpret_cast<unsigned*>(nd.scratch + kNoAllocPartialBytes);

    if (n == 0) {
        e = cudaMemsetAsync(sumsq_dev, 0, sizeof(double), s);
        if (e != cudaSuccess) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_CUDA, "cudaMemsetAsync failed: %s", cudaGetErrorString(e));
        return GXPO_OK;
    }
    // The array keeps whatever the last call left: the counter must start at zero (an
    // earlier call that failed to launch could have left it mid-count); the partial slots
    // need no clearing because every slot that is read is written first.
    e = cudaMemsetAsync(ticket, 0, sizeof(unsigned), s);
    if (e != cudaSuccess) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_CUDA, "cudaMemsetAsync failed: %s", cudaGetErrorString(e));

    StepParams p;
    std::memset(&p, 0, sizeof(p));
    p.which_grad = 2;
    p.want_norm = 1;
    p.write_state = 1;
    p.lr = (float)opt->lr;
    if (adamw) {
        const double t = (double)t_opt, b1 = opt->beta1, b2 = opt->beta2, lr = opt->lr;
        p.beta1 = (float)b1;
        p.beta2 = (float)b2;
        p.omb1 = (float)(1.0 - b1);
        p.omb2 = (float)(1.0 - b2);
        p.eps = (float)opt->eps;
        p.decay = (float)(1.0 - lr * opt->weight_decay);
        p.step_size = (float)(lr / (1.0 - std::pow(b1, t)));
        p.inv_sqrt_bc2 = (float)(1.0 / std::sqrt(1.0 - std::pow(b2, t)));
    }
    fill_step_pairs(p);
    TensorDesc d;
    std::memset(&d, 0, sizeof(d));
    d.theta = theta; d.m = m; d.v = v; d.g[2] = g_slow; d.n = n;
    const long long num_chunks = (n + kChunk - 1) / kChunk;
    long long grid = (long long)nd.sm_count * kDefaultCtasStep;
    if (grid > num_chunks) grid = num_chunks;
    const bool bf16 = grad_dtype == GXPO_BF16;
    if (adamw) {
        if (bf16) step_flat_perchunk_kernel<true, uint16_t><<<(int)grid, kThreads, 0, s>>>(d, num_chunks, p, partials, ticket, sumsq_dev);
        else      step_flat_perchunk_kernel<true, float><<<(int)grid, kThreads, 0, s>>>(d, num_chunks, p, partials, ticket, sumsq_dev);
    } else {
        if (bf16) step_flat_perchunk_kernel<false, uint16_t><<<(int)grid, kThreads, 0, s>>>(d, num_chunks, p, partials, ticket, sumsq_dev);
        else      step_flat_perchunk_kernel<false, float><<<(int)grid, kThreads, 0, s>>>(d, num_chunks, p, partials, ticket, sumsq_dev);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return noalloc_fail(errbuf, errbuf_len, GXPO_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return GXPO_OK;
}
