/*
 * GXPO oracle: a plain, slow, single-threaded CPU statement of the active-phase
 * parameter update of Gradient Extrapolation-Based Policy Optimization.
 *
 * THIS IS TEST INFRASTRUCTURE. It exists to decide whether the CUDA library
 * computes what the paper states. Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it; the product library never does,
 * and the two share no code.
 *
 * Arithmetic is IEEE double throughout (build with -ffp-contract=off so that no
 * fused multiply-add changes the written order of operations).  Every array is
 * double.  Each entry point takes `round_f32`: when non-zero, every value the
 * entry point stores is rounded once to the nearest float and widened back,
 * which models a caller that keeps theta, m and v in fp32 between calls.  With
 * `round_f32 == 0` the functions are the paper's real-number formulas in double
 * and are what the closed-form pins are checked against.
 *
 * Pins (tests/test_oracle_*.py):
 *   optim_step_gd + extrapolate : closed form of Corollary 1 / Appendix A.6 on a
 *                                 diagonal quadratic, brute-force K explicit steps
 *   scale factor                : identities of Eq. (scale_factor), Eq. (geom_sum_def)
 *   optim_step_adamw            : one library AdamW step in float64, three in a row; whole
 *                                 active steps against the library optimizer with a
 *                                 hand-written closed-form reposition
 *   bf16 rounding, clip coef    : the library conversion / clipping routine
 *   l2norm                      : closed forms, a library norm
 *   gate                        : hand-built norm streams, a library mean/std,
 *                                 printed (shutoff step, total backward passes) rows
 *   active-step diagnostics     : a hand-computed example, closed forms on the diagonal
 *                                 quadratic, library mean/std/dot, degenerate cases
 * The AdamW *hyper-parameter defaults* and the gate's window, epsilon, warm-up
 * and std convention are not fixed by the paper: for those, parity is unpinned
 * (they are parameters here, never constants).
 */
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <limits>

namespace {

inline double store(double x, int round_f32) {
    return round_f32 ? static_cast<double>(static_cast<float>(x)) : x;
}

/* S_n(x) = sum_{k=0}^{n-1} x^k  -- Eq. (geom_sum_def); S_n(1) = n falls out of the sum. */
inline double geom_sum(double x, int n) {
    double s = 0.0;
    double p = 1.0;
    for (int k = 0; k < n; ++k) {
        s += p;
        p *= x;
    }
    return s;
}

}  // namespace

extern "C" {

/* ---- OptimStep, plain gradient descent (Sec. 2.1: theta_1 = theta_0 - eta g_0;
 *      Appendix A.3: theta_{n+1} = theta_n - eta g_n). ------------------------- */
void gxo_optim_step_gd(double* theta, const double* g, int64_t n, double lr, int round_f32) {
    for (int64_t i = 0; i < n; ++i) {
        theta[i] = store(theta[i] - lr * g[i], round_f32);
    }
}

/* ---- OptimStep, AdamW (Sec. 2: "AdamW in our experiments", decoupled weight
 *      decay).  `t_opt` is the optimizer's step count AFTER this step's increment
 *      (1 for the very first step); Sec. 2.3 says the two fast steps advance the
 *      optimizer state and the third step uses g_slow, so an active step calls
 *      this three times with t_opt, t_opt+1, t_opt+2.
 *        m <- b1 m + (1-b1) g ;  v <- b2 v + (1-b2) g^2
 *        theta <- theta (1 - lr wd) - lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps) */
void gxo_optim_step_adamw(double* theta, double* m, double* v, const double* g, int64_t n,
                          int64_t t_opt, double lr, double beta1, double beta2, double eps,
                          double weight_decay, int round_f32) {
    const double bc1 = 1.0 - std::pow(beta1, static_cast<double>(t_opt));
    const double bc2 = 1.0 - std::pow(beta2, static_cast<double>(t_opt));
    for (int64_t i = 0; i < n; ++i) {
        const double gi = g[i];
        const double mi = beta1 * m[i] + (1.0 - beta1) * gi;
        const double vi = beta2 * v[i] + (1.0 - beta2) * gi * gi;
        const double m_hat = mi / bc1;
        const double v_hat = vi / bc2;
        const double decayed = theta[i] * (1.0 - lr * weight_decay);
        theta[i] = store(decayed - lr * m_hat / (std::sqrt(v_hat) + eps), round_f32);
        m[i] = store(mi, round_f32);
        v[i] = store(vi, round_f32);
    }
}

/* ---- Active set, retention ratio, geometric scale, extrapolation, reposition
 *      (Algorithm 1, the block between the second fast step and backward pass 3;
 *      Eqs. (retention), (scale_factor), (k_step_position), (blend_step)).
 *
 *      per coordinate i:
 *        active      : |g0_i| > delta              (strict)
 *        r           = g1_i / g0_i                 on the active set
 *        scale       = S_K(r) / S_2(r)             on the active set, 1 elsewhere
 *        theta_K     = theta0 + (theta2 - theta0) * scale
 *        theta_tilde = theta0 + alpha * (theta_K - theta0)
 *
 *      The paper mentions denominator stabilisers without defining them.  Reading
 *      taken here: none by default (den_eps == 0 is the literal formula, so r = -1
 *      divides by zero); with den_eps > 0 a coordinate whose |S_2(r)| <= den_eps is
 *      treated like an inactive one (scale = 1).
 *      `theta_K_out` and `scale_out` may be null; they are never rounded. */
void gxo_extrapolate(double* theta_tilde, double* theta_K_out, double* scale_out,
                     const double* theta0, const double* theta2, const double* g0,
                     const double* g1, int64_t n, int K, double alpha, double delta,
                     double den_eps, int round_f32) {
    for (int64_t i = 0; i < n; ++i) {
        double scale = 1.0;
        if (std::fabs(g0[i]) > delta) {
            const double r = g1[i] / g0[i];
            const double s2 = geom_sum(r, 2);
            if (!(den_eps > 0.0 && std::fabs(s2) <= den_eps)) {
                scale = geom_sum(r, K) / s2;
            }
        }
        const double theta_K = theta0[i] + (theta2[i] - theta0[i]) * scale;
        if (theta_K_out) theta_K_out[i] = theta_K;
        if (scale_out) scale_out[i] = scale;
        theta_tilde[i] = store(theta0[i] + alpha * (theta_K - theta0[i]), round_f32);
    }
}

/* ---- ||g||_2, the quantity the gate watches (Eq. (z_score)). ------------------ */
double gxo_sum_squares(const double* g, int64_t n) {
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) s += g[i] * g[i];
    return s;
}

double gxo_l2norm(const double* g, int64_t n) { return std::sqrt(gxo_sum_squares(g, n)); }

/* ---- float32 -> bfloat16, round to nearest even: the model-weight copy a bf16 trainer
 *      runs its forward and backward passes on (the paper trains in bf16; the master
 *      parameters here are fp32).  bfloat16 is the upper 16 bits of the float32 pattern;
 *      rounding adds half of the dropped field, ties to the even 16-bit pattern; a NaN
 *      stays a (quiet) NaN.  Returns the 16-bit pattern. */
uint16_t gxo_f32_to_bf16(float x) {
    uint32_t u;
    std::memcpy(&u, &x, sizeof(u));
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

/* theta (double holding float32 values) -> bfloat16 patterns, element by element */
void gxo_round_to_bf16(const double* theta, uint16_t* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = gxo_f32_to_bf16(static_cast<float>(theta[i]));
}

/* ---- Global-norm gradient clipping (the paper's recipe: "gradient clipping at 1.0";
 *      a trainer step, not part of Algorithm 1).  The paper gives no formula; this is
 *      the trainers' usual one: every gradient is multiplied by
 *      min(1, max_norm / (||g||_2 + 1e-6)). */
double gxo_clip_coef(double norm, double max_norm) {
    const double c = max_norm / (norm + 1e-6);
    return c < 1.0 ? c : 1.0;
}

/* ---- Per-step diagnostics of the active phase, the quantities the paper's appendix
 *      tabulates ("Active-phase GXPO diagnostics": gradient norms, cos(g0, g_slow),
 *      retention ratio mean +- std, ||Delta_K|| / ||Delta_2||, scale mean, inactive
 *      fraction).  Plain definitions, two passes where a mean is needed first.
 *
 *      A coordinate is "regular" unless it is active and its ratio r or its scale
 *      factor does not fit a finite float (the update stores float32, so such a
 *      coordinate has no usable scale); irregular coordinates are counted and left out
 *      of the ratio, scale and displacement statistics.  Inactive coordinates have
 *      scale 1 and no ratio.
 *        out[0..2]  ||g0||, ||g1||, ||g_slow||           (all coordinates)
 *        out[3]     cos(g0, g_slow) = <g0, g_slow> / (||g0|| ||g_slow||)
 *        out[4..5]  mean and population std of r over regular active coordinates
 *        out[6]     mean of scale over regular coordinates (inactive ones count as 1)
 *        out[7]     ||Delta_K|| / ||Delta_2||, Delta_2 = theta2 - theta0,
 *                   Delta_K = Delta_2 * scale, over regular coordinates
 *        out[8]     inactive fraction = 1 - |A_t| / n
 *        out[9]     |A_t|;   out[10]  number of irregular coordinates              */
void gxo_active_diagnostics(const double* theta0, const double* theta2, const double* g0,
                            const double* g1, const double* g_slow, int64_t n, int K, double delta,
                            double den_eps, double* out) {
    double s00 = 0.0, s11 = 0.0, sss = 0.0, s0s = 0.0;
    double sum_r = 0.0, sum_scale = 0.0, d2 = 0.0, dk = 0.0;
    int64_t n_active = 0, n_irregular = 0, n_ratio = 0;
    for (int64_t i = 0; i < n; ++i) {
        s00 += g0[i] * g0[i];
        s11 += g1[i] * g1[i];
        sss += g_slow[i] * g_slow[i];
        s0s += g0[i] * g_slow[i];
        double scale = 1.0;
        if (std::fabs(g0[i]) > delta) {
            n_active += 1;
            const double r = g1[i] / g0[i];
            const double s2 = geom_sum(r, 2);
            if (!(den_eps > 0.0 && std::fabs(s2) <= den_eps)) scale = geom_sum(r, K) / s2;
            if (!std::isfinite(static_cast<float>(r)) || !std::isfinite(static_cast<float>(scale))) {
                n_irregular += 1;
                continue;
            }
            sum_r += r;
            n_ratio += 1;
        }
        const double d = theta2[i] - theta0[i];
        sum_scale += scale;
        d2 += d * d;
        dk += (d * scale) * (d * scale);
    }
    const double nan = std::numeric_limits<double>::quiet_NaN();
    const double mean_r = n_ratio > 0 ? sum_r / n_ratio : nan;
    double var_r = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (!(std::fabs(g0[i]) > delta)) continue;
        const double r = g1[i] / g0[i];
        double scale = 1.0;
        const double s2 = geom_sum(r, 2);
        if (!(den_eps > 0.0 && std::fabs(s2) <= den_eps)) scale = geom_sum(r, K) / s2;
        if (!std::isfinite(static_cast<float>(r)) || !std::isfinite(static_cast<float>(scale))) continue;
        var_r += (r - mean_r) * (r - mean_r);
    }
    const int64_t n_regular = n - n_irregular;
    out[0] = std::sqrt(s00);
    out[1] = std::sqrt(s11);
    out[2] = std::sqrt(sss);
    out[3] = s0s / (std::sqrt(s00) * std::sqrt(sss));
    out[4] = mean_r;
    out[5] = n_ratio > 0 ? std::sqrt(var_r / n_ratio) : nan;
    out[6] = n_regular > 0 ? sum_scale / n_regular : nan;
    out[7] = std::sqrt(dk) / std::sqrt(d2);
    out[8] = n > 0 ? 1.0 - static_cast<double>(n_active) / n : nan;
    out[9] = static_cast<double>(n_active);
    out[10] = static_cast<double>(n_irregular);
}

/* ---- Rolling z-score gate ("Adaptive rule in practice"; Algorithm 1, the block
 *      after the slow correction).
 *      Before the current norm is inserted: mu, sigma over the stored past norms
 *      (at most `window` of them), Z = (norm - mu) / (sigma + eps); Z >= tau sets
 *      s_star = t + 1, permanently.  The check runs only once the buffer holds at
 *      least `min_history` norms (Algorithm 1: more than one).  The norm is pushed
 *      whether or not the gate tripped.
 *      Not from the paper: a non-finite norm trips the gate. */
struct gxo_gate {
    double tau, eps;
    int window, min_history, ddof;
    double* buf;      /* chronological ring: buf[(head + k) % window], k = 0 oldest */
    int head, count;
    int64_t t;        /* index of the next training step */
    int64_t s_star;   /* -1 = +infinity */
};

gxo_gate* gxo_gate_create(double tau, double eps, int window, int min_history, int ddof) {
    if (window < 1 || min_history < 1 || ddof < 0) return nullptr;
    gxo_gate* g = static_cast<gxo_gate*>(std::malloc(sizeof(gxo_gate)));
    g->tau = tau;
    g->eps = eps;
    g->window = window;
    g->min_history = min_history;
    g->ddof = ddof;
    g->buf = static_cast<double*>(std::calloc(static_cast<size_t>(window), sizeof(double)));
    g->head = 0;
    g->count = 0;
    g->t = 0;
    g->s_star = -1;
    return g;
}

void gxo_gate_destroy(gxo_gate* g) {
    if (!g) return;
    std::free(g->buf);
    std::free(g);
}

/* 1 while training step g->t would run the active phase (t < s_star). */
int gxo_gate_active(const gxo_gate* g) { return (g->s_star < 0 || g->t < g->s_star) ? 1 : 0; }
int64_t gxo_gate_s_star(const gxo_gate* g) { return g->s_star; }
int64_t gxo_gate_t(const gxo_gate* g) { return g->t; }

/* End of an ACTIVE step t: consume ||g_slow||, maybe trip, push, advance t.
 * Returns 1 if this call tripped the gate.  z/mu/sigma are NaN when the check
 * did not run (warm-up). */
int gxo_gate_update(gxo_gate* g, double norm, double* z_out, double* mu_out, double* sigma_out) {
    const double nan = std::numeric_limits<double>::quiet_NaN();
    double z = nan, mu = nan, sigma = nan;
    int tripped = 0;
    if (g->count >= g->min_history && g->count > g->ddof) {
        double sum = 0.0;
        for (int k = 0; k < g->count; ++k) sum += g->buf[(g->head + k) % g->window];
        mu = sum / g->count;
        double ss = 0.0;
        for (int k = 0; k < g->count; ++k) {
            const double d = g->buf[(g->head + k) % g->window] - mu;
            ss += d * d;
        }
        sigma = std::sqrt(ss / (g->count - g->ddof));
        z = (norm - mu) / (sigma + g->eps);
        if (z >= g->tau) tripped = 1;
    }
    if (!std::isfinite(norm)) tripped = 1;
    if (tripped && g->s_star < 0) g->s_star = g->t + 1;
    /* push (outside the `if` of Algorithm 1) */
    if (g->count < g->window) {
        g->buf[(g->head + g->count) % g->window] = norm;
        g->count += 1;
    } else {
        g->buf[g->head] = norm;
        g->head = (g->head + 1) % g->window;
    }
    g->t += 1;
    if (z_out) *z_out = z;
    if (mu_out) *mu_out = mu;
    if (sigma_out) *sigma_out = sigma;
    return tripped;
}

/* End of a FALLBACK step: nothing is measured, only t advances. */
void gxo_gate_fallback_tick(gxo_gate* g) { g->t += 1; }

/* Backward passes over T steps when the gate trips at s_star (Sec. 2.3, last
 * sentence of the adaptive rule): 3 s_star + (T - s_star); 3 T if it never trips. */
int64_t gxo_backward_budget(int64_t s_star, int64_t T) {
    if (s_star < 0 || s_star > T) s_star = T;
    return 3 * s_star + (T - s_star);
}

}  /* extern "C" */
