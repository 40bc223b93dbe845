/*
 * CPU oracle for Local OPT with the Quadratic Synchronization Rule  --  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, scalar restatement of the paper's algorithm, used to check the CUDA library.
 * It is not part of the product: only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may build, load or call it, and it shares no code, header, table or constant generator with
 * the CUDA path.
 *
 * What follows which passage of the paper (arXiv 2310.14423):
 *   orc_lr            learning-rate schedule eta_t: linear warm-up from 0 to eta_max, then cosine
 *                     decay (Sec. 2 "Dealing with Learning Rate Warmup"; Sec. 4), the step schedule
 *                     2^round(log2 eta_cos(t)) and linear decay (Sec. 4, ablation on schedules).
 *   orc_round_length  Eq. 2: H = max{H_base, floor((alpha/eta_t)^2)} at the round's first global
 *                     step, the warm-up recommendation of Sec. 2 and the forced final
 *                     synchronization H := T - t; also the general power rule (gamma = 1: H ~ 1/eta,
 *                     gamma = 3: the cubic rule of App. G), the post-local schedule (Sec. 1) and the
 *                     modified SWAP schedule (App. H).
 *   orc_local_step    Eq. 1 / the inner loop of Algorithm 2: every worker applies OPT with the
 *                     learning rate of the *global* step; OPT is SGD with heavy-ball momentum and
 *                     L2 weight decay (App. C.1) or AdamW with decoupled weight decay (App. C.2).
 *   orc_sync          the All-Reduce line of Algorithm 2: the next global iterate is the mean of
 *                     the workers' local iterates, which every worker then copies.
 *   orc_parallel_step Algorithm 1 (Parallel OPT): the K gradients are taken at one point, averaged (the
 *                     All-Reduce line) and fed to one OPT step.
 *   gradient clipping inside orc_local_step: each worker's gradient scaled by min(1, c/(||g|| + 1e-6))
 *                     before OPT (App. C.2; the form is that of the paper's software).
 *   orc_run           Algorithm 2 as a whole: rounds of GetH, local steps, averaging, t += H.
 *   orc_philox4x32_10 the Philox-4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw,
 *                     "Parallel random numbers: as easy as 1, 2, 3", SC'11), and orc_noise, the
 *                     standard normal it is turned into by the Box-Muller transform.  The paper
 *                     samples mini-batches; the synthetic workload replaces fwd/bwd by a diagonal
 *                     quadratic loss plus this noise.
 *
 * Arithmetic is binary64 throughout.  Built with -DORC_REAL=float the same file gives the "mirror", a
 * yardstick for what binary32 costs on a given run: parameters, optimizer state, gradients and means
 * are STORED in binary32 and the synthetic gradient lambda*(theta - theta_star) + sigma*z is evaluated
 * in binary32 (its cancellation is the one ill-conditioned spot of the path, and it is there for any
 * implementation that keeps the gradient in fp32), while the optimizer update and the mean are
 * evaluated in binary64 from the stored values and rounded once when they are stored.  The mirror's
 * distance from the binary64 build is therefore close to the least error an fp32 path can have on that
 * run, and it is large exactly where the run is ill-conditioned.  In the binary64 build every cast to
 * `real` is a no-op.
 *
 * Parity pins (tests/test_oracle_*.py): the schedule against the communication volumes the paper
 * prints in Tables 1-3 and against threshold crossings derived by inverting the cosine; SGD against
 * the closed-form solution of the heavy-ball recurrence and against torch.optim.SGD; AdamW against
 * torch.optim.AdamW and the constant-gradient closed form; the mean against its invariants; Philox
 * against the known-answer vectors published with the generator; the normal against its moments;
 * the other rules and schedules against the 13.2 % / 14.4 % of App. G's step-decay table and against
 * threshold crossings; Algorithm 1 against torch.optim with the mean gradient and the H = 1 remark of
 * Sec. 3; clipping against torch's clip_grad_norm_; per-tensor weight decay against torch parameter groups.
 * Parity unpinned by the paper (a stated reading only): the round length used during warm-up when
 * (alpha/eta_max)^2 exceeds H_base, the warm-up's first value (eta_0 = 0), what happens to
 * optimizer state at a synchronization (kept per worker), uniform weight decay on all tensors, and the
 * exact round boundaries of the post-local and modified-SWAP schedules (the paper prints no number for them).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#ifndef ORC_REAL
#define ORC_REAL double
#endif
typedef ORC_REAL real;

enum { ORC_OPT_SGDM = 0, ORC_OPT_ADAMW = 1 };
enum { ORC_SCHED_COSINE = 0, ORC_SCHED_STEP_POW2 = 1, ORC_SCHED_LINEAR = 2, ORC_SCHED_CONST = 3,
       ORC_SCHED_HALVING = 4, ORC_SCHED_COSINE_HELD = 5 };
enum { ORC_RULE_QSR = 0, ORC_RULE_CONST_H = 1, ORC_RULE_POWER = 2, ORC_RULE_POST_LOCAL = 3, ORC_RULE_SWAP = 4 };
enum { ORC_STATE_KEEP = 0, ORC_STATE_AVERAGE = 1, ORC_STATE_RESET = 2 };

typedef struct {
    int32_t opt;
    int32_t sched;
    int32_t rule;
    int32_t state_sync;
    double momentum, beta1, beta2, eps, weight_decay;
    double eta_max, eta_min;
    double alpha;
    double noise_std;
    int64_t T, T_warmup, H_base;
    uint64_t seed;
    double gamma;            /* exponent of the power rule H = max{H_base, floor((alpha/eta)^gamma)} (Sec. 2, App. G) */
    int64_t t_switch;        /* post-local: parallel (H = 1) before it; SWAP variant: one final round after it       */
    int64_t t_hold, t_period;/* halving schedule: peak until t_hold, then halved every t_period steps (App. G);      */
                             /* held cosine: the cosine stops decaying at t_hold (App. G)                            */
    const double *wd_scale;  /* NULL, or one factor on the weight decay per column (per-tensor weight decay; the     */
                             /* paper uses one value for the whole model, App. C)                                    */
    double clip_norm;        /* > 0: global-norm gradient clipping threshold per worker (App. C.2); 0: off            */
} orc_config;

int orc_sizeof_real(void) { return (int)sizeof(real); }

/* ------------------------------------------------------------------ learning-rate schedule */

/* eta_t for t in {0, ..., T-1} (Sec. 2).  Warm-up rises linearly from eta_0 = 0 and reaches eta_max at
 * t = T_warmup; after it the schedule decays over the remaining T - T_warmup iterations. */
double orc_lr(const orc_config *c, int64_t t)
{
    const double pi = 3.14159265358979323846;
    if (t < c->T_warmup)
        return c->eta_max * (double)t / (double)c->T_warmup;
    if (c->sched == ORC_SCHED_CONST)
        return c->eta_max;
    if (c->sched == ORC_SCHED_HALVING) {
        /* App. G: "remains at its peak until [t_hold], after which it is divided by 2 every [t_period]" -- the first
         * halving happens at t_hold itself (this reading reproduces the 13.2 % and 14.4 % of the step-decay table). */
        if (t < c->t_hold)
            return c->eta_max;
        return ldexp(c->eta_max, -(int)(1 + (t - c->t_hold) / c->t_period));
    }
    if (c->sched == ORC_SCHED_COSINE_HELD && t > c->t_hold)
        t = c->t_hold;       /* the modified cosine of App. G: constant from t_hold on */
    double x = (double)(t - c->T_warmup) / (double)(c->T - c->T_warmup);
    if (c->sched == ORC_SCHED_LINEAR)
        return c->eta_min + (c->eta_max - c->eta_min) * (1.0 - x);
    double eta_cos = c->eta_min + 0.5 * (c->eta_max - c->eta_min) * (1.0 + cos(pi * x));
    if (c->sched == ORC_SCHED_COSINE || c->sched == ORC_SCHED_COSINE_HELD)
        return eta_cos;
    /* step schedule: the cosine value rounded to the nearest power of two in the exponent */
    if (eta_cos <= 0.0)
        return 0.0;
    return exp2(floor(log2(eta_cos) + 0.5));
}

/* ------------------------------------------------------------------ round length (Eq. 2) */

/* H for a round whose first global step is t.  During warm-up the rule is evaluated at the first
 * step after warm-up (Sec. 2); a round never runs past T (forced synchronization at the last step). */
int64_t orc_round_length(const orc_config *c, int64_t t)
{
    int64_t H;
    if (c->rule == ORC_RULE_CONST_H) {
        H = c->H_base;
    } else if (c->rule == ORC_RULE_POST_LOCAL) {
        /* Post-local schedule (Sec. 1): data-parallel training, i.e. H = 1, until t_switch; then a constant H. */
        H = t < c->t_switch ? 1 : c->H_base;
    } else if (c->rule == ORC_RULE_SWAP) {
        /* The modified SWAP of App. H: constant H_base until t_switch (the last such round is cut there), then
         * local steps only, with one final averaging at T. */
        if (t < c->t_switch)
            H = c->H_base < c->t_switch - t ? c->H_base : c->t_switch - t;
        else
            H = c->T - t;
    } else {
        int64_t t_eval = t < c->T_warmup ? c->T_warmup : t;
        double eta = orc_lr(c, t_eval);
        if (!(eta > 0.0)) {
            H = c->T - t;
        } else {
            double ratio = c->alpha / eta;
            double q = c->rule == ORC_RULE_POWER ? pow(ratio, c->gamma) : ratio * ratio;
            if (!(q < 4611686018427387904.0)) /* 2^62: beyond any T */
                H = c->T - t;
            else {
                H = (int64_t)floor(q);
                if (H < c->H_base)
                    H = c->H_base;
            }
        }
    }
    if (H > c->T - t)
        H = c->T - t;
    return H;
}

/* ------------------------------------------------------------------ counter-based noise */

/* Philox-4x32 with 10 rounds: 128-bit counter, 64-bit key, 128-bit output. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The two halves of the Box-Muller transform on the 23-bit fields a and b of two generator words: the
 * uniforms are u1 = (a + 1/2) / 2^23 and u2 = (b + 1/2) / 2^23, which lie strictly inside (0,1) and are
 * exact in binary32 and binary64; radius = sqrt(-2 ln u1), and the sine and cosine of the angle 2 pi u2. */
void orc_box_muller_parts(uint32_t a, uint32_t b, double *radius, double *sine, double *cosine)
{
    const double two_pi = 6.28318530717958647692;
    double u1 = ((double)a + 0.5) / 8388608.0;
    double u2 = ((double)b + 0.5) / 8388608.0;
    *radius = sqrt(-2.0 * log(u1));
    *sine = sin(two_pi * u2);
    *cosine = cos(two_pi * u2);
}

/* The same for arrays of fields: a convenience for tests that walk the whole 23-bit grid. */
void orc_box_muller_parts_fill(const uint32_t *a, const uint32_t *b, int64_t n, double *radius, double *sine, double *cosine)
{
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < n; ++c)
        orc_box_muller_parts(a[c], b[c], radius + c, sine + c, cosine + c);
}

/* Standard normal for (seed, worker k, global step u, coordinate i).
 * One Philox block serves coordinates 4j..4j+3: counter = (low(j), high(j), u, k), key = seed.
 * Words (0,1) feed the Box-Muller pair for coordinates 4j (cosine branch) and 4j+1 (sine branch),
 * words (2,3) the pair for 4j+2 and 4j+3.  Each word gives a 23-bit field (its top 23 bits). */
double orc_noise(uint64_t seed, int64_t k, int64_t u, int64_t i)
{
    uint64_t j = (uint64_t)i >> 2;
    uint32_t ctr[4] = { (uint32_t)j, (uint32_t)(j >> 32), (uint32_t)u, (uint32_t)k };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t r[4];
    orc_philox4x32_10(ctr, key, r);
    int lane = (int)(i & 3);
    uint32_t a = r[(lane >> 1) * 2] >> 9;
    uint32_t b = r[(lane >> 1) * 2 + 1] >> 9;
    double radius, sine, cosine;
    orc_box_muller_parts(a, b, &radius, &sine, &cosine);
    return (lane & 1) ? radius * sine : radius * cosine;
}

/* out[c] = orc_noise(seed, k, u, i0 + c) for c in [0, n): a convenience for statistical tests. */
void orc_noise_fill(uint64_t seed, int64_t k, int64_t u, int64_t i0, int64_t n, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < n; ++c)
        out[c] = orc_noise(seed, k, u, i0 + c);
}

/* ------------------------------------------------------------------ one local step (Eq. 1) */

/* All `rows` workers take the local step of global iteration t on the coordinates idx[0..n).
 * theta, s1, s2 are [rows, n]; row r is worker k0 + r.  idx == NULL means coordinate c is c itself.
 * grads == NULL: g = lambda*(theta - theta_star) + noise_std * z(seed, k, t, i); otherwise g = grads[r, c].
 * n_state counts the steps the optimizer state has seen before this one (bias correction uses n_state + 1).
 * With clip_norm > 0 each worker's gradient is first scaled by min(1, clip_norm / (||g||_2 + 1e-6)), the norm taken
 * over the n coordinates passed (gradient clipping of App. C.2, in the form of the paper's software); clipping
 * couples the coordinates, so it is only the algorithm's clipping when all P coordinates are passed.
 * Returns 0, or -1 if memory for one row of gradients cannot be had. */
int orc_local_step(const orc_config *c, int64_t rows, int64_t k0, int64_t n, const int64_t *idx,
                   const real *lambda, const real *theta_star,
                   real *theta, real *s1, real *s2, const real *grads,
                   int64_t t, int64_t n_state)
{
    const double eta = orc_lr(c, t);
    const double mu = c->momentum;
    const double b1 = c->beta1, b2 = c->beta2, eps = c->eps;
    const double bc1 = 1.0 - pow(c->beta1, (double)(n_state + 1));
    const double bc2 = 1.0 - pow(c->beta2, (double)(n_state + 1));
    real *g_row = (real *)malloc((size_t)(n > 0 ? n : 1) * sizeof(real));
    if (!g_row)
        return -1;
    for (int64_t r = 0; r < rows; ++r) {
        const int64_t k = k0 + r;
        /* the worker's gradient at its current parameters */
#pragma omp parallel for schedule(static)
        for (int64_t col = 0; col < n; ++col) {
            const int64_t i = idx ? idx[col] : col;
            const int64_t e = r * n + col;
            if (grads)
                g_row[col] = grads[e];
            else
                g_row[col] = lambda[col] * (theta[e] - theta_star[col]) + (real)(c->noise_std * orc_noise(c->seed, k, t, i));
        }
        double clip_coef = 1.0;
        if (c->clip_norm > 0.0) {
            double sum_sq = 0.0;
            for (int64_t col = 0; col < n; ++col)
                sum_sq += (double)g_row[col] * (double)g_row[col];
            double coef = c->clip_norm / (sqrt(sum_sq) + 1e-6);
            clip_coef = coef < 1.0 ? coef : 1.0;
        }
        /* OPT (Eq. 1) */
#pragma omp parallel for schedule(static)
        for (int64_t col = 0; col < n; ++col) {
            const int64_t e = r * n + col;
            const double wd = c->weight_decay * (c->wd_scale ? c->wd_scale[col] : 1.0);
            double g = clip_coef * (double)g_row[col];
            if (c->opt == ORC_OPT_SGDM) {
                g = g + wd * (double)theta[e];
                s1[e] = (real)(mu * (double)s1[e] + g);
                theta[e] = (real)((double)theta[e] - eta * (double)s1[e]);
            } else {
                double decayed = (double)theta[e] * (1.0 - eta * wd);
                s1[e] = (real)(b1 * (double)s1[e] + (1.0 - b1) * g);
                s2[e] = (real)(b2 * (double)s2[e] + (1.0 - b2) * g * g);
                double m_hat = (double)s1[e] / bc1;
                double denom = sqrt((double)s2[e]) / sqrt(bc2) + eps;
                theta[e] = (real)(decayed - eta * m_hat / denom);
            }
        }
    }
    free(g_row);
    return 0;
}

/* ------------------------------------------------------------------ Algorithm 1 (Parallel OPT) */

/* One iteration of the data-parallel baseline: all K workers evaluate their gradient at the SAME parameters
 * theta [n], the gradients are averaged (the All-Reduce line of Algorithm 1) and ONE optimizer step is taken with
 * the mean.  grads == NULL: worker k's gradient is lambda*(theta - theta_star) + noise_std * z(seed, k, t, i);
 * otherwise grads is [K, n].  Returns 0, or -1 if memory for the mean gradient cannot be had. */
int orc_parallel_step(const orc_config *c, int64_t K, int64_t n, const int64_t *idx,
                      const real *lambda, const real *theta_star,
                      real *theta, real *s1, real *s2, const real *grads,
                      int64_t t, int64_t n_state)
{
    real *g_mean = (real *)malloc((size_t)(n > 0 ? n : 1) * sizeof(real));
    if (!g_mean)
        return -1;
    for (int64_t col = 0; col < n; ++col) {
        const int64_t i = idx ? idx[col] : col;
        double sum = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            if (grads)
                sum += (double)grads[k * n + col];
            else
                sum += (double)lambda[col] * ((double)theta[col] - (double)theta_star[col])
                       + c->noise_std * orc_noise(c->seed, k, t, i);
        }
        g_mean[col] = (real)(sum / (double)K);
    }
    /* clipping, when on, acts on the averaged gradient, as for the paper's parallel AdamW baseline */
    int rc = orc_local_step(c, 1, 0, n, idx, lambda, theta_star, theta, s1, s2, g_mean, t, n_state);
    free(g_mean);
    return rc;
}

/* ------------------------------------------------------------------ synchronization */

static void mean_rows(int64_t rows, int64_t n, real *x)
{
#pragma omp parallel for schedule(static)
    for (int64_t col = 0; col < n; ++col) {
        double sum = 0.0;
        for (int64_t r = 0; r < rows; ++r)
            sum += (double)x[r * n + col];
        real mean = (real)(sum / (double)rows);
        for (int64_t r = 0; r < rows; ++r)
            x[r * n + col] = mean;
    }
}

/* theta_bar = (1/K) sum_k theta_k, copied back to every worker.  Optimizer state: kept per worker,
 * averaged like the parameters, or reset to zero (the caller then restarts the bias-correction count). */
void orc_sync(const orc_config *c, int64_t rows, int64_t n, real *theta, real *s1, real *s2)
{
    mean_rows(rows, n, theta);
    if (c->state_sync == ORC_STATE_AVERAGE) {
        mean_rows(rows, n, s1);
        if (c->opt == ORC_OPT_ADAMW)
            mean_rows(rows, n, s2);
    } else if (c->state_sync == ORC_STATE_RESET) {
        for (int64_t e = 0; e < rows * n; ++e) {
            s1[e] = 0;
            if (c->opt == ORC_OPT_ADAMW)
                s2[e] = 0;
        }
    }
}

/* ------------------------------------------------------------------ Algorithm 2 */

/* Runs the rounds that start in [t_begin, t_end) (t_begin must be a round start; a round that starts
 * before t_end is run to its end).  *t_state_origin is the global step at which the optimizer state was
 * last zero (0 at the start of training); it moves only in state mode RESET.  Writes the start and the
 * length of every round run, up to cap entries.  Returns the number of rounds, or -1 on bad arguments. */
int64_t orc_run(const orc_config *c, int64_t K, int64_t n, const int64_t *idx,
                const real *lambda, const real *theta_star,
                real *theta, real *s1, real *s2,
                int64_t t_begin, int64_t t_end, int64_t *t_state_origin,
                int64_t *round_start, int64_t *round_H, int64_t cap)
{
    if (K < 1 || n < 0 || t_begin < 0 || t_end > c->T || c->T_warmup >= c->T || c->H_base < 1)
        return -1;
    int64_t t = t_begin, s = 0;
    while (t < t_end) {
        int64_t H = orc_round_length(c, t);
        for (int64_t h = 0; h < H; ++h)
            if (orc_local_step(c, K, 0, n, idx, lambda, theta_star, theta, s1, s2, NULL,
                               t + h, t + h - *t_state_origin) != 0)
                return -1;
        orc_sync(c, K, n, theta, s1, s2);
        if (c->state_sync == ORC_STATE_RESET)
            *t_state_origin = t + H;
        if (s < cap) {
            round_start[s] = t;
            round_H[s] = H;
        }
        ++s;
        t += H;
    }
    return s;
}

/* The schedule alone: every (start, H) from t = 0 to T.  Returns the number of rounds. */
int64_t orc_schedule(const orc_config *c, int64_t *round_start, int64_t *round_H, int64_t cap)
{
    if (c->T_warmup >= c->T || c->H_base < 1)
        return -1;
    int64_t t = 0, s = 0;
    while (t < c->T) {
        int64_t H = orc_round_length(c, t);
        if (s < cap) {
            round_start[s] = t;
            round_H[s] = H;
        }
        ++s;
        t += H;
    }
    return s;
}
