// Host-side schedule of Local OPT: learning rate eta_t and round length H (Sec. 2, Eq. 2 of arXiv 2310.14423).
// Pure binary64 host arithmetic; no CUDA in this file.  The integer H is decided here and nowhere else, so the
// order of the floating-point operations below is part of the library's contract (it is spelled out in qsr.h).
#include <cmath>
#include <cstdint>
#include <initializer_list>
#include <limits>

#include "../../include/qsr.h"
#include "internal.h"

namespace qsr {

static bool finite_all(std::initializer_list<double> xs)
{
    for (double x : xs)
        if (!std::isfinite(x)) return false;
    return true;
}

// Rows that start on a large power-of-two boundary stream measurably faster on B200 (see qsr.h): align to 2^a floats
// with a = min(20, floor(log2 P) - 4), so that the padding stays below P/16; short rows are only rounded up to 4.
int64_t row_stride_hint(int64_t P)
{
    int log2p = 0;
    while ((int64_t(2) << log2p) <= P) ++log2p;
    int a = log2p - 4;
    if (a > 20) a = 20;
    if (a < 2) a = 2;
    const int64_t unit = int64_t(1) << a;
    return (P + unit - 1) / unit * unit;
}

int check_config(const qsr_config &c)
{
    if (c.K < 1 || c.P < 1) return QSR_EINVAL;
    if (c.opt != QSR_OPT_SGDM && c.opt != QSR_OPT_ADAMW) return QSR_EINVAL;
    if (c.sched < QSR_SCHED_COSINE || c.sched > QSR_SCHED_COSINE_HELD) return QSR_EINVAL;
    if (c.rule < QSR_RULE_QSR || c.rule > QSR_RULE_SWAP) return QSR_EINVAL;
    if (c.rule == QSR_RULE_POWER && !(std::isfinite(c.gamma) && c.gamma > 0.0)) return QSR_EINVAL;
    if ((c.rule == QSR_RULE_POST_LOCAL || c.rule == QSR_RULE_SWAP) && (c.t_switch < 0 || c.t_switch > c.T)) return QSR_ERANGE;
    if (c.sched == QSR_SCHED_HALVING && (c.t_period < 1 || c.t_hold < 0)) return QSR_ERANGE;
    if (c.sched == QSR_SCHED_COSINE_HELD && c.t_hold < c.T_warmup) return QSR_ERANGE;
    if (c.state_sync < QSR_STATE_KEEP || c.state_sync > QSR_STATE_RESET) return QSR_EINVAL;
    if (!finite_all({c.momentum, c.beta1, c.beta2, c.eps, c.weight_decay, c.eta_max, c.eta_min, c.alpha, c.noise_std}))
        return QSR_EINVAL;
    if (c.eta_max < 0.0 || c.eta_min < 0.0 || c.eta_min > c.eta_max || c.alpha < 0.0 || c.noise_std < 0.0) return QSR_EINVAL;
    if (c.opt == QSR_OPT_ADAMW && !(c.beta1 >= 0.0 && c.beta1 < 1.0 && c.beta2 >= 0.0 && c.beta2 < 1.0 && c.eps >= 0.0))
        return QSR_EINVAL;
    if (c.row_stride % 4 != 0 || c.row_stride < c.P) return QSR_EALIGN;
    if (c.T < 1 || c.T_warmup < 0 || c.T_warmup >= c.T || c.H_base < 1) return QSR_ERANGE;
    if (c.T > (int64_t(1) << 32) || c.worker_offset < 0) return QSR_ERANGE;
    if (c.t_state_origin < 0 || c.t_state_origin > c.T) return QSR_ERANGE;
    return QSR_OK;
}

// eta_t.  Warm-up is linear from eta_0 = 0 and meets eta_max at t = T_warmup; the decay then spans the remaining
// T - T_warmup steps.
double learning_rate(const qsr_config &c, int64_t t)
{
    if (t < c.T_warmup) return c.eta_max * double(t) / double(c.T_warmup);
    switch (c.sched) {
    case QSR_SCHED_CONST:
        return c.eta_max;
    case QSR_SCHED_HALVING: {
        // Peak until t_hold; the first halving takes effect at t_hold itself, the next ones every t_period steps.
        if (t < c.t_hold) return c.eta_max;
        const int64_t halvings = 1 + (t - c.t_hold) / c.t_period;
        return std::ldexp(c.eta_max, -int(halvings < 2000 ? halvings : 2000));
    }
    case QSR_SCHED_COSINE_HELD:
        if (t > c.t_hold) t = c.t_hold;   // the cosine stops decaying here
        break;
    default:
        break;
    }
    const double x = double(t - c.T_warmup) / double(c.T - c.T_warmup);
    if (c.sched == QSR_SCHED_LINEAR) return c.eta_min + (c.eta_max - c.eta_min) * (1.0 - x);
    const double pi = 3.14159265358979323846;
    const double cosine = c.eta_min + 0.5 * (c.eta_max - c.eta_min) * (1.0 + std::cos(pi * x));
    if (c.sched != QSR_SCHED_STEP_POW2) return cosine;
    // Step schedule: the cosine value with its base-2 logarithm rounded to the nearest integer.
    return cosine > 0.0 ? std::exp2(std::floor(std::log2(cosine) + 0.5)) : 0.0;
}

// Eq. 2 with its two side rules: rounds that begin in warm-up take the value Eq. 2 gives at the end of warm-up,
// and no round reaches beyond T.
int64_t round_length(const qsr_config &c, int64_t t)
{
    const int64_t left = c.T - t;
    int64_t H = c.H_base;
    switch (c.rule) {
    case QSR_RULE_POST_LOCAL:
        if (t < c.t_switch) H = 1;          // data-parallel phase: a synchronization after every step
        break;
    case QSR_RULE_SWAP:
        if (t >= c.t_switch) H = left;      // local steps only, one final averaging
        else if (c.t_switch - t < H) H = c.t_switch - t;
        break;
    case QSR_RULE_QSR:
    case QSR_RULE_POWER: {
        const double eta = learning_rate(c, t < c.T_warmup ? c.T_warmup : t);
        if (eta > 0.0) {
            const double ratio = c.alpha / eta;
            const double q = c.rule == QSR_RULE_POWER ? std::pow(ratio, c.gamma) : ratio * ratio;
            if (q < 4611686018427387904.0) {  // 2^62
                const int64_t fl = int64_t(std::floor(q));
                if (fl > H) H = fl;
            } else {
                H = left;
            }
        } else {
            H = left;  // the learning rate has reached zero: one round to the end
        }
        break;
    }
    default:
        break;
    }
    return H < left ? H : left;
}

}  // namespace qsr

extern "C" {

int qsr_config_check(const qsr_config *cfg) { return cfg ? qsr::check_config(*cfg) : QSR_EINVAL; }

int64_t qsr_row_stride_hint(int64_t P) { return P < 1 ? int64_t(QSR_EINVAL) : qsr::row_stride_hint(P); }

double qsr_config_learning_rate(const qsr_config *cfg, int64_t t)
{
    if (!cfg || qsr::check_config(*cfg) != QSR_OK || t < 0 || t >= cfg->T) return std::numeric_limits<double>::quiet_NaN();
    return qsr::learning_rate(*cfg, t);
}

int64_t qsr_config_round_length(const qsr_config *cfg, int64_t t)
{
    if (!cfg) return QSR_EINVAL;
    if (int rc = qsr::check_config(*cfg)) return rc;
    if (t < 0 || t >= cfg->T) return QSR_ERANGE;
    return qsr::round_length(*cfg, t);
}

int64_t qsr_config_schedule(const qsr_config *cfg, int64_t *round_start, int64_t *round_len, int64_t cap)
{
    if (!cfg || cap < 0 || (cap > 0 && (!round_start || !round_len))) return QSR_EINVAL;
    if (int rc = qsr::check_config(*cfg)) return rc;
    int64_t n = 0;
    for (int64_t t = 0; t < cfg->T;) {
        const int64_t H = qsr::round_length(*cfg, t);
        if (n < cap) {
            round_start[n] = t;
            round_len[n] = H;
        }
        ++n;
        t += H;
    }
    return n;
}

const char *qsr_strerror(int status)
{
    switch (status) {
    case QSR_OK: return "ok";
    case QSR_EINVAL: return "invalid argument (NULL pointer, bad count, unknown enum value or non-finite number)";
    case QSR_EALIGN: return "device pointer not 16-byte aligned, or row_stride not a multiple of 4 / smaller than P";
    case QSR_ECUDA: return "CUDA runtime error";
    case QSR_ERANGE: return "value out of range (step outside [0,T), warm-up >= T, H_base < 1, workspace too small)";
    case QSR_ESTATE: return "call out of order";
    default: return "unknown qsr status";
    }
}

}  // extern "C"
