// C ABI of the library: argument checks, host-side scalars of each step, launches.  See include/qsr.h.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "internal.h"

// A chain of step-kernel nodes that has been instantiated once and is replayed with new arguments: `n_plain` plain
// steps, then (if `fused`) the round's last step with the replica mean.
struct StepGraph {
    int n_plain;
    bool fused;
    cudaGraph_t graph;
    cudaGraphExec_t exec;
    std::vector<cudaGraphNode_t> nodes;
    qsr::StepLaunch plain, last;      // kernel instance and geometry of the plain nodes and of the fused last node
};

struct qsr_ctx {
    qsr_config cfg;
    float *theta, *s1, *s2;
    const float *lambda, *theta_star;
    cudaStream_t stream;
    int device;               // ordinal of the device that was current at qsr_init
    int sm_count;             // its number of multiprocessors
    qsr::LaunchShape shape;
    int64_t t_state_origin;
    int64_t launches;
    bool partial_pending;
    int32_t n_tensors;
    const int64_t *tensor_end;
    const float *wd_scale;
    double clip_norm;         // > 0: gradient clipping on
    float *clip_ws;           // caller's workspace for the norm partials and the factors
    int32_t graph_steps;      // > 0: qsr_run replays its launches from CUDA graphs of at most this many steps
    int32_t resident_steps;   // > 0: qsr_run packs up to this many consecutive steps into one register-resident launch
    std::vector<StepGraph> graphs;
};

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int64_t round_up4(int64_t n) { return (n + 3) & ~int64_t(3); }

int n_state_slabs(const qsr_config &c) { return c.opt == QSR_OPT_ADAMW ? 2 : 1; }

// Scalars of the local step at global iteration t (Eq. 1): everything that depends on t is evaluated here in
// binary64 and rounded to fp32 once.
qsr::StepParams step_params(const qsr_ctx &x, int64_t t, const float *grads)
{
    const qsr_config &c = x.cfg;
    qsr::StepParams p;
    std::memset(&p, 0, sizeof p);
    p.theta = x.theta; p.s1 = x.s1; p.s2 = x.s2;
    p.grads = grads; p.lambda = x.lambda; p.theta_star = x.theta_star;
    p.P = c.P; p.stride = c.row_stride; p.K = c.K;
    p.worker0 = uint32_t(c.worker_offset);
    // Philox-4x32 key schedule (Salmon et al., SC'11): the key halves advance by the Weyl constants every round
    for (uint32_t r = 0; r < 10; ++r) {
        p.round_key[2 * r] = uint32_t(c.seed) + r * 0x9E3779B9u;
        p.round_key[2 * r + 1] = uint32_t(c.seed >> 32) + r * 0xBB67AE85u;
    }
    p.step = uint32_t(t);
    p.sigma = float(c.noise_std);
    const double eta = qsr::learning_rate(c, t);
    p.eta = float(eta); p.wd = float(c.weight_decay); p.mu = float(c.momentum);
    const double n = double(t + 1 - x.t_state_origin);
    const double bc1 = 1.0 - std::pow(c.beta1, n), bc2 = 1.0 - std::pow(c.beta2, n);
    p.eta_wd = float(eta * c.weight_decay);
    p.beta1 = float(c.beta1); p.beta2 = float(c.beta2);
    p.omb1 = float(1.0 - c.beta1); p.omb2 = float(1.0 - c.beta2);
    p.step_size = float(eta / bc1);
    p.inv_sqrt_bc2 = float(1.0 / std::sqrt(bc2));
    p.eps = float(c.eps);
    p.inv_K = 1.0f / float(c.K);
    p.n_tensors = x.n_tensors; p.tensor_end = x.tensor_end; p.wd_scale = x.wd_scale;
    return p;
}

qsr::SyncParams sync_params(const qsr_ctx &x)
{
    const qsr_config &c = x.cfg;
    qsr::SyncParams p;
    std::memset(&p, 0, sizeof p);
    p.slab[0] = x.theta; p.slab[1] = x.s1; p.slab[2] = x.s2;
    const int ns = n_state_slabs(c);
    p.n_mean = c.state_sync == QSR_STATE_AVERAGE ? 1 + ns : 1;
    p.n_zero = c.state_sync == QSR_STATE_RESET ? ns : 0;
    p.P = c.P; p.stride = c.row_stride; p.K = c.K;
    p.P4 = round_up4(c.P);
    p.divisor = float(c.K);
    return p;
}

int cuda_rc(int err) { return err == 0 ? QSR_OK : QSR_ECUDA; }

// NVTX range for one communication round; a no-op unless a profiler is attached.
struct RoundRange {
    RoundRange(int64_t s, int64_t t, int64_t H)
    {
        char name[64];
        std::snprintf(name, sizeof name, "qsr round %lld: t=%lld H=%lld", (long long)s, (long long)t, (long long)H);
        nvtxRangePushA(name);
    }
    ~RoundRange() { nvtxRangePop(); }
};

// With clipping on: enqueue the norm pass and the factor pass for this step and make the step kernel use the factors.
// `partials_ready`: the preceding step of the same round, launched by qsr_run, has already left this step's norm
// partials in the workspace (Local OPT with generated gradients only), so only the factor pass is needed.
int prepare_clip(qsr_ctx &x, qsr::StepParams &p, bool parallel, bool partials_ready = false)
{
    if (!(x.clip_norm > 0.0)) return QSR_OK;
    if (parallel) {
        x.launches += 2;
        if (int err = qsr::launch_clip_coef_parallel(p, x.clip_norm, x.clip_ws, x.stream)) return cuda_rc(err);
        p.clip_coef = x.clip_ws + qsr::clip_grid(x.cfg.P);
        return QSR_OK;
    }
    const int64_t blocks = qsr::clip_norm_blocks(x.cfg.P, x.shape.step_threads);
    if (!partials_ready) {
        x.launches++;
        if (int err = qsr::launch_clip_norms(p, x.clip_ws, x.shape, x.stream)) return cuda_rc(err);
    }
    x.launches++;
    if (int err = qsr::launch_clip_factors(x.clip_ws, blocks, x.cfg.K, x.clip_norm, x.stream)) return cuda_rc(err);
    p.clip_coef = x.clip_ws + blocks * x.cfg.K;
    return QSR_OK;
}

// Inside a round qsr_run issues every step itself and nothing else touches the parameters in between, so with
// clipping on a plain step can compute its successor's gradient norms on the side (the new parameters are in its
// registers) and the successor skips its norm pass.  Needs room for K x threads sums next to the step's ring.
// A step that also evaluates the next step's noise is bound by its instruction stream rather than by the bytes it
// keeps in flight, and gains more from a third or fourth resident block than from a deep ring: at most four rows in
// flight (ViT-B/16 shape, K = 16: 6.24 ms per step with eight, 5.84 with four; the block size stays, because the norm
// partials are laid out per block of the step).
qsr::LaunchShape clip_fold_shape(const qsr_ctx &x)
{
    qsr::LaunchShape s = x.shape;
    if (s.step_rows == 0 || s.step_rows > 4) s.step_rows = 4;
    return s;
}

bool clip_fold_applies(const qsr_ctx &x)
{
    if (!(x.clip_norm > 0.0)) return false;
    const qsr::LaunchShape s = clip_fold_shape(x);
    return qsr::step_shared_bytes(x.cfg.opt, false, s.step_rows, s.step_threads, x.cfg.K) <= size_t(227) * 1024;
}

// A plain local step of qsr_run's own loop (generated gradients).
int run_local_step(qsr_ctx &x, int64_t t, bool partials_ready, bool leave_next_partials)
{
    qsr::StepParams p = step_params(x, t, nullptr);
    if (int rc = prepare_clip(x, p, false, partials_ready)) return rc;
    if (leave_next_partials) p.norm_partial = x.clip_ws;
    x.launches++;
    return cuda_rc(qsr::launch_step(p, x.cfg.opt, leave_next_partials ? clip_fold_shape(x) : x.shape, x.stream));
}

constexpr size_t kMaxCachedGraphs = 48;

void drop_graphs(qsr_ctx &x)
{
    for (StepGraph &g : x.graphs) {
        if (g.exec) cudaGraphExecDestroy(g.exec);
        if (g.graph) cudaGraphDestroy(g.graph);
    }
    x.graphs.clear();
}

// Graph replay covers the launches qsr_run issues by itself: plain steps with generated gradients, and the fused
// last step when the state is kept per worker.  Clipping adds two launches per step whose arguments move with the
// workspace, so it stays on the direct path.
bool graph_replay_applies(const qsr_ctx &x) { return x.graph_steps > 0 && !(x.clip_norm > 0.0); }

// Register-resident launches cover what qsr_run issues by itself with the plain kernel instance: generated gradients,
// uniform weight decay, no clipping, and few enough workers for one block to hold all rows of its columns.
bool resident_applies(const qsr_ctx &x)
{
    return x.resident_steps > 0 && !(x.clip_norm > 0.0) && x.n_tensors == 0 && x.cfg.K <= qsr::kMaxResidentK;
}

// Algorithm 2 over the rounds that start in [t_begin, t_end) with consecutive steps packed into register-resident
// launches of at most resident_steps steps.  With the state kept per worker a launch runs across round ends (the
// averaging is block-local); in the other state modes a launch stops at the round end and the stand-alone
// synchronization follows, which also moves the bias-correction origin in RESET mode before the next step's scalars
// are formed.
int run_resident(qsr_ctx &x, int64_t t_begin, int64_t t_end, int64_t *round_start, int64_t *round_len, int64_t cap,
                 int64_t *n_rounds)
{
    const bool keep = x.cfg.state_sync == QSR_STATE_KEEP;
    qsr::ResidentParams q;
    std::memset(&q, 0, sizeof q);
    // Columns per block (threads = columns x K, whole warps, at most 1024): 32 gives each warp 512 contiguous bytes of a
    // row, but a small problem has only a few blocks per multiprocessor and whole blocks of imbalance (P = 65,536, K = 4:
    // 512 blocks of 128 threads on 148 multiprocessors, i.e. 3 or 4 each); narrower blocks even that out, and the rows
    // are only touched once per launch.  Take a narrower width only where it fills the last wave by 2 % more.
    {
        const int64_t n_col = (x.cfg.P + 3) >> 2;
        double best = -1.0;
        for (int cx : {64, 32, 16, 8}) {
            const int threads = cx * x.cfg.K;
            if (threads % 32 != 0 || threads > 1024 || (cx == 64 && x.cfg.K > 2)) continue;
            const int64_t blocks = (n_col + cx - 1) / cx;
            const int64_t waves = (blocks + x.sm_count - 1) / x.sm_count;
            const double fill = double(blocks) / double(waves * x.sm_count);
            if (fill > best + 0.02) { best = fill; q.cols_per_block = cx; }
        }
        if (best < 0.0) q.cols_per_block = 32;     // K = 1 with 32 columns is one warp per block: always valid
    }
    auto flush = [&]() -> int {
        if (q.n_steps == 0) return QSR_OK;
        x.launches++;
        const int err = qsr::launch_resident_steps(q, x.cfg.opt, x.stream);
        q.n_steps = 0;
        std::memset(q.sync_after, 0, sizeof q.sync_after);
        return cuda_rc(err);
    };
    int64_t s = 0;
    for (int64_t t = t_begin; t < t_end;) {
        const int64_t H = qsr::round_length(x.cfg, t);       // GetH
        const RoundRange range(s, t, H);
        for (int64_t h = 0; h < H; ++h) {
            const qsr::StepParams sp = step_params(x, t + h, nullptr);
            if (q.n_steps == 0) q.base = sp;                 // pointers, constants and the first step's index
            q.per_step[q.n_steps] = qsr::ResidentScalars{sp.eta, sp.eta_wd, sp.step_size, sp.inv_sqrt_bc2};
            if (keep && h == H - 1) q.sync_after[q.n_steps >> 5] |= 1u << (q.n_steps & 31);
            if (++q.n_steps == x.resident_steps)
                if (int rc = flush()) return rc;
        }
        if (!keep) {
            if (int rc = flush()) return rc;
            if (int rc = qsr_sync(&x, t + H)) return rc;
        }
        if (s < cap) {
            round_start[s] = t;
            round_len[s] = H;
        }
        ++s;
        t += H;
    }
    if (int rc = flush()) return rc;
    if (n_rounds) *n_rounds = s;
    return QSR_OK;
}

cudaKernelNodeParams node_params(const qsr::StepLaunch &L, void **args)
{
    cudaKernelNodeParams k;
    std::memset(&k, 0, sizeof k);
    k.func = const_cast<void *>(L.func);
    k.gridDim = dim3(L.grid);
    k.blockDim = dim3(unsigned(L.threads));
    k.sharedMemBytes = unsigned(L.smem);
    k.kernelParams = args;
    k.extra = nullptr;
    return k;
}

// Steps t .. t + n_plain - 1 as plain local steps and, if `fused`, step t + n_plain as the round's last step with
// the replica mean, enqueued as ONE graph launch.  The chain for (n_plain, fused) is built and instantiated the first
// time it is needed and kept; every replay first rewrites each node's StepParams (the learning rate, the bias
// corrections and the Philox counter word change with t).  An update only affects launches made after it, so the
// executable graph may still be running an earlier replay while it is being updated.  Returns QSR_OK, QSR_ECUDA,
// or 1 when the cache is full and the caller should launch directly.
int replay_steps(qsr_ctx &x, int64_t t, int n_plain, bool fused)
{
    const int n = n_plain + (fused ? 1 : 0);
    StepGraph *g = nullptr;
    for (StepGraph &c : x.graphs)
        if (c.n_plain == n_plain && c.fused == fused) { g = &c; break; }
    std::vector<qsr::StepParams> params;
    params.resize(size_t(n));
    for (int i = 0; i < n; ++i) params[size_t(i)] = step_params(x, t + i, nullptr);
    if (!g) {
        if (x.graphs.size() >= kMaxCachedGraphs) return 1;
        StepGraph fresh;
        fresh.n_plain = n_plain; fresh.fused = fused; fresh.graph = nullptr; fresh.exec = nullptr;
        if (qsr::resolve_step(params[0], x.cfg.opt, x.shape, qsr::FUSE_NONE, &fresh.plain) != 0 ||
            qsr::resolve_step(params[0], x.cfg.opt, x.shape, qsr::FUSE_MEAN, &fresh.last) != 0)
            return QSR_ECUDA;
        if (cudaGraphCreate(&fresh.graph, 0) != cudaSuccess) return QSR_ECUDA;
        bool ok = true;
        for (int i = 0; i < n && ok; ++i) {
            void *args[] = {&params[size_t(i)]};
            const cudaKernelNodeParams k = node_params((fused && i == n - 1) ? fresh.last : fresh.plain, args);
            cudaGraphNode_t node = nullptr;
            const cudaGraphNode_t *dep = fresh.nodes.empty() ? nullptr : &fresh.nodes.back();
            ok = cudaGraphAddKernelNode(&node, fresh.graph, dep, dep ? 1 : 0, &k) == cudaSuccess;
            if (ok) fresh.nodes.push_back(node);
        }
        if (ok) ok = cudaGraphInstantiate(&fresh.exec, fresh.graph, 0) == cudaSuccess;
        if (!ok) {
            if (fresh.exec) cudaGraphExecDestroy(fresh.exec);
            cudaGraphDestroy(fresh.graph);
            cudaGetLastError();
            return QSR_ECUDA;
        }
        x.graphs.push_back(fresh);
        g = &x.graphs.back();     // instantiated with this replay's arguments: no update needed
    } else {
        for (int i = 0; i < n; ++i) {
            void *args[] = {&params[size_t(i)]};
            const cudaKernelNodeParams k = node_params((fused && i == n - 1) ? g->last : g->plain, args);
            if (cudaGraphExecKernelNodeSetParams(g->exec, g->nodes[size_t(i)], &k) != cudaSuccess) return QSR_ECUDA;
        }
    }
    if (cudaGraphLaunch(g->exec, x.stream) != cudaSuccess) return QSR_ECUDA;
    x.launches += n;
    return QSR_OK;
}

}  // namespace

extern "C" {

int qsr_init(qsr_ctx **out, const qsr_config *cfg, float *params, float *state1, float *state2,
             const float *lambda, const float *theta_star, void *cuda_stream)
{
    if (!out) return QSR_EINVAL;
    *out = nullptr;
    if (!cfg || !params || !state1) return QSR_EINVAL;
    if (int rc = qsr::check_config(*cfg)) return rc;
    if (cfg->opt == QSR_OPT_ADAMW && !state2) return QSR_EINVAL;
    if ((lambda == nullptr) != (theta_star == nullptr)) return QSR_EINVAL;
    if (!aligned16(params) || !aligned16(state1) || !aligned16(state2) || !aligned16(lambda) || !aligned16(theta_star))
        return QSR_EALIGN;
    if (int64_t(cfg->worker_offset) + cfg->K > (int64_t(1) << 32)) return QSR_ERANGE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return QSR_ECUDA;
    qsr_ctx *x = new (std::nothrow) qsr_ctx;
    if (!x) return QSR_EINVAL;
    x->cfg = *cfg;
    x->theta = params; x->s1 = state1; x->s2 = cfg->opt == QSR_OPT_ADAMW ? state2 : nullptr;
    x->lambda = lambda; x->theta_star = theta_star;
    x->stream = static_cast<cudaStream_t>(cuda_stream);
    x->device = dev;
    x->sm_count = 148;
    cudaDeviceGetAttribute(&x->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (x->sm_count < 1) x->sm_count = 148;
    x->shape = qsr::LaunchShape();
    if (cfg->opt == QSR_OPT_SGDM) x->shape.step_threads = 128;
    // Slabs that stay resident in L2 between steps are served with far lower latency than HBM: a 4-row ring in
    // 128-thread blocks (more blocks per SM, shorter prologue) then beats the 8-row ring (K = 8, P = 2^20 AdamW on
    // B200: 31.3 us against 35.7 us per step).
    int l2_bytes = 0;
    if (cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, dev) == cudaSuccess) {
        const int64_t state_bytes = int64_t(1 + n_state_slabs(*cfg)) * cfg->K * cfg->row_stride * int64_t(sizeof(float));
        if (state_bytes <= int64_t(l2_bytes) / 5 * 4) {
            x->shape.step_threads = 128;
            x->shape.step_rows = 4;
        }
    }
    x->t_state_origin = cfg->t_state_origin;
    x->launches = 0;
    x->partial_pending = false;
    x->n_tensors = 0; x->tensor_end = nullptr; x->wd_scale = nullptr;
    x->clip_norm = 0.0; x->clip_ws = nullptr;
    x->graph_steps = 0;
    x->resident_steps = 0;
    *out = x;
    return QSR_OK;
}

int qsr_destroy(qsr_ctx *ctx)
{
    if (ctx) drop_graphs(*ctx);
    delete ctx;
    return QSR_OK;
}

int64_t qsr_round_length(const qsr_ctx *ctx, int64_t t)
{
    if (!ctx) return QSR_EINVAL;
    if (t < 0 || t >= ctx->cfg.T) return QSR_ERANGE;
    return qsr::round_length(ctx->cfg, t);
}

int qsr_set_params(qsr_ctx *ctx, const float *theta0_dev)
{
    if (!ctx || !theta0_dev) return QSR_EINVAL;
    if (!aligned16(theta0_dev)) return QSR_EALIGN;
    ctx->launches++;
    return cuda_rc(qsr::launch_broadcast(ctx->theta, theta0_dev, ctx->cfg.P, ctx->cfg.row_stride, ctx->cfg.K,
                                         ctx->shape, ctx->stream));
}

int qsr_local_step(qsr_ctx *ctx, int64_t t, const float *grads)
{
    if (!ctx) return QSR_EINVAL;
    if (t < 0 || t >= ctx->cfg.T || t < ctx->t_state_origin) return QSR_ERANGE;
    if (!grads && !ctx->lambda) return QSR_EINVAL;
    if (!aligned16(grads)) return QSR_EALIGN;
    qsr::StepParams p = step_params(*ctx, t, grads);
    if (int rc = prepare_clip(*ctx, p, false)) return rc;
    ctx->launches++;
    return cuda_rc(qsr::launch_step(p, ctx->cfg.opt, ctx->shape, ctx->stream));
}

int qsr_set_tensor_table(qsr_ctx *ctx, int32_t n_tensors, const int64_t *tensor_end_dev, const float *wd_scale_dev)
{
    if (!ctx || n_tensors < 0) return QSR_EINVAL;
    if (n_tensors > 0) {
        if (!tensor_end_dev || !wd_scale_dev) return QSR_EINVAL;
        if ((reinterpret_cast<uintptr_t>(tensor_end_dev) & 7u) || (reinterpret_cast<uintptr_t>(wd_scale_dev) & 3u)) return QSR_EALIGN;
    }
    // A table switches the step to the kernel instance that looks the factors up; cached graph chains were built
    // around the other instance and would go on replaying it, so they are discarded whenever the choice changes.
    if ((ctx->n_tensors > 0) != (n_tensors > 0)) drop_graphs(*ctx);
    if (n_tensors == 0) {
        ctx->n_tensors = 0; ctx->tensor_end = nullptr; ctx->wd_scale = nullptr;
        return QSR_OK;
    }
    ctx->n_tensors = n_tensors; ctx->tensor_end = tensor_end_dev; ctx->wd_scale = wd_scale_dev;
    return QSR_OK;
}

int64_t qsr_clip_workspace_floats(const qsr_ctx *ctx)
{
    if (!ctx) return QSR_EINVAL;
    // Local OPT: partials [blocks of a step launch, K] followed by the K factors; the smallest block (64 threads) gives
    // the most blocks.  Algorithm 1: at most kNormGrid partials and one factor.
    const int64_t local = qsr::clip_norm_blocks(ctx->cfg.P, 64) * ctx->cfg.K + ctx->cfg.K;
    const int64_t parallel = int64_t(qsr::kNormGrid) + 1;
    return round_up4(local > parallel ? local : parallel);
}

int qsr_set_grad_clip(qsr_ctx *ctx, double max_norm, float *workspace_dev)
{
    if (!ctx) return QSR_EINVAL;
    if (!(max_norm > 0.0) || std::isinf(max_norm)) {     // off (also for NaN)
        ctx->clip_norm = 0.0; ctx->clip_ws = nullptr;
        return QSR_OK;
    }
    if (!workspace_dev) return QSR_EINVAL;
    if (!aligned16(workspace_dev)) return QSR_EALIGN;
    if (ctx->cfg.K > qsr::kMaxClipK) return QSR_ERANGE;   // the norm pass keeps K x (step threads) sums in shared memory
    ctx->clip_norm = max_norm; ctx->clip_ws = workspace_dev;
    return QSR_OK;
}

int qsr_parallel_step(qsr_ctx *ctx, int64_t t, const float *grads)
{
    if (!ctx) return QSR_EINVAL;
    if (t < 0 || t >= ctx->cfg.T || t < ctx->t_state_origin) return QSR_ERANGE;
    if (!grads && !ctx->lambda) return QSR_EINVAL;
    if (!aligned16(grads)) return QSR_EALIGN;
    qsr::StepParams p = step_params(*ctx, t, grads);
    if (int rc = prepare_clip(*ctx, p, true)) return rc;
    ctx->launches++;
    return cuda_rc(qsr::launch_parallel_step(p, ctx->cfg.opt, ctx->shape, ctx->stream));
}

// The round's last step and its synchronization.  `partials_ready` as in prepare_clip (qsr_run only).
static int local_step_sync_impl(qsr_ctx *ctx, int64_t t, const float *grads, int64_t t_next, bool partials_ready)
{
    if (!ctx) return QSR_EINVAL;
    if (t < 0 || t >= ctx->cfg.T || t < ctx->t_state_origin || t_next < 0 || t_next > ctx->cfg.T) return QSR_ERANGE;
    if (!grads && !ctx->lambda) return QSR_EINVAL;
    if (!aligned16(grads)) return QSR_EALIGN;
    qsr::StepParams p = step_params(*ctx, t, grads);
    if (int rc = prepare_clip(*ctx, p, false, partials_ready)) return rc;
    ctx->launches++;
    if (ctx->cfg.state_sync != QSR_STATE_KEEP) {
        // Averaging or resetting the optimizer state needs the stand-alone kernel: a plain step, then the sync.
        if (int rc = cuda_rc(qsr::launch_step(p, ctx->cfg.opt, ctx->shape, ctx->stream))) return rc;
        return qsr_sync(ctx, t_next);
    }
    return cuda_rc(qsr::launch_step_mean(p, ctx->cfg.opt, ctx->shape, ctx->stream));
}

int qsr_local_step_sync(qsr_ctx *ctx, int64_t t, const float *grads, int64_t t_next)
{
    return local_step_sync_impl(ctx, t, grads, t_next, false);
}

int qsr_sync(qsr_ctx *ctx, int64_t t_next)
{
    if (!ctx) return QSR_EINVAL;
    if (t_next < 0 || t_next > ctx->cfg.T) return QSR_ERANGE;
    const qsr::SyncParams p = sync_params(*ctx);
    ctx->launches += qsr::sync_launches(p);
    const int rc = cuda_rc(qsr::launch_sync(p, ctx->shape, ctx->stream));
    if (rc == QSR_OK && ctx->cfg.state_sync == QSR_STATE_RESET) ctx->t_state_origin = t_next;
    return rc;
}

int qsr_local_step_partial(qsr_ctx *ctx, int64_t t, const float *grads, float *sum)
{
    if (!ctx || !sum) return QSR_EINVAL;
    if (!aligned16(sum)) return QSR_EALIGN;
    if (ctx->cfg.state_sync != QSR_STATE_KEEP) {
        // the state slabs need their own sums (AVERAGE) or nothing fused is gained (RESET): two launches
        if (int rc = qsr_local_step(ctx, t, grads)) return rc;
        return qsr_sync_partial(ctx, sum);
    }
    if (t < 0 || t >= ctx->cfg.T || t < ctx->t_state_origin) return QSR_ERANGE;
    if (!grads && !ctx->lambda) return QSR_EINVAL;
    if (!aligned16(grads)) return QSR_EALIGN;
    qsr::StepParams p = step_params(*ctx, t, grads);
    if (int rc = prepare_clip(*ctx, p, false)) return rc;
    p.sum_out = sum;
    ctx->launches++;
    const int rc = cuda_rc(qsr::launch_step_sum(p, ctx->cfg.opt, ctx->shape, ctx->stream));
    if (rc == QSR_OK) ctx->partial_pending = true;
    return rc;
}

int64_t qsr_sync_sum_floats(const qsr_ctx *ctx)
{
    if (!ctx) return QSR_EINVAL;
    const int n_mean = ctx->cfg.state_sync == QSR_STATE_AVERAGE ? 1 + n_state_slabs(ctx->cfg) : 1;
    return n_mean * round_up4(ctx->cfg.P);
}

int qsr_sync_partial(qsr_ctx *ctx, float *sum)
{
    if (!ctx || !sum) return QSR_EINVAL;
    if (!aligned16(sum)) return QSR_EALIGN;
    qsr::SyncParams p = sync_params(*ctx);
    p.sum_out = sum;
    ctx->launches++;
    const int rc = cuda_rc(qsr::launch_sync_partial(p, ctx->shape, ctx->stream));
    if (rc == QSR_OK) ctx->partial_pending = true;
    return rc;
}

int qsr_sync_finish(qsr_ctx *ctx, const float *sum, int32_t K_total, int64_t t_next)
{
    if (!ctx || !sum) return QSR_EINVAL;
    if (!aligned16(sum)) return QSR_EALIGN;
    if (K_total < ctx->cfg.K || t_next < 0 || t_next > ctx->cfg.T) return QSR_ERANGE;
    if (!ctx->partial_pending) return QSR_ESTATE;
    qsr::SyncParams p = sync_params(*ctx);
    p.sum_in = sum;
    p.divisor = float(K_total);
    ctx->launches += qsr::sync_launches(p);
    const int rc = cuda_rc(qsr::launch_sync_finish(p, ctx->shape, ctx->stream));
    if (rc == QSR_OK) {
        ctx->partial_pending = false;
        if (ctx->cfg.state_sync == QSR_STATE_RESET) ctx->t_state_origin = t_next;
    }
    return rc;
}

int qsr_sync_static(qsr_ctx *ctx, int64_t t_next)
{
    if (!ctx) return QSR_EINVAL;
    if (t_next < 0 || t_next > ctx->cfg.T) return QSR_ERANGE;
    const qsr::SyncParams p = sync_params(*ctx);
    if (int64_t(p.n_mean) * p.P4 > int64_t(QSR_STATIC_SCRATCH_FLOATS)) return QSR_ERANGE;   // nothing was launched
    const int err = qsr::launch_sync_static(p, ctx->shape, ctx->device, ctx->stream);
    if (err != 0) return err == -1 ? QSR_ERANGE : (err == -2 ? QSR_ESTATE : QSR_ECUDA);
    ctx->launches += 1 + qsr::sync_launches(p);
    if (ctx->cfg.state_sync == QSR_STATE_RESET) ctx->t_state_origin = t_next;
    return QSR_OK;
}

int qsr_debug_box_muller(const uint32_t *words_dev, int64_t n, float *radius_dev, float *sin_dev, float *cos_dev,
                         void *cuda_stream)
{
    if (n < 0) return QSR_EINVAL;
    if (n == 0) return QSR_OK;
    if (!words_dev || !radius_dev || !sin_dev || !cos_dev) return QSR_EINVAL;
    if ((reinterpret_cast<uintptr_t>(words_dev) | reinterpret_cast<uintptr_t>(radius_dev) |
         reinterpret_cast<uintptr_t>(sin_dev) | reinterpret_cast<uintptr_t>(cos_dev)) & 3u)
        return QSR_EALIGN;
    return cuda_rc(qsr::launch_box_muller_parts(words_dev, n, radius_dev, sin_dev, cos_dev, cuda_stream));
}

int qsr_debug_fast_math(const float *x_dev, int64_t n, float *sqrt_dev, float *rcp_dev, void *cuda_stream)
{
    if (n < 0) return QSR_EINVAL;
    if (n == 0) return QSR_OK;
    if (!x_dev || !sqrt_dev || !rcp_dev) return QSR_EINVAL;
    if ((reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(sqrt_dev) | reinterpret_cast<uintptr_t>(rcp_dev)) & 3u)
        return QSR_EALIGN;
    return cuda_rc(qsr::launch_fast_math(x_dev, n, sqrt_dev, rcp_dev, cuda_stream));
}

int qsr_run(qsr_ctx *ctx, int64_t t_begin, int64_t t_end,
            int64_t *round_start, int64_t *round_len, int64_t cap, int64_t *n_rounds)
{
    if (!ctx || cap < 0 || (cap > 0 && (!round_start || !round_len))) return QSR_EINVAL;
    if (t_begin < 0 || t_end > ctx->cfg.T || t_begin > t_end) return QSR_ERANGE;
    if (!ctx->lambda) return QSR_EINVAL;
    if (resident_applies(*ctx)) return run_resident(*ctx, t_begin, t_end, round_start, round_len, cap, n_rounds);
    int64_t s = 0;
    for (int64_t t = t_begin; t < t_end;) {
        const int64_t H = qsr::round_length(ctx->cfg, t);       // GetH
        const RoundRange range(s, t, H);
        const bool fuse_last = ctx->cfg.state_sync == QSR_STATE_KEEP;
        int64_t h = 0;
        if (graph_replay_applies(*ctx)) {
            // whole segments of at most graph_steps launches; a round's tail takes its fused last step along
            while (h < H) {
                const int64_t left = H - h;
                const bool tail = left <= ctx->graph_steps;
                const int n_plain = int(tail ? left - 1 : ctx->graph_steps);
                const bool fused = tail && fuse_last;
                if (n_plain + (fused ? 1 : 0) == 0) break;      // only the unfused last step remains
                const int rc = replay_steps(*ctx, t + h, n_plain, fused);
                if (rc < 0) return rc;
                if (rc > 0) break;                              // cache full: finish the round with direct launches
                h += n_plain + (fused ? 1 : 0);
            }
        }
        // with clipping on, each plain step leaves its successor's gradient-norm partials behind (clip_fold_applies)
        const bool fold = h == 0 && clip_fold_applies(*ctx);
        bool partials_ready = false;
        for (; h + 1 < H; ++h) {
            if (int rc = run_local_step(*ctx, t + h, partials_ready, fold)) return rc;
            partials_ready = fold;
        }
        // the round's last step and the parameter averaging, in one launch when the state is kept per worker
        if (h < H)
            if (int rc = local_step_sync_impl(ctx, t + H - 1, nullptr, t + H, partials_ready)) return rc;
        if (s < cap) {
            round_start[s] = t;
            round_len[s] = H;
        }
        ++s;
        t += H;
    }
    if (n_rounds) *n_rounds = s;
    return QSR_OK;
}

int qsr_set_graph_replay(qsr_ctx *ctx, int32_t max_steps_per_graph)
{
    if (!ctx) return QSR_EINVAL;
    if (max_steps_per_graph < 0 || max_steps_per_graph > 1024) return QSR_ERANGE;
    if (max_steps_per_graph != ctx->graph_steps) drop_graphs(*ctx);
    ctx->graph_steps = max_steps_per_graph;
    return QSR_OK;
}

int qsr_set_resident_steps(qsr_ctx *ctx, int32_t max_steps_per_launch)
{
    if (!ctx) return QSR_EINVAL;
    if (max_steps_per_launch < 0 || max_steps_per_launch > qsr::kMaxResidentSteps) return QSR_ERANGE;
    if (max_steps_per_launch > 0 && ctx->cfg.K > qsr::kMaxResidentK) return QSR_ERANGE;
    ctx->resident_steps = max_steps_per_launch;
    return QSR_OK;
}

int64_t qsr_launch_count(const qsr_ctx *ctx) { return ctx ? ctx->launches : int64_t(QSR_EINVAL); }

int qsr_set_launch_shape(qsr_ctx *ctx, int32_t step_threads, int32_t step_rows_in_flight, int32_t sync_threads)
{
    if (!ctx) return QSR_EINVAL;
    auto ok_threads = [](int32_t n, int32_t hi) { return n == 0 || (n >= 64 && n <= hi && n % 32 == 0); };
    if (!ok_threads(step_threads, 1024) || !ok_threads(sync_threads, 512)) return QSR_ERANGE;
    if (step_rows_in_flight != 0 && step_rows_in_flight != 1 && step_rows_in_flight != 2 && step_rows_in_flight != 4 &&
        step_rows_in_flight != 8)
        return QSR_ERANGE;
    drop_graphs(*ctx);      // cached graphs carry the old geometry
    if (step_threads) ctx->shape.step_threads = step_threads;
    if (step_rows_in_flight) ctx->shape.step_rows = step_rows_in_flight;
    if (sync_threads) ctx->shape.sync_threads = sync_threads;
    return QSR_OK;
}

int64_t qsr_workspace_bytes(const qsr_config *cfg)
{
    if (!cfg) return QSR_EINVAL;
    qsr_config c = *cfg;
    c.row_stride = qsr::row_stride_hint(c.P);
    if (int rc = qsr::check_config(c)) return rc;
    const int64_t slabs = 1 + n_state_slabs(c);
    return (slabs * c.K * c.row_stride + 3 * c.row_stride) * int64_t(sizeof(float));
}

int qsr_train_host(const qsr_config *cfg, const float *theta0_host, const float *lambda_host,
                   const float *theta_star_host, float *theta_out_host,
                   void *workspace_dev, int64_t workspace_bytes, int64_t t_end, void *cuda_stream,
                   int64_t *round_start, int64_t *round_len, int64_t cap, int64_t *n_rounds, int64_t *launches)
{
    if (launches) *launches = 0;
    if (n_rounds) *n_rounds = 0;
    if (!cfg || !theta0_host || !lambda_host || !theta_star_host || !theta_out_host || !workspace_dev) return QSR_EINVAL;
    qsr_config c = *cfg;
    c.row_stride = qsr::row_stride_hint(c.P);
    c.t_state_origin = 0;
    if (int rc = qsr::check_config(c)) return rc;
    if ((reinterpret_cast<uintptr_t>(workspace_dev) & 255u) != 0) return QSR_EALIGN;
    const int64_t need = qsr_workspace_bytes(&c);
    if (workspace_bytes < need || t_end < 0 || t_end > c.T) return QSR_ERANGE;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    float *w = static_cast<float *>(workspace_dev);
    const int64_t slab = int64_t(c.K) * c.row_stride;
    float *theta = w, *s1 = w + slab, *s2 = c.opt == QSR_OPT_ADAMW ? w + 2 * slab : nullptr;
    float *vec = w + (1 + n_state_slabs(c)) * slab;
    float *lambda = vec, *theta_star = vec + c.row_stride, *theta0 = vec + 2 * c.row_stride;
    const size_t row_bytes = size_t(c.P) * sizeof(float);

    // Every check that can fail on the host comes before the first copy is enqueued (the context only records
    // pointers); from here on, whatever happens, the call waits for the stream before it returns, so the caller's
    // host buffers are never still in use by a copy when it gets them back.
    qsr_ctx *x = nullptr;
    if (int rc = qsr_init(&x, &c, theta, s1, s2, lambda, theta_star, cuda_stream)) return rc;
    int rc = QSR_OK;
    if (cudaMemcpyAsync(lambda, lambda_host, row_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(theta_star, theta_star_host, row_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(theta0, theta0_host, row_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemsetAsync(s1, 0, size_t(n_state_slabs(c)) * slab * sizeof(float), st) != cudaSuccess)
        rc = QSR_ECUDA;
    if (rc == QSR_OK) rc = qsr_set_params(x, theta0);
    if (rc == QSR_OK) rc = qsr_run(x, 0, t_end, round_start, round_len, cap, n_rounds);
    if (rc == QSR_OK && cudaMemcpyAsync(theta_out_host, theta, row_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        rc = QSR_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess && rc == QSR_OK) rc = QSR_ECUDA;
    if (launches) *launches = x->launches;
    qsr_destroy(x);
    return rc;
}

}  // extern "C"
