/*
 * qsr.h -- C ABI of the Local-OPT / Quadratic-Synchronization-Rule hot path for NVIDIA B200 (sm_100a).
 *
 * The library runs Algorithm 2 ("Local OPT") of "A Quadratic Synchronization Rule for Distributed Deep
 * Learning" (arXiv 2310.14423) with the K workers laid out as the rows of [K, P] fp32 slabs in one GPU's
 * memory: every worker takes local optimizer steps on its own stochastic gradient (Eq. 1), at the end of a
 * round all workers replace their parameters by the mean over workers (the All-Reduce line of Algorithm 2,
 * here a mean over the replica axis), and the length of each round follows Eq. 2.
 *
 * Conventions that hold for every call unless a comment says otherwise
 *   - Pointers named params / state1 / state2 / grads / lambda / theta_star / sum / theta0_dev are DEVICE
 *     pointers, 16-byte aligned; the caller owns them and keeps them alive until qsr_destroy.  The library
 *     allocates no device memory and frees none.  Pointers with "host" in their name are HOST pointers.
 *   - Slabs are row-major [K, row_stride] floats; worker k's coordinate i is slab[k * row_stride + i],
 *     i < P <= row_stride, row_stride a multiple of 4.  Elements with i >= P are never read or written.
 *     Any such stride works; qsr_row_stride_hint(P) is the one the kernels stream fastest with.
 *   - Device work is enqueued on the CUDA stream given to qsr_init; no call waits for the device except
 *     qsr_train_host.  The host-side schedule functions do no device work at all.
 *   - Every function returns QSR_OK (0) or a negative qsr_status; none aborts, throws or exits.  A failed
 *     call leaves the slabs untouched unless the failure is QSR_ECUDA from a launch.
 *   - A context is used from one host thread at a time.
 */
#ifndef QSR_H_
#define QSR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qsr_ctx qsr_ctx; /* opaque; host memory owned by the library */

typedef enum {
    QSR_OK = 0,
    QSR_EINVAL = -1, /* NULL where a pointer is required, K < 1, P < 1, unknown enum value, non-finite number */
    QSR_EALIGN = -2, /* a device pointer is not 16-byte aligned, or row_stride is not a multiple of 4 or < P */
    QSR_ECUDA = -3,  /* the CUDA runtime reported an error (no device, launch failure, failed copy)          */
    QSR_ERANGE = -4, /* t outside [0, T), T_warmup >= T, H_base < 1, K or t beyond 2^32, workspace too small */
    QSR_ESTATE = -5  /* call out of order (e.g. qsr_sync_finish without qsr_sync_partial)                     */
} qsr_status;

enum { QSR_OPT_SGDM = 0, QSR_OPT_ADAMW = 1 };
enum { QSR_SCHED_COSINE = 0, QSR_SCHED_STEP_POW2 = 1, QSR_SCHED_LINEAR = 2, QSR_SCHED_CONST = 3,
       QSR_SCHED_HALVING = 4, QSR_SCHED_COSINE_HELD = 5 };
enum { QSR_RULE_QSR = 0, QSR_RULE_CONST_H = 1, QSR_RULE_POWER = 2, QSR_RULE_POST_LOCAL = 3, QSR_RULE_SWAP = 4 };
enum { QSR_STATE_KEEP = 0, QSR_STATE_AVERAGE = 1, QSR_STATE_RESET = 2 };

/*
 * One run.  Plain data; the library copies it.
 *
 * OPT (Eq. 1; hyper-parameters of App. C):
 *   QSR_OPT_SGDM   g' = g + weight_decay*theta;  v <- momentum*v + g';  theta <- theta - eta_t*v   (state1 = v)
 *   QSR_OPT_ADAMW  theta <- theta*(1 - eta_t*weight_decay);  m <- beta1*m + (1-beta1)*g;  v <- beta2*v + (1-beta2)*g^2;
 *                  theta <- theta - eta_t * (m/(1-beta1^n)) / (sqrt(v)/sqrt(1-beta2^n) + eps)        (state1 = m, state2 = v)
 *                  n = t + 1 - t_state_origin counts the steps the state has seen.
 * Learning rate eta_t, t in {0..T-1} (Sec. 2): eta_max*t/T_warmup during warm-up, then, with
 *   x = (t - T_warmup)/(T - T_warmup):  COSINE eta_min + (eta_max-eta_min)*(1+cos(pi*x))/2;  STEP_POW2 that value
 *   rounded to 2^round(log2(.)) (Sec. 4, step-decay ablation);  LINEAR eta_min + (eta_max-eta_min)*(1-x);  CONST eta_max;
 *   HALVING (App. G) eta_max until t_hold, then eta_max / 2^(1 + (t - t_hold)/t_period) (integer division);
 *   COSINE_HELD (App. G) the cosine value of min(t, t_hold).
 * Round length (Eq. 2): QSR_RULE_QSR H = max(H_base, floor((alpha/eta_t)^2)) with eta_t taken at the round's first
 *   step, or at t = T_warmup for rounds that start during warm-up (Sec. 2); QSR_RULE_POWER the same with exponent
 *   gamma, pow(alpha/eta_t, gamma) (Sec. 2; gamma = 1 is H ~ 1/eta, gamma = 3 the cubic rule of App. G);
 *   QSR_RULE_CONST_H H = H_base; QSR_RULE_POST_LOCAL H = 1 while t < t_switch, then H_base (Sec. 1);
 *   QSR_RULE_SWAP H = min(H_base, t_switch - t) while t < t_switch, then one round to T (App. H).  In all cases H is
 *   cut to T - t so that the last round ends at T.
 * Synthetic gradient (stands in for Sample() and back-propagation of Algorithm 2 when no gradient slab is
 *   passed): g[k,i] = lambda[i]*(theta[k,i] - theta_star[i]) + noise_std*z(seed, worker_offset + k, t, i), where z is
 *   a standard normal obtained by Box-Muller from Philox-4x32-10 with counter (i/4 low, i/4 high, t, worker) and
 *   key = the two halves of seed; words (0,1) of the block serve i%4 in {0 (cos), 1 (sin)}, words (2,3) serve {2, 3};
 *   each uniform is (top 23 bits + 1/2) / 2^23.
 */
typedef struct qsr_config {
    int32_t K;              /* workers (rows) held in this process's slabs                                  */
    int32_t worker_offset;  /* global index of row 0 (0 unless the workers are sharded over several GPUs)   */
    int64_t P;              /* parameters per worker                                                        */
    int64_t row_stride;     /* floats between consecutive rows                                              */
    int32_t opt;            /* QSR_OPT_*                                                                    */
    int32_t sched;          /* QSR_SCHED_*                                                                  */
    int32_t rule;           /* QSR_RULE_*                                                                   */
    int32_t state_sync;     /* QSR_STATE_*: what a synchronization does to state1/state2 (KEEP: nothing;   */
                            /* AVERAGE: averaged like the parameters; RESET: zeroed, n restarts at 1)      */
    double momentum, beta1, beta2, eps, weight_decay;
    double eta_max, eta_min;
    double alpha;           /* growth coefficient of Eq. 2                                                  */
    double noise_std;
    int64_t T, T_warmup, H_base;
    int64_t t_state_origin; /* global step at which state1/state2 were last all-zero (0 for a fresh run)    */
    uint64_t seed;
    double gamma;           /* QSR_RULE_POWER: exponent                                                     */
    int64_t t_switch;       /* QSR_RULE_POST_LOCAL / QSR_RULE_SWAP: switching step                          */
    int64_t t_hold;         /* QSR_SCHED_HALVING / QSR_SCHED_COSINE_HELD: see above                         */
    int64_t t_period;       /* QSR_SCHED_HALVING: steps between halvings (>= 1)                             */
} qsr_config;

/* ---- host-only schedule (no device, no context) ------------------------------------------------------- */

/* Validates the scalar fields (not the pointers).  QSR_OK, QSR_EINVAL, QSR_EALIGN or QSR_ERANGE. */
int qsr_config_check(const qsr_config *cfg);

/* eta_t in binary64 (Sec. 2; formulas above).  NaN if cfg is invalid or t is outside [0, T). */
double qsr_config_learning_rate(const qsr_config *cfg, int64_t t);

/* H of a round whose first global step is t (Eq. 2 with the warm-up and last-round rules).  Negative
 * qsr_status on error. */
int64_t qsr_config_round_length(const qsr_config *cfg, int64_t t);

/* Writes the start step and the length of every round from t = 0 to T into round_start / round_len (host arrays
 * of `cap` entries; entries beyond cap are counted but not written).  Returns the number of rounds, or a negative
 * qsr_status.  The share of steps that synchronize (the "Comm." column of Tables 1-3) is rounds / T. */
int64_t qsr_config_schedule(const qsr_config *cfg, int64_t *round_start, int64_t *round_len, int64_t cap);

/* A row stride (in floats, a multiple of 4, >= P) that lets the kernels stream at full rate.  Any stride that obeys
 * the conventions above is legal, but where the K rows of a slab start matters to the memory system: on B200, with
 * K = 16 rows of P = 86,415,592 floats packed at P, the AdamW step takes 5.33 ms; with every row on a 16 KiB boundary
 * 5.19 ms, on a 256 KiB boundary 5.16 ms, on a 4 MiB boundary 5.12 ms (the averaging kernel 1.77 -> 1.68 ms; K = 32:
 * 10.76 -> 10.26 ms).  The hint rounds P up to a multiple of 2^a floats, a = min(20, floor(log2 P) - 4) but at least
 * 2, so the padding stays below P/16 (at most 4 MiB per row); padding is never read or written.  The base addresses
 * of params / state1 / state2 should agree modulo 4 KiB as well (state slabs shifted by 128 bytes against params cost
 * 1.6 %; shifts of 4 KiB and more cost nothing); large blocks from cudaMalloc or a caching allocator do.  Negative
 * qsr_status if P < 1. */
int64_t qsr_row_stride_hint(int64_t P);

/* Bytes of device workspace that qsr_train_host needs for cfg (slabs plus the two input vectors). */
int64_t qsr_workspace_bytes(const qsr_config *cfg);

/* ---- context ------------------------------------------------------------------------------------------ */

/* Creates a context over caller-owned slabs (Algorithm 2's workers).  params and state1 are [K, row_stride];
 * state2 is required for QSR_OPT_ADAMW and ignored for QSR_OPT_SGDM; lambda and theta_star are [P] and may be NULL
 * if every qsr_local_step will be given gradients.  cuda_stream is a cudaStream_t (NULL = the legacy default
 * stream).  Nothing is written to the slabs.  The device current at this call is the one the context uses. */
int qsr_init(qsr_ctx **out, const qsr_config *cfg, float *params, float *state1, float *state2,
             const float *lambda, const float *theta_star, void *cuda_stream);

/* Frees the context (host memory only).  NULL is accepted. */
int qsr_destroy(qsr_ctx *ctx);

/* Same as qsr_config_round_length on the context's configuration: GetH of Algorithm 2. */
int64_t qsr_round_length(const qsr_ctx *ctx, int64_t t);

/* Per-tensor weight decay.  The paper uses one weight-decay value for the whole model (App. C); recipes that exempt
 * normalization and bias tensors are common, so each tensor of the flattened parameter set may carry a factor on it.
 * tensor_end_dev [n_tensors] (device, int64): one past the last coordinate of each tensor, ascending, every entry a
 * multiple of 4 except the last, which is P; wd_scale_dev [n_tensors] (device, float): the factor (0 switches weight
 * decay off for that tensor, 1 leaves it).  Both arrays are borrowed until qsr_destroy or the next call;
 * n_tensors = 0 restores the uniform weight decay.  The library does not read the arrays on the host, so a table that
 * breaks these rules is not detected. */
int qsr_set_tensor_table(qsr_ctx *ctx, int32_t n_tensors, const int64_t *tensor_end_dev, const float *wd_scale_dev);

/* Gradient clipping by global norm (App. C.2: threshold 1 for parallel AdamW, 4 for Local AdamW with constant H under
 * linear decay, off in the QSR runs), in the form of the paper's software: before OPT each worker's gradient is scaled
 * by min(1, max_norm / (||g||_2 + 1e-6)), the norm over all P coordinates of that worker (for qsr_parallel_step: of the
 * averaged gradient).  While it is on, every step launches two more kernels first: per-worker partial sums of g^2
 * (generated gradients are recomputed, not stored) and the K factors.  Inside qsr_run, where the library issues the
 * steps of a round itself and nothing else touches the parameters in between, a plain step also computes its
 * successor's partial sums from the new parameters it holds in registers, so only the first step of a round pays the
 * norm pass (two launches per step instead of three, and no second read of the parameters); the factors are the same
 * bits either way.  workspace_dev: caller-owned device memory of qsr_clip_workspace_floats(ctx) floats (one partial
 * sum per worker and block of a step launch, so it grows with P: K * P / 256 + K floats), 16-byte aligned, borrowed
 * until clipping is switched off or the context is destroyed.  max_norm <= 0, infinite or NaN switches clipping off.
 * QSR_ERANGE if K exceeds 96.  The norm pass keeps K x (step threads) sums in shared memory: a step block size
 * above 512 with K near 96 does not fit and makes the step return QSR_ECUDA. */
int64_t qsr_clip_workspace_floats(const qsr_ctx *ctx);
int qsr_set_grad_clip(qsr_ctx *ctx, double max_norm, float *workspace_dev);

/* theta[k, :] <- theta0_dev[0..P) for every worker k: "each worker gets a local copy of the global iterate"
 * (Sec. 2).  Asynchronous. */
int qsr_set_params(qsr_ctx *ctx, const float *theta0_dev);

/* One local step of every worker at global iteration t (Eq. 1, inner loop of Algorithm 2), with learning rate
 * eta_t and, for AdamW, bias corrections for n = t + 1 - t_state_origin, all evaluated on the host in binary64.
 * grads == NULL: the gradient is generated inside the kernel (formula above) and never stored.
 * grads != NULL: [K, row_stride] device slab read as the workers' gradients.  One kernel launch; asynchronous. */
int qsr_local_step(qsr_ctx *ctx, int64_t t, const float *grads);

/* End of a round (Algorithm 2): theta_bar[i] = (1/K) * sum_k theta[k,i], summed in fp32 for k = 0..K-1 and divided
 * by K, then copied to every row; optimizer state treated per state_sync.  In RESET mode the bias-correction origin
 * moves to t_next (the first step of the next round).  One kernel launch, two in RESET mode (the zero-fill of the
 * state slabs is a launch of its own: a pure write stream is fastest when it is not mixed into the averaging's
 * loads); asynchronous. */
int qsr_sync(qsr_ctx *ctx, int64_t t_next);

/* The last local step of a round and the averaging that ends it (Eq. 1 followed by the All-Reduce line of
 * Algorithm 2) in ONE launch: the result is bit-identical to qsr_local_step(ctx, t, grads) followed by
 * qsr_sync(ctx, t_next), but the parameters are read once and written once, so the averaging adds no memory
 * traffic.  Only state_sync = QSR_STATE_KEEP can be fused; in the other modes this call issues the two launches.
 * qsr_run uses it for the last step of every round.  Asynchronous. */
int qsr_local_step_sync(qsr_ctx *ctx, int64_t t, const float *grads, int64_t t_next);

/* One iteration of Algorithm 1 (Parallel OPT), the data-parallel baseline that synchronizes at every step: the single
 * model is ROW 0 of params / state1 / state2 (rows 1..K-1 are neither read nor written); the K workers' gradients
 * are taken at that one point, summed in fp32 for k = 0..K-1, divided by K (the All-Reduce line), and one
 * optimizer step with learning rate eta_t follows.  grads as in qsr_local_step (NULL: generated; else [K, row_stride]).
 * With SGD (momentum included, state kept) this is what Local SGD does with H = 1 (Sec. 3).  One launch; asynchronous. */
int qsr_parallel_step(qsr_ctx *ctx, int64_t t, const float *grads);

/* The same synchronization split in two for workers sharded over several GPUs: qsr_sync_partial writes
 * sum[i] = sum_k theta[k,i] over this process's rows (and, in AVERAGE mode, the sums of state1 / state2 to
 * sum + P and sum + 2P, each region rounded up to a multiple of 4 floats); the caller all-reduces `sum` over
 * processes (SUM); qsr_sync_finish divides by K_total and writes every local row (and applies state_sync).
 * `sum` holds qsr_sync_sum_floats(ctx) floats. */
int64_t qsr_sync_sum_floats(const qsr_ctx *ctx);
int qsr_sync_partial(qsr_ctx *ctx, float *sum);
/* The round's last local step fused with qsr_sync_partial (state_sync = QSR_STATE_KEEP; otherwise the two launches are
 * issued): the kernel writes the row sums of the NEW parameters to `sum` and does not write the parameter rows at all
 * -- qsr_sync_finish overwrites every row with the global mean anyway -- so a sharded round end costs 4 B per update
 * less than a plain step.  After this call the parameter slab holds the pre-step values until qsr_sync_finish runs. */
int qsr_local_step_partial(qsr_ctx *ctx, int64_t t, const float *grads, float *sum);
int qsr_sync_finish(qsr_ctx *ctx, const float *sum, int32_t K_total, int64_t t_next);

/* A synchronization for callers that have no device buffer to spare and may not create one.  The paper has no
 * counterpart to this call: it exists for the way this library gets used.  Some hosts of this code run inside a
 * process whose device memory is handed out once, up front, by another component (a serving runtime, a framework's
 * caching allocator with a hard budget, a job that has already filled the GPU with its slabs), and some call from
 * places where cudaMalloc is not welcome because it stalls the whole device or is simply not permitted there.
 * Such callers cannot provide the `sum` buffer that qsr_sync_partial / qsr_sync_finish need.
 *
 * qsr_sync_static does the same two phases -- row sums, then rows <- sums / K (and the state_sync treatment) --
 * through a fixed array of QSR_STATIC_SCRATCH_FLOATS floats that is part of the library image, so every GPU that
 * loads the library holds that much memory until the process exits.  The call allocates and frees nothing.  The
 * result equals qsr_sync's: the same fp32 sum over k = 0..K-1 and the same single division by K.
 *
 * Limits and rules
 *   - The sums must fit: (P rounded up to 4) floats, times 1 + the number of state slabs in AVERAGE mode, must not
 *     exceed QSR_STATIC_SCRATCH_FLOATS.  Larger problems get QSR_ERANGE and nothing is launched; use qsr_sync, or
 *     qsr_sync_partial / qsr_sync_finish with a buffer of your own.
 *   - The first call on a device looks up the array's device address (once per device) and keeps it for the life of
 *     the process.  Make that first call before any stream capture begins.  The device the context was created on
 *     must be current (QSR_ESTATE otherwise, nothing launched).  Contexts on different host threads may make their
 *     first calls at the same time.  cudaDeviceReset destroys the array the kept address points to: do not call
 *     qsr_sync_static in a process that has reset the device after using it.
 *   - All contexts and all calls in the process share the one array.  Each call overwrites what it needs before
 *     reading it, so an earlier call's leftovers are harmless; but two calls whose kernels can overlap on the GPU
 *     (different streams, no ordering between them) race on it.  Keep the calls on one stream or order them.
 * Two kernel launches (three in RESET mode); asynchronous. */
#define QSR_STATIC_SCRATCH_FLOATS (1 << 20) /* 4 MiB */
int qsr_sync_static(qsr_ctx *ctx, int64_t t_next);

/* Algorithm 2 from t_begin (which must be the first step of a round) until the first round end >= t_end
 * (t_end <= T): per round GetH, H local steps with generated gradients, one synchronization.  The start and
 * length of each round are written to the host arrays round_start / round_len (cap entries, may be NULL with
 * cap = 0) and their count to *n_rounds (may be NULL).  Asynchronous: kernels are only enqueued. */
int qsr_run(qsr_ctx *ctx, int64_t t_begin, int64_t t_end,
            int64_t *round_start, int64_t *round_len, int64_t cap, int64_t *n_rounds);

/* Replays qsr_run's launches from CUDA graphs (Algorithm 2's round as one graph).  For small parameter sets a local
 * step takes a few microseconds on the device and a run is bound by the cost of launching H(s) kernels per round;
 * with max_steps_per_graph = G > 0, qsr_run enqueues each round as chains of at most G step kernels, each chain one
 * graph launch (a round's last chain ends in the fused step-and-average launch when state_sync = QSR_STATE_KEEP).
 * A chain of a given length is built and instantiated once, kept in the context (at most 48 distinct lengths; beyond
 * that, and whenever gradient clipping is on, qsr_run launches directly as before) and replayed with the arguments of
 * its steps -- learning rate, bias corrections, noise counter -- rewritten on the host before every replay.  The
 * kernels, their order and their arguments are those of the direct path, so the results are bit-identical.
 * G = 0 (the default) switches replay off.  QSR_ERANGE unless 0 <= G <= 1024.  Changing the launch shape discards the
 * cached graphs.  qsr_run must not itself be called while its stream is being captured when replay is on.
 * Whether it pays depends on the host: rewriting a node's arguments costs about as much host time as launching the
 * kernel, so on B200 with 1 MiB slabs and rounds of 4-8 steps a replayed run was 12 % slower than the direct one;
 * it is off unless asked for. */
int qsr_set_graph_replay(qsr_ctx *ctx, int32_t max_steps_per_graph);

/* BENCHMARK-ONLY: several local steps per launch with the parameters and the optimizer state held in registers in
 * between (Algorithm 2's inner "for h" loop inside one kernel).  This is possible only because the synthetic gradient
 * is generated in the kernel; a training loop has to return to the host after every step for its next gradient, so
 * no number measured with this switch on describes the path a real run takes.  What it shows is what the per-step
 * launches cost when the whole problem fits in cache: with 1 MiB slabs a step kernel takes ~4 us of launch latency
 * for ~0.5 us of arithmetic.
 * With max_steps_per_launch = N in 1..128, qsr_run packs consecutive steps into launches of at most N steps: every
 * thread owns one worker's four coordinates, reads them once, takes the steps (per-step learning rate and bias
 * corrections arrive as kernel arguments) and writes them once.  One block holds all K rows of its columns, so with
 * state_sync = QSR_STATE_KEEP the averaging at a round end happens inside the launch (through shared memory, k
 * ascending, one division: the bits of qsr_local_step_sync) and a launch runs across round ends; in the other state
 * modes a launch stops at the round end and qsr_sync follows.  Results are bit-identical to per-step launches.
 * N = 0 (the default) switches it off.  QSR_ERANGE for N outside 0..128 or K > 32.  While a tensor table or gradient
 * clipping is set, qsr_run launches per step as before.  Takes precedence over graph replay. */
int qsr_set_resident_steps(qsr_ctx *ctx, int32_t max_steps_per_launch);

/* Kernel launches issued through this context so far (a replayed graph counts its kernels). */
int64_t qsr_launch_count(const qsr_ctx *ctx);

/* Overrides the launch shape of the step kernel (threads per block: 64..1024, a multiple of 32; rows in flight per
 * thread, i.e. the depth of its cp.async ring: 1, 2, 4 or 8) and of the sync kernel (threads per block: 64..512).
 * 0 keeps the current value.  The ring takes rows x operands x threads x 16 bytes of shared memory (operands: 2 for
 * SGD, 3 for AdamW, one more with a gradient slab); a shape beyond 227 KB makes the next step return QSR_ECUDA. */
int qsr_set_launch_shape(qsr_ctx *ctx, int32_t step_threads, int32_t step_rows_in_flight, int32_t sync_threads);

/* ---- whole run from host memory ----------------------------------------------------------------------- */

/* Algorithm 2 from theta_bar(0) to theta_bar(R) for callers whose data lives in host memory: copies
 * theta0_host, lambda_host, theta_star_host ([P] each, pinned or pageable) to the device workspace, gives every
 * worker a copy of theta0, zeroes the optimizer state, runs steps [0, t_end) as qsr_run does, copies worker 0's
 * parameters (all workers are equal after the last synchronization) to theta_out_host [P], and waits for the
 * stream.  workspace_dev: caller-owned device memory of at least qsr_workspace_bytes(cfg) bytes, 256-byte aligned.
 * cfg->row_stride is ignored (rows are laid out at qsr_row_stride_hint(P)).  round_* / n_rounds as in qsr_run;
 * *launches (may be NULL) receives the number of kernel launches. */
int qsr_train_host(const qsr_config *cfg, const float *theta0_host, const float *lambda_host,
                   const float *theta_star_host, float *theta_out_host,
                   void *workspace_dev, int64_t workspace_bytes, int64_t t_end, void *cuda_stream,
                   int64_t *round_start, int64_t *round_len, int64_t cap, int64_t *n_rounds, int64_t *launches);

/* ---- test hook ---------------------------------------------------------------------------------------- */

/* The two halves of the Box-Muller transform that turns generator words into the synthetic gradient's noise (the
 * stand-in for Sample() and back-propagation in Algorithm 2; formula at qsr_config), evaluated by the same device
 * code the step kernels inline.  For each of the n words w in words_dev (device, uint32), with the 23-bit field
 * a = w >> 9 and u = (a + 1/2) / 2^23:  radius_dev[i] = sqrt(-2 ln u), sin_dev[i] = sin(2 pi u), cos_dev[i] = cos(2 pi u)
 * (device, float, n each; 4-byte aligned).  A step uses the radius of one word with the sine / cosine of the next.
 * The field has only 2^23 values, so a test can compare every one with binary64.  No context; one launch on
 * cuda_stream; asynchronous.  QSR_EINVAL for n < 0 or a NULL array with n > 0. */
int qsr_debug_box_muller(const uint32_t *words_dev, int64_t n, float *radius_dev, float *sin_dev, float *cos_dev,
                         void *cuda_stream);

/* The two single-instruction special functions inside OPT of Eq. 1 as this library evaluates it (App. C.2's AdamW:
 * the root of the second moment and the quotient m / denominator; the root also gives the Box-Muller radius):
 * sqrt_dev[i] = sqrt.approx.ftz(x_dev[i]), rcp_dev[i] = rcp.approx.ftz(x_dev[i]) for n floats (device arrays, 4-byte
 * aligned).  For tests that bound their error against binary64.  No context; one launch on cuda_stream; asynchronous. */
int qsr_debug_fast_math(const float *x_dev, int64_t n, float *sqrt_dev, float *rcp_dev, void *cuda_stream);

/* Text for a qsr_status. Never NULL. */
const char *qsr_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* QSR_H_ */
