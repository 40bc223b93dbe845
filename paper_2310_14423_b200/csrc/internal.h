// Internal declarations shared by the library's translation units (not part of the C ABI).
#ifndef QSR_INTERNAL_H_
#define QSR_INTERNAL_H_

#include <cstddef>
#include <cstdint>

#include "../../include/qsr.h"

namespace qsr {

// schedule.cpp
int check_config(const qsr_config &c);
int64_t row_stride_hint(int64_t P);
double learning_rate(const qsr_config &c, int64_t t);
int64_t round_length(const qsr_config &c, int64_t t);

// Arguments of one local-step launch.  Scalars are evaluated on the host in binary64 and rounded once.
struct StepParams {
    float *theta, *s1, *s2;
    const float *grads;       // NULL: generate the gradient in the kernel
    const float *lambda, *theta_star;
    int64_t P, stride;
    int32_t K;
    uint32_t worker0;         // global index of row 0
    uint32_t round_key[20];   // Philox key schedule: round r uses (key0 + r*W0, key1 + r*W1) at [2r], [2r+1]
    uint32_t step;            // global iteration t (Philox counter word 2)
    float sigma;              // noise_std
    float eta, wd, mu;        // SGD with momentum
    float eta_wd;             // AdamW: eta * weight_decay
    float beta1, beta2, omb1, omb2;
    float step_size;          // AdamW: eta / (1 - beta1^n)
    float inv_sqrt_bc2;       // AdamW: 1 / sqrt(1 - beta2^n)
    float eps;
    float inv_K;              // 1 / K (exact when K is a power of two)
    int32_t n_tensors;             // 0: uniform weight decay
    const int64_t *tensor_end;     // device [n_tensors]: one past each tensor's last coordinate, ascending
    const float *wd_scale;         // device [n_tensors]: factor on the weight decay of each tensor
    const float *clip_coef;        // NULL, or device [K] ([1] for Algorithm 1): gradient-clipping factor per worker
    float *sum_out;                // step fused with the partial sums of a sharded synchronization: device [P4]
    float *norm_partial;           // not NULL: the step also leaves the NEXT step's gradient-norm partials here
};

constexpr int kNormGrid = 1184;    // blocks of Algorithm 1's gradient-norm pass (8 per SM on a 148-SM part)
constexpr int kNormThreads = 128;  // its block size
constexpr int kMaxClipK = 96;      // Local OPT's norm pass keeps K x threads sums in shared memory

struct SyncParams {
    float *slab[3];           // arrays to average (theta first), then arrays to zero
    int32_t n_mean, n_zero;
    int64_t P, stride;
    int32_t K;
    float *sum_out;           // partial mode: per-array sums, array a at sum_out + a*P4
    const float *sum_in;      // finish mode: all-reduced sums
    int64_t P4;               // P rounded up to a multiple of 4
    float divisor;            // K (or the global worker count in finish mode)
};

struct LaunchShape {
    // Defaults from sustained sweeps on B200 at the ViT-B/16 and ResNet-152 shapes (K = 16): an 8-row cp.async ring
    // per thread, in 256-thread blocks for AdamW (96 KiB of ring, two blocks per SM) and 128-thread blocks for SGD
    // (32 KiB, 0.7 % faster there than 256; qsr_init picks).  Grids capped at a few CTAs per SM with a grid-stride loop
    // were 15-30 % slower than one thread per column.
    int step_threads = 256;
    int step_rows = 0;        // rows in flight per thread (ring depth); 0 = default (8)
    int sync_threads = 128;
};

// How the step kernel ends: plainly, with the replica mean written to every row (a round's last step), or with the
// row sums written to StepParams::sum_out (a round's last step when the workers are sharded over GPUs).
enum { FUSE_NONE = 0, FUSE_MEAN = 1, FUSE_SUM = 2 };

// Several consecutive local steps in ONE launch, parameters and optimizer state held in registers in between
// (possible only because the synthetic gradient is generated in the kernel: a training loop has to leave the device
// code after every step to get its next gradient).  Per-step scalars travel as kernel arguments.
constexpr int kMaxResidentSteps = 128;   // 2 KB of per-step scalars: the whole argument block stays below 4 KB
constexpr int kMaxResidentK = 32;        // the K rows of a column sit in one block of 32 columns x K threads
struct ResidentScalars {
    float eta, eta_wd, step_size, inv_sqrt_bc2;    // as in StepParams, for one step
};
struct ResidentParams {
    StepParams base;                     // pointers, sizes, noise key, constants; base.step is the first step
    int32_t n_steps;                     // 1..kMaxResidentSteps
    int32_t cols_per_block;
    uint32_t sync_after[kMaxResidentSteps / 32];   // bit h: step h ends a round -> average the parameters over the rows
    ResidentScalars per_step[kMaxResidentSteps];
};
int launch_resident_steps(const ResidentParams &q, int opt, void *stream);

// One instance of the step kernel with its launch geometry: what cudaLaunchKernel or a CUDA-graph kernel node needs.
// The kernel's only argument is a StepParams by value.
struct StepLaunch {
    const void *func;
    unsigned grid;
    int threads;
    size_t smem;
};
int resolve_step(const StepParams &p, int opt, const LaunchShape &shape, int fuse, StepLaunch *out);

// kernels.cu -- each returns a cudaError_t cast to int (0 = success) after enqueueing one kernel.
int launch_step(const StepParams &p, int opt, const LaunchShape &shape, void *stream);
int launch_step_mean(const StepParams &p, int opt, const LaunchShape &shape, void *stream);   // step + replica mean
int launch_step_sum(const StepParams &p, int opt, const LaunchShape &shape, void *stream);    // step + row sums to p.sum_out
int launch_parallel_step(const StepParams &p, int opt, const LaunchShape &shape, void *stream);  // Algorithm 1, row 0
// A synchronization that resets the optimizer state (n_zero > 0) zero-fills it in a second launch.
int launch_sync(const SyncParams &p, const LaunchShape &shape, void *stream);          // mean + write back [+ reset launch]
int launch_sync_partial(const SyncParams &p, const LaunchShape &shape, void *stream);  // sums only
int launch_sync_finish(const SyncParams &p, const LaunchShape &shape, void *stream);   // sums -> rows [+ reset launch]
inline int sync_launches(const SyncParams &p) { return p.n_zero > 0 ? 2 : 1; }       // of launch_sync / launch_sync_finish
int launch_broadcast(float *theta, const float *theta0, int64_t P, int64_t stride, int32_t K,
                     const LaunchShape &shape, void *stream);
// Gradient clipping.  Local OPT: the norm pass writes clip_norm_blocks(P, step threads) x K partial sums to ws (a step
// launched with StepParams::norm_partial set leaves the same numbers for its successor), the factor pass turns them
// into K factors at ws + blocks * K.  Algorithm 1: both passes at once, the factor at ws + clip_grid(P).
int clip_grid(int64_t P);
int64_t clip_norm_blocks(int64_t P, int threads);
int launch_clip_norms(const StepParams &p, float *ws, const LaunchShape &shape, void *stream);
int launch_clip_factors(float *ws, int64_t blocks, int rows, double max_norm, void *stream);
int launch_clip_coef_parallel(const StepParams &p, double max_norm, float *ws, void *stream);
// Dynamic shared memory of a step launch (the ring, plus next_norm_rows x threads floats).
size_t step_shared_bytes(int opt, bool ext_grad, int stages, int threads, int next_norm_rows);
// Test hook: radius, sine and cosine of the Box-Muller transform for n generator words (all device arrays).
int launch_box_muller_parts(const uint32_t *words, int64_t n, float *radius, float *sine, float *cosine, void *stream);
// Test hook: sqrt.approx.ftz and rcp.approx.ftz of n floats, as the optimizer update uses them.
int launch_fast_math(const float *x, int64_t n, float *root, float *reciprocal, void *stream);
// Both phases through the library's own static scratch; -1 if the sums exceed QSR_STATIC_SCRATCH_FLOATS, -2 if
// `device` (the context's) is not the current device.
int launch_sync_static(const SyncParams &p, const LaunchShape &shape, int device, void *stream);

}  // namespace qsr
#endif
