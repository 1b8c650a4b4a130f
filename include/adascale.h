/*
 * adascale.h - C ABI of the AdaScale SGD gain-ratio step on one NVIDIA B200 (sm_100a).
 *
 * Paper: Johnson, Agrawal, Gu, Guestrin, "AdaScale SGD: A User-Friendly Algorithm for
 * Distributed Training" (ICML 2020).  One call of adascale_step is one iteration of the
 * paper's Algorithm 2 after the S per-batch gradients have been produced:
 *
 *   gbar     = (1/S) sum_i g_i                                   (Sec. 2, "scaled SGD")
 *   sigma^2  = 1/(S-1) sum_i ||g_i||^2 - S/(S-1) ||gbar||^2       (App. B.3)
 *   mu^2     = ||gbar||^2 - sigma^2 / S                           (App. B.3)
 *   clamps, moving averages with parameter theta                 (App. B.3, Sec. 3.4)
 *   r_t      = (sigma_bar^2 + mu_bar^2) / (sigma_bar^2/S + mu_bar^2)   (Eq. 3)
 *   eta_t    = r_t * lr(floor(tau_t));  tau_{t+1} = tau_t + r_t   (Sec. 3.2)
 *   v <- rho v + (gbar + lambda w);  w <- w - eta_t v              (Eq. 2 with momentum, Sec. 3.4)
 *
 * Everything above runs in CUDA kernels; nothing is computed on the host and no call
 * except adascale_get_gain_tau(blocking), adascale_get_state, adascale_set_state,
 * adascale_step_host and adascale_destroy waits for the device (one exception: the call that
 * first sees a new tiling uploads it and waits for that upload, see adascale_step).
 *
 * Conventions
 *   - "device pointer" = address in the global memory of the context's GPU;
 *     "host pointer"   = ordinary host memory.  Arrays OF pointers are always host arrays.
 *   - The caller owns gradients, parameters and momentum.  The library owns the mean
 *     gradient, its scratch and its state, all allocated in adascale_init.
 *   - Tensors are dense and contiguous.  A tensor whose S gradient pointers (or whose
 *     parameter/momentum pointers) are all 16-byte aligned takes the 128-bit path; any
 *     other alignment (to the element size) is accepted and takes a scalar path.
 *   - Every function returns an adascale_status; nothing throws, aborts or traps.
 *   - One context is used from one stream at a time.  Calls on a context are not
 *     thread-safe against each other.
 */
#ifndef ADASCALE_H_
#define ADASCALE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adascale_ctx adascale_ctx; /* opaque */

typedef enum {
    ADASCALE_OK = 0,
    ADASCALE_ERR_INVALID_ARG = 1, /* null pointer, S < 1, no tensors, bad enum, ...      */
    ADASCALE_ERR_ALIGNMENT = 2,   /* a pointer is not aligned to its element size        */
    ADASCALE_ERR_CUDA = 3,        /* a CUDA runtime call failed; see adascale_last_error */
    ADASCALE_ERR_STATE = 4,       /* call order (update before reduce, capture rules)    */
    ADASCALE_ERR_TOO_LARGE = 5    /* size beyond a documented maximum                    */
} adascale_status;

typedef enum { ADASCALE_F32 = 0, ADASCALE_BF16 = 1 } adascale_dtype;

/* Learning-rate families of App. B.1; t is floor(tau_t) unless ADASCALE_FLAG_CONT_TAU. */
typedef enum {
    ADASCALE_LR_CONST = 0, /* lr(t) = eta0                                            */
    ADASCALE_LR_EXP = 1,   /* lr(t) = eta0 * decay^(t / t_s1)                          */
    ADASCALE_LR_STEP = 2   /* lr(t) = eta0 * decay^(#{i : t > milestones[i]})  (strict) */
} adascale_lr_kind;

#define ADASCALE_MAX_MILESTONES 8

typedef struct {
    int32_t kind;         /* adascale_lr_kind                                        */
    int32_t n_milestones; /* 0..ADASCALE_MAX_MILESTONES, step family only             */
    double eta0;          /* eta_0 > 0                                                */
    double decay;         /* d > 0                                                    */
    double t_s1;          /* T_{S=1} > 0, exponential family only                     */
    double milestones[ADASCALE_MAX_MILESTONES]; /* w_i, in scale-invariant iterations */
} adascale_lr_schedule;

/* flags */
#define ADASCALE_FLAG_LAGGED 1u   /* r_t from the averages of prior iterations only, r_0 = 1
                                     (the variant App. B.3 says the paper's runs used)    */
#define ADASCALE_FLAG_CONT_TAU 2u /* evaluate lr at tau_t instead of floor(tau_t)          */
#define ADASCALE_FLAG_RATIO 4u    /* estimator of Sec. 3.4: r = (m1 + eps) / (m2 + eps)    */
#define ADASCALE_FLAG_FUSED 8u    /* with ADASCALE_FLAG_LAGGED only: eta_t is known before the
                                     gradients are read, so one kernel reads the S rows, w and v
                                     and writes w and v; the mean gradient is never stored.  Only
                                     adascale_step and adascale_step_host run an iteration
                                     (reduce, update, mean_grad return ERR_STATE), and non-finite
                                     gradients have already reached their own coordinates of w
                                     and v when they are detected (the state and tau still skip) */
#define ADASCALE_FLAG_GRADS_READY 16u /* the caller vouches that every gradient row was completely
                                     written before the step's first kernel can start: the rows were
                                     produced on another stream and joined by an event, or the last
                                     kernel before the step on `cuda_stream` does not trigger
                                     programmatic dependent launches before its last gradient store
                                     (kernels that never use that feature qualify).  The reduce kernel
                                     then starts streaming the rows while the previous kernel in the
                                     stream still drains.  Without the flag it waits for that kernel
                                     first, which is always safe.  No counterpart in the paper.      */

typedef struct {
    int32_t S;              /* scale: gradient rows per iteration, >= 1                */
    int32_t max_S;          /* largest S adascale_set_scale may set; 0 means S         */
    int32_t n_tensors;      /* T >= 1                                                  */
    int32_t grad_dtype;     /* adascale_dtype of the gradient rows                     */
    const int64_t *numel;   /* host array [T], elements per tensor (>= 0); copied      */
    double momentum;        /* rho                                                     */
    double weight_decay;    /* lambda, added to gbar in the update only                */
    double eps;             /* epsilon of App. B.3 / Sec. 3.4; the paper suggests 1e-6 */
    double theta;           /* moving-average parameter in [0,1); < 0 selects the
                               paper's rule max(1 - S/1000, 0), which follows S        */
    uint32_t flags;         /* ADASCALE_FLAG_*                                         */
    int32_t device;         /* CUDA device ordinal                                     */
} adascale_config;

/* status bits reported in adascale_stats.status_bits */
#define ADASCALE_STATUS_NONFINITE 1u    /* last step saw inf/nan sums and was skipped           */
#define ADASCALE_STATUS_WAIT_TIMEOUT 2u /* sticky: a bounded wait inside the reduce kernel gave up.
                                           That step and every later one is skipped: the state and
                                           tau do not advance, `skipped` counts them, and w and v
                                           stay as they were (one-pass mode: the tiles that the
                                           kernel had reached before giving up are already updated).
                                           The mean gradient of that step is incomplete.
                                           adascale_set_state clears the condition.              */

typedef struct {
    double r;           /* gain ratio r_t of the last step                            */
    double tau;         /* scale-invariant iteration after the last step, tau_{t+1}   */
    double eta;         /* learning rate the last step applied, r_t * lr              */
    double lr;          /* lr(floor(tau_t))                                            */
    double sigma2_raw;  /* sigma_hat^2 before the clamp                                */
    double mu2_raw;     /* mu_hat^2 before the clamp                                   */
    double sigma2_avg;  /* sigma_bar^2  (ratio estimator: m1)                          */
    double mu2_avg;     /* mu_bar^2     (ratio estimator: m2)                          */
    double gbar_sqnorm; /* ||gbar||^2                                                  */
    double dev_sqsum;   /* sum_i ||g_i - gbar||^2                                      */
    int64_t t;          /* iterations applied                                          */
    int64_t n_samples;  /* samples absorbed by the moving averages                     */
    int64_t skipped;    /* iterations skipped because of non-finite sums               */
    uint32_t status_bits;
    uint32_t reserved;
} adascale_stats;

#define ADASCALE_STATE_BYTES 128

/*
 * Algorithm 2, inputs (w_0, lr, T_SI, X, S): fixes S, the tensor list and the constants,
 * allocates the library's device memory (mean gradient 4*P bytes, per-block partial
 * sums, pointer tables, state) on cfg->device and zeroes the state (tau_0 = 0).
 * cfg and cfg->numel are host pointers, read during the call only.  *out receives the
 * context.  Errors: INVALID_ARG (null, S < 1, T < 1, negative numel, theta >= 1,
 * unknown dtype), CUDA.  Launches no kernel.
 */
adascale_status adascale_init(const adascale_config *cfg, adascale_ctx **out);

/*
 * One iteration (Sec. 3.2, App. B.3, Eq. 2-3): reduce + update, two kernel launches on
 * `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream); three for jobs whose
 * tiles are handed out in runs (see adascale_tiling), where a small kernel between the two
 * adds up the partial sums of the runs.  Returns after
 * enqueueing.  It waits for the device in one case only: when the tiling has to be rebuilt
 * (first call, a new S, a tensor whose 16-byte alignment changed) the tile descriptors are
 * uploaded and the call waits for that upload.
 *   grads    host array [S * T] of device pointers; row i, tensor k at [i*T + k];
 *            element type cfg.grad_dtype; read only.
 *   params   host array [T] of device pointers, float32, updated in place.
 *   momentum host array [T] of device pointers, float32, updated in place.
 *   sched    host pointer, read during the call.
 * When the pointer values differ from the previous call the library re-uploads its
 * pointer table with one asynchronous copy from pinned memory; inside a stream capture
 * that is refused with ERR_STATE (capture a step whose pointers were already seen).
 * A step whose sums are not finite changes nothing (state, tau, parameters, momentum)
 * and raises ADASCALE_STATUS_NONFINITE; this policy is an extension, the paper is silent.
 * Ordering on the stream: the step's kernels are launched with programmatic dependent launch
 * among themselves.  The gradient rows are read only after the kernel that precedes the step
 * on `cuda_stream` has completed, unless cfg.flags carries ADASCALE_FLAG_GRADS_READY.
 */
adascale_status adascale_step(adascale_ctx *ctx, const void *const *grads, void *const *params,
                              void *const *momentum, const adascale_lr_schedule *sched,
                              void *cuda_stream);

/*
 * First half of adascale_step: streams the S x P gradient matrix once, writes gbar,
 * forms sum_i ||g_i - gbar||^2 and ||gbar||^2 and runs the scalar part (estimates,
 * averages, r_t, eta_t, tau_{t+1}) on the device (Sec. 3.2, App. B.3, Eq. 3).
 * Arguments as in adascale_step.  One kernel launch, two when the tiles are handed out in runs.
 * Where the scalar part runs is the library's business: the reduce kernel stops at pairs of
 * partial sums (one per block; with runs, one per run, brought down to a few dozen by a small
 * second kernel) and the kernel that follows completes the iteration - the update kernel of
 * adascale_update / adascale_step, each of whose blocks adds up the pairs itself, or, when
 * adascale_get_gain_tau, adascale_get_state, adascale_apply_sums or another adascale_reduce
 * comes first, a one-block kernel that the library enqueues before serving that call (one
 * more launch in adascale_launch_count).  The state a caller reads is the same either way.
 */
adascale_status adascale_reduce(adascale_ctx *ctx, const void *const *grads,
                                const adascale_lr_schedule *sched, void *cuda_stream);

/*
 * Second half: v <- rho v + (gbar + lambda w); w <- w - eta_t v with the eta_t that the
 * preceding adascale_reduce left on the device (Eq. 2, Sec. 3.4), or that this kernel
 * completes itself where the reduce launch left the scalar part open.  ERR_STATE if no
 * reduce precedes it.  One kernel launch.
 */
adascale_status adascale_update(adascale_ctx *ctx, void *const *params, void *const *momentum,
                                void *cuda_stream);

/*
 * Column-sharded use on several GPUs (Sec. 2: the S workers' gradients are combined; here
 * every GPU holds all S rows of ITS slice of the parameters, its own context over that
 * slice, and the only exchange is the pair of sums).  adascale_reduce_sums is
 * adascale_reduce without the scalar part: it writes the mean gradient of the slice and the
 * slice's two sums, sums[0] = sum_i ||g_i - gbar||^2 and sums[1] = ||gbar||^2 (device
 * pointer, 2 float64, 8-byte aligned), and leaves the state alone.  The caller adds the
 * pairs of all GPUs (for instance an NCCL all-reduce of 16 bytes on the same stream), after
 * which adascale_apply_sums runs the scalar part of App. B.3 / Eq. 3 / Sec. 3.2 on the
 * completed sums and then the update of Eq. 2 for the slice.  Every GPU sees the identical
 * two numbers and therefore computes the identical r_t, eta_t and tau.  Other arguments as in
 * adascale_step.  Errors as there; ERR_STATE in the one-pass (fused) mode.
 */
adascale_status adascale_reduce_sums(adascale_ctx *ctx, const void *const *grads, void *sums, void *cuda_stream);
adascale_status adascale_apply_sums(adascale_ctx *ctx, const void *sums, const adascale_lr_schedule *sched,
                                    void *const *params, void *const *momentum, void *cuda_stream);

/*
 * tau drives the caller's stopping test tau_t >= T_SI (Sec. 3.2); r_t and eta_t are what
 * the paper plots.  Copies the device state into *out (host pointer).  blocking != 0
 * waits for every step enqueued so far on the context's last stream; blocking == 0
 * returns the most recent snapshot that has already arrived (zeros before the first)
 * and enqueues a fresh asynchronous snapshot.
 */
adascale_status adascale_get_gain_tau(adascale_ctx *ctx, adascale_stats *out, int blocking);

/*
 * *gbar (host array [T], filled by the call) receives device pointers to the float32
 * mean gradient of each tensor (Sec. 2).  Library-owned; contents valid after a reduce
 * completes and until the next one starts.
 */
adascale_status adascale_mean_grad(adascale_ctx *ctx, const void **gbar);

/*
 * Elastic scaling (Sec. 4, the imagenet experiment of Fig. 4: S changes abruptly, nothing
 * else does): sets S for the following steps, 1 <= S <= max_S.  The moving averages and tau
 * carry over; theta follows S when it was left to the paper's rule.
 */
adascale_status adascale_set_scale(adascale_ctx *ctx, int32_t S);

/*
 * Every wait inside the reduce kernel (consumer warps waiting for a stage of rows, the producer
 * warp waiting for a free stage) gives up after a number of polls and raises
 * ADASCALE_STATUS_WAIT_TIMEOUT instead of hanging.  This sets that number for the following
 * steps (default 4,194,304; 0 makes every such wait give up at once).  It exists so that the
 * give-up path can be exercised by a test; the wait for copies that are already in flight when
 * a block gives up keeps its own fixed bound, so a block never leaves while data is still
 * arriving in its shared memory.  No counterpart in the paper.
 */
adascale_status adascale_set_wait_limit(adascale_ctx *ctx, uint32_t polls);

/*
 * How the reduce kernel hands its tiles to the blocks, for the following steps: run_tiles = -1
 * (default) lets the library choose by the job's size (see adascale_tiling); 0 assigns tile t to
 * block t mod grid; 1 .. 64 hands out runs of that many consecutive tiles from a device
 * counter (the tiles of the last runs of a launch - two runs per block, at most half of all -
 * one by one).  Every setting gives sums that are reproducible from run to run; different settings
 * add the same terms in different orders and so may differ in the last bits.  It exists for
 * tests (so that small jobs can exercise the path of large ones) and for tuning.  No counterpart
 * in the paper.  Errors: INVALID_ARG.
 */
adascale_status adascale_set_tile_runs(adascale_ctx *ctx, int32_t run_tiles);

/*
 * Checkpoint / resume of the scalar state (tau, averages, counters): buf is a host
 * buffer of ADASCALE_STATE_BYTES.  Both calls wait for the device.  set_state rejects a
 * buffer that get_state did not write (INVALID_ARG).  No counterpart in the paper.
 */
adascale_status adascale_get_state(adascale_ctx *ctx, void *buf);
adascale_status adascale_set_state(adascale_ctx *ctx, const void *buf);

/*
 * adascale_step for callers whose gradients live in host memory: grads is a host array
 * [S * T] of HOST pointers.  The rows are copied to library-owned device staging
 * (allocated on first use, S * P elements), the step runs, the statistics are copied
 * back into *out (may be NULL) and the call returns after the device has finished.
 * params and momentum stay device pointers: they are the optimiser's resident state.
 */
adascale_status adascale_step_host(adascale_ctx *ctx, const void *const *grads, void *const *params,
                                   void *const *momentum, const adascale_lr_schedule *sched,
                                   adascale_stats *out, void *cuda_stream);

/*
 * Bandwidth probes used to calibrate the roofline (no counterpart in the paper):
 * kind 0 reads `a` (n_bytes) and folds it into a checksum (b: device scratch of at least
 * 16 bytes), kind 1 copies a -> b, kind 2 does a[i] += b[i] in place (read a, read b,
 * write a).  a, b: device pointers on the current device, 16-byte aligned, n_bytes a
 * multiple of 16.  One launch on `cuda_stream`.
 */
adascale_status adascale_stream_probe(int32_t kind, void *a, void *b, int64_t n_bytes, void *cuda_stream);

/*
 * Host-only view of how the reduce kernel tiles a tensor list (no counterpart in the paper;
 * used by tests and for sizing).  numel: host array [n_tensors]; aligned: host array
 * [n_tensors], non-zero where all S gradient pointers of the tensor are 16-byte aligned
 * (NULL = all aligned); n_blocks: grid size the tiling is tuned for.  Writes the number of
 * staged tiles before each tensor into tprefix[0..n_tensors] and of scalar-path tiles into
 * sprefix[0..n_tensors], the columns of one staged tile into *tile_cols and the rows of one
 * shared-memory stage into *rows.  With fewer than 32768 staged tiles, or S <= 8, tile t is
 * processed by block t mod gridDim; larger jobs hand runs of 2 or 4 consecutive tiles (single
 * tiles at the end of a launch) to the blocks as they become free, and the sums are added up
 * per run and then over the runs in a fixed order, so the result does not depend on which block
 * processed which run (see adascale_set_tile_runs).  Makes no CUDA call.  Errors: INVALID_ARG.
 */
adascale_status adascale_tiling(const int64_t *numel, int32_t n_tensors, int32_t grad_dtype, int32_t S,
                                const uint8_t *aligned, int32_t n_blocks, int64_t *tprefix, int64_t *sprefix,
                                int32_t *tile_cols, int32_t *rows);

/*
 * The two sums and the mean gradient of ONE tensor without any allocation (the paper has no
 * counterpart; the sums are those of App. B.3 in the form the reduce kernel uses:
 * sums[0] = sum_i ||g_i - gbar||^2, sums[1] = ||gbar||^2).
 *
 * Who needs it: every other entry point works on a context, and adascale_init calls
 * cudaMalloc.  That is no use to a caller that is not allowed to allocate device memory: a
 * component that runs after start-up in a process where all device memory has already been
 * handed to another allocator, or one that must never risk the late failure or the implicit
 * device synchronisation that an allocation can bring.  Such a caller brings its own buffers
 * for inputs and outputs; what the kernel needs beyond them (a counter and one pair of
 * partial sums per block, about 16 KB) sits in a fixed array inside the library that every
 * GPU which loads the library holds until the process exits.  The row pointers are passed to
 * the kernel by value.  The call makes no cudaMalloc, cudaFree or other allocating call and
 * copies nothing from host memory.
 *
 *   rows        host array [S] of device pointers, 16-byte aligned, n elements of grad_dtype each
 *   S           1 .. ADASCALE_STATIC_MAX_ROWS
 *   n           1 .. ADASCALE_STATIC_MAX_NUMEL
 *   gbar        device pointer, n float32, 16-byte aligned: receives the mean gradient
 *   sums        device pointer, 2 float64, 8-byte aligned: receives the two sums
 *   cuda_stream stream of the current device; the call enqueues and returns
 * Larger S or n: ADASCALE_ERR_TOO_LARGE ("size beyond the documented maximum"); null or bad
 * dtype: INVALID_ARG; misaligned pointers: ALIGNMENT; a failing CUDA call: ERR_CUDA.
 *
 * The first call on a device looks up the array's device address and the device's size; make
 * that first call outside of any stream capture.  All calls on a device share the one array
 * and it keeps what the last call left there (the call resets what has to start at zero), so
 * two calls that can overlap on the GPU - different streams without an ordering between them,
 * or different host threads - race on it and give wrong results; order them.
 */
#define ADASCALE_STATIC_MAX_ROWS 32
#define ADASCALE_STATIC_MAX_NUMEL 2147483640LL
adascale_status adascale_grad_stats_static(const void *const *rows, int32_t S, int32_t grad_dtype, int64_t n,
                                           void *gbar, void *sums, void *cuda_stream);

/* Number of kernels the library has launched through this context since init. */
int64_t adascale_launch_count(const adascale_ctx *ctx);

/* Frees everything adascale_init allocated.  NULL is accepted. */
adascale_status adascale_destroy(adascale_ctx *ctx);

/* Static string for a status code. */
const char *adascale_strerror(adascale_status s);

/* Text of the last CUDA error seen by this context ("" if none); valid until the next call. */
const char *adascale_last_error(const adascale_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* ADASCALE_H_ */
