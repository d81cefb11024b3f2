/*
 * adagc.h -- C ABI of the fused AdaGC + AdamW optimizer step for NVIDIA B200 (sm_100a).
 *
 * The library implements one step of "AdamW with AdaGC" (Algorithm 1 of the paper):
 *   - per-tensor gradient norms ||g_t,i|| (Eq. 3) and, during warm-up, the global norm (Eq. 2);
 *   - the clip factor h: global-norm clipping against lambda_abs for the first T_start steps
 *     (warm-up branch of Algorithm 1), afterwards per tensor against lambda_rel * gamma_{t-1,i}
 *     (Eq. 3), where gamma_i is the EMA of that tensor's *clipped* norms;
 *   - the gamma update (min-seeding in warm-up, EMA with beta afterwards);
 *   - AdamW moments, bias correction, decoupled weight decay on the clipped gradient
 *     (last four lines of Algorithm 1).
 *
 * Conventions
 *   - All tensors of a model live in flat "arenas": params, grads, m, v share one element-offset
 *     table (tensor i occupies elements [offset, offset + numel) of every arena).
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller owns every
 *     buffer, including the workspace.  No entry point declared in this header allocates or frees
 *     device memory.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     adagc_step / adagc_clip only enqueue work; they never synchronise.
 *   - `step` is 1-based.  Steps 1..warmup use global-norm clipping; step warmup+1 is the first
 *     per-tensor AdaGC step.  At step 1 the incoming content of `d_ema` is ignored and gamma is
 *     seeded from that step's clipped norms, so no initialisation of `d_ema` is required.
 *   - Return value: 0 on success, a negative adagc_status otherwise; on error nothing was enqueued.
 *     Conditions found on the device (non-finite gradient norm) are reported through the status
 *     word returned by adagc_get_stats.  The library never prints and never aborts.
 */
#ifndef ADAGC_H_
#define ADAGC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adagc_ctx adagc_ctx; /* opaque, host-side */

typedef enum { ADAGC_F32 = 0, ADAGC_BF16 = 1 } adagc_dtype;

typedef enum {
  ADAGC_OK = 0,
  ADAGC_E_INVALID_ARG = -1, /* null pointer, numel <= 0, hyper-parameter outside its domain, ... */
  ADAGC_E_MISALIGNED = -2,  /* a tensor offset or an arena pointer is not 16-byte aligned */
  ADAGC_E_OVERLAP = -3,     /* two tensors of the descriptor overlap */
  ADAGC_E_WORKSPACE = -4,   /* workspace too small or misaligned */
  ADAGC_E_DTYPE = -5,       /* unsupported dtype combination */
  ADAGC_E_CUDA = -6,        /* a CUDA runtime call failed (no device, launch error, ...) */
  ADAGC_E_NOMEM = -7,       /* host allocation of the context failed */
  ADAGC_E_TOO_LARGE = -8,   /* adagc_sumsq_noalloc: more elements than its fixed scratch covers */
  ADAGC_E_POISONED = -9     /* ADAGC_FUSED_SMALL context after adagc_get_stats reported ADAGC_E_TIMEOUT */
} adagc_status;

/* Bits of the device status word (adagc_get_stats). */
#define ADAGC_W_NONFINITE 1 /* some tensor's sum of squares was Inf or NaN in some step */
#define ADAGC_E_TIMEOUT 2   /* a bounded device-side wait gave up (a bulk copy never completed): the
                               update of that step is incomplete */
#define ADAGC_E_BOUNDS 4    /* only in a library built with -DADAGC_BOUNDS_CHECK: a kernel found a chunk-table entry
                               that points outside the arenas (or is otherwise malformed); the blocks that saw it
                               returned without touching the arenas */

/* adagc_desc.flags: which kernel runs the AdamW update phase.  AUTO (0) currently picks the bulk-async
 * kernel (cp.async.bulk + mbarrier pipeline through shared memory), which measured 1-2 % faster than the
 * register-streaming kernel; the other two values force one path (the tests cover both). */
#define ADAGC_UPDATE_PATH_AUTO 0
#define ADAGC_UPDATE_PATH_REGISTERS 1
#define ADAGC_UPDATE_PATH_BULK 2
#define ADAGC_UPDATE_PATH_MASK 3
/* Two variants from the paper's ablations (Section 5), OR-ed into adagc_desc.flags:
 *   ADAGC_EMA_KEEP_INITIAL      "constant initialization": gamma is not seeded at step 1; the values the
 *                               caller put into d_ema (e.g. 0.5 or 1.0) serve as gamma_0.
 *   ADAGC_CLIP_GLOBAL_ADAPTIVE  "Global AdaGC": one adaptive threshold for the whole model -- the same
 *                               algorithm applied to the single tensor that all gradients form together.
 *                               Every tensor gets that clip factor and flag; all n_tensors entries of
 *                               d_ema hold the one gamma (entry 0 is the one read). */
#define ADAGC_EMA_KEEP_INITIAL 4
#define ADAGC_CLIP_GLOBAL_ADAPTIVE 8
/* Sharded use (Section 4.3 "Communication": with a tensor split over several devices, the per-tensor norm
 * needs one all-reduce of the partial sums of squares).  With this flag a tensor of the descriptor may have
 * numel == 0 -- this rank holds no element of it -- so that every rank keeps the same tensor numbering and
 * the same n_tensors-long vectors (gamma, sums of squares); the offset of an empty tensor is ignored. */
#define ADAGC_ALLOW_EMPTY 16
/* Small layouts: adagc_step runs as ONE kernel (norm, decisions and AdamW separated by grid-wide barriers inside a
 * cooperative launch) instead of two (four on warm-up steps).  Worth it only where the dependent launches cost more
 * than the data movement: measured on B200 against a three-launch step it halved the step time below about 100 chunks
 * of 16384 elements, broke even near 150 chunks (one per SM) and lost beyond (against today's two-launch step, 10.4
 * instead of 16.5 us on a layout of 37 chunks); accepted for layouts of at most 4096 chunks (adagc_create
 * returns ADAGC_E_INVALID_ARG beyond that, with ADAGC_CLIP_GLOBAL_ADAPTIVE, or on a device without cooperative
 * launch).  Only adagc_step takes the fused route; every other entry point of the context is unchanged.  The
 * barriers wait with a time limit; if one gives up, ADAGC_E_TIMEOUT is set in the status word and the context must
 * be created anew: once adagc_get_stats has read that bit, every later adagc_step of the context returns
 * ADAGC_E_POISONED and enqueues nothing (until then the steps still return ADAGC_OK, each waiting out its limit). */
#define ADAGC_FUSED_SMALL 32

/*
 * Optimizer state stored as bfloat16 (adagc_desc.state_dtype = ADAGC_BF16).  The paper trains in bfloat16 / float8
 * precision (Appendix "Hyper-Parameters") and does not say how stored optimizer state is rounded; this library's
 * reading: theta stays an fp32 master copy; d_m and d_v (d_m alone for Lion and momentum SGD) are bfloat16 arenas
 * with the descriptor's element offsets; a step reads the stored moments exactly, computes in fp32, updates theta
 * from the UNROUNDED new moments and rounds the moments to the nearest bfloat16, ties to even, where it stores them.
 * The update phase then moves 18 instead of 26 bytes per parameter (bf16 gradients).  Every entry point that takes
 * d_m / d_v follows the descriptor's state dtype.
 * Which bfloat16 neighbour is stored is a discrete decision, so its precision is part of the interface: the value that
 * is rounded is computed in single precision, each operation rounded once (fl), coefficients rounded to fp32 first:
 *     gh = fl(h g);   m' = fl(beta1 m + fl((1 - beta1) gh));   v' = fl(beta2 v + fl((1 - beta2) fl(gh gh)))       (AdamW)
 *     m' = fl(beta2 m + fl((1 - beta2) gh))                                                                        (Lion)
 *     m' = fl(momentum m + fl(wd theta + gh))                                                                      (SGD)
 * where each outer sum with its first product is one fused multiply-add.  (With bfloat16 g and m and beta1 = 0.9 the
 * exact value of m' lies precisely half-way between two bfloat16 values for about one element in twenty; a float64
 * evaluation resolves such ties by the rounding error of 0.9 itself.)  Note that with a decay close to 1 a stored bfloat16 moment stops
 * moving once (1 - beta)|target - x| drops below half its spacing, i.e. within spacing / (2 (1 - beta)) of the value
 * an fp32 moment would reach: 10 spacings (8 %) for beta2 = 0.95, 500 spacings for beta2 = 0.999.
 */

/* On AdaGC steps (step > warmup) the per-tensor decisions are taken in the tail of the norm kernel, so the step is two
 * launches.  With this flag they run as a kernel of their own, as on warm-up steps (three launches).  Results are
 * bit-identical either way.  (Contexts with ADAGC_ALLOW_EMPTY tensors of numel 0 always use the separate kernel.) */
#define ADAGC_SEPARATE_FINALIZE 64

/* One parameter tensor. */
typedef struct {
  int64_t numel;    /* > 0 (0 allowed with ADAGC_ALLOW_EMPTY); offset + numel <= 2^34 */
  int64_t offset;   /* element offset into every arena; offset * sizeof(element) must be a
                       multiple of 16 bytes for every arena dtype (multiple of 8 elements with
                       bf16 gradients, of 4 with fp32 gradients) */
  int32_t ndim;     /* 0..4; informational.  If > 0 the product of shape[0..ndim) must be numel */
  int32_t reserved; /* set to 0 */
  int64_t shape[4];
} adagc_tensor;

/* The model: a list of tensors plus the dtypes of the arenas. */
typedef struct {
  int32_t n_tensors;           /* 1 .. 2^24 */
  int32_t param_dtype;         /* ADAGC_F32 */
  int32_t grad_dtype;          /* ADAGC_F32 or ADAGC_BF16 */
  int32_t state_dtype;         /* dtype of the m and v arenas: ADAGC_F32, or ADAGC_BF16 (see "Optimizer state stored as
                                  bfloat16" below); every tensor offset must then be a multiple of 8 elements */
  const adagc_tensor* tensors; /* host array, copied by adagc_create */
  double lambda_abs;           /* warm-up global-norm threshold of Eq. 2, > 0 (paper: 1.0) */
  int32_t flags;               /* 0, or one ADAGC_UPDATE_PATH_* value, optionally OR-ed with the other ADAGC_* flags above */
  int32_t reserved;            /* set to 0 */
} adagc_desc;

/* Bytes of device workspace adagc_create needs for this descriptor (chunk table, per-chunk
 * partial sums, per-tensor statistics).  Returns 0 if the descriptor is invalid. */
size_t adagc_workspace_bytes(const adagc_desc* desc);

/* Number of fixed-size chunks the tensors are cut into (one partial sum per chunk).
 * Returns a negative adagc_status if the descriptor is invalid.  Host-only. */
int64_t adagc_num_chunks(const adagc_desc* desc);

/* Validate the descriptor, build the chunk table and upload it into `d_workspace`
 * (device memory, 256-byte aligned, at least adagc_workspace_bytes(desc) bytes, owned by the
 * caller and kept alive until adagc_destroy).  Synchronises `cuda_stream` once.
 * The CUDA device current at this call is the one the context is bound to: the step and clip entry
 * points return ADAGC_E_INVALID_ARG when another device is current.  A context is not
 * thread-safe: one caller at a time. */
int adagc_create(const adagc_desc* desc, void* d_workspace, size_t workspace_bytes,
                 void* cuda_stream, adagc_ctx** out);

/* Frees the host-side context (not the workspace). */
int adagc_destroy(adagc_ctx* ctx);

/*
 * One fused step of Algorithm 1.
 *   d_params           : fp32 arena, updated in place
 *   d_m, d_v           : arenas in the descriptor's state dtype (fp32 or bfloat16), updated in place
 *   d_grads            : gradient arena in the descriptor's grad dtype, read only
 *   d_ema              : gamma, n_tensors fp32 values, updated in place (Section 4.3 "Memory":
 *                        one 32-bit float per tensor)
 *   step               : t >= 1
 *   lr, beta1, beta2, eps, wd : eta_t, beta_1, beta_2, epsilon, lambda_w of Algorithm 1
 *   lambda_rel, beta   : relative threshold and EMA coefficient of Eq. 3
 *   warmup             : T_start >= 0
 * Domain: 0 <= beta < 1, 0 <= beta1, beta2 < 1, lambda_rel > 0, eps >= 0, lr and wd finite.
 * Arena pointers must be 16-byte aligned.
 */
int adagc_step(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v,
               float* d_ema, int64_t step, double lr, double beta1, double beta2, double eps,
               double wd, double lambda_rel, double beta, int64_t warmup, void* cuda_stream);

/*
 * adagc_step for CUDA graphs: the enqueued work is identical for every step, so a graph captured once can be
 * replayed for the whole run.  What adagc_step takes from its `step` argument is kept on the device instead:
 *   - t = (steps this context has executed so far) + 1, read from the context's device-side counter (the one
 *     adagc_get_stats reports as steps_done; every step-type entry point advances it).  The warm-up switch
 *     (t <= warmup), the seeding of gamma at t = 1 and the bias corrections 1 - beta^t follow from it on the
 *     device, in float64 as on the host.  After a restart set the counter with adagc_set_step_counter.
 *   - eta_t: if d_lr is not NULL it points to one fp32 value in DEVICE memory that is read at every execution
 *     (update it between replays to follow a schedule); if NULL the value `lr` is used.
 * The other arguments are those of adagc_step.  Five launches per step (prologue, norm, per-tensor
 * finalize, warm-up finalize -- which returns at once outside warm-up -- and update) instead of two.
 * Results agree with adagc_step's to the last bit whenever the device and host evaluations of beta^t round
 * to the same fp32 coefficients, and within the library's tolerance (1e-5) always.
 */
int adagc_step_capturable(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v,
                          float* d_ema, const float* d_lr, double lr, double beta1, double beta2, double eps,
                          double wd, double lambda_rel, double beta, int64_t warmup, void* cuda_stream);

/* Sets the device-side step counter (steps executed so far) -- for adagc_step_capturable after a restart from
 * saved state at step t0: pass t0 - 1.  Enqueues one tiny kernel. */
int adagc_set_step_counter(adagc_ctx* ctx, uint64_t steps_done, void* cuda_stream);

/*
 * adagc_step that also emits the model's working copy of the parameters: mixed-precision training keeps fp32
 * master parameters in the optimizer and runs the model on a bf16 copy (the paper's runs use bfloat16
 * precision).  Besides everything adagc_step does, d_params_bf16[j] = bf16(theta_t[j]) (round to nearest even)
 * is written for every element of every tensor, from the same kernel, so no separate cast pass re-reads theta.
 * d_params_bf16 is a bf16 arena with the descriptor's element offsets, 16-byte aligned; every tensor offset
 * must then be a multiple of 8 elements (ADAGC_E_MISALIGNED otherwise).  28 B/param instead of 26.
 */
int adagc_step_emit_bf16(adagc_ctx* ctx, void* d_params, void* d_params_bf16, const void* d_grads, void* d_m,
                         void* d_v, float* d_ema, int64_t step, double lr, double beta1, double beta2,
                         double eps, double wd, double lambda_rel, double beta, int64_t warmup,
                         void* cuda_stream);

/*
 * The same clip fused with Lion instead of AdamW (Section 4.2 of the paper: AdaGC is optimizer-agnostic
 * and is used with Lion).  Phases 1 and 2 are those of adagc_step; the update phase applies Lion's rule
 * to the clipped gradient hat(g) = h_i g:
 *     c = beta1 m + (1 - beta1) hat(g);   theta <- theta - lr (sign(c) + wd theta);
 *     m <- beta2 m + (1 - beta2) hat(g)
 * d_params and d_m are fp32 arenas updated in place (Lion keeps one state per parameter, there is no v).
 * Everything elementwise is fp32; where the two terms of c cancel to within fp32 rounding the sign is a
 * near-tie and may differ from a float64 evaluation.  Typical beta1 0.9, beta2 0.99.
 */
int adagc_step_lion(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, float* d_ema,
                    int64_t step, double lr, double beta1, double beta2, double wd, double lambda_rel,
                    double beta, int64_t warmup, void* cuda_stream);

/*
 * The same clip fused with SGD with momentum (heavy-ball form, L2 weight decay folded into the gradient):
 *     d = hat(g) + wd theta;   m <- momentum m + d;   theta <- theta - lr m          (m_0 = 0)
 * d_params and d_m are fp32 arenas updated in place; 0 <= momentum < 1.
 */
int adagc_step_sgdm(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, float* d_ema,
                    int64_t step, double lr, double momentum, double wd, double lambda_rel, double beta,
                    int64_t warmup, void* cuda_stream);

/*
 * Clip-only entry (Section 4.2: the clip is optimizer-agnostic): same norms, decisions and
 * gamma update as adagc_step, then writes the clipped gradient h_i * g_i in the gradient dtype.
 * d_grads_out may equal d_grads_in (in place); in place, tensors with h == 1 are not rewritten.
 */
int adagc_clip(adagc_ctx* ctx, const void* d_grads_in, void* d_grads_out, float* d_ema,
               int64_t step, double lambda_rel, double beta, int64_t warmup, void* cuda_stream);

/*
 * The step cut in two for models whose tensors are SHARDED over several GPUs (ZeRO-style flat shards,
 * tensor parallelism).  Section 4.3 ("Communication"): a tensor's norm then needs one all-reduce of the
 * partial sums of squares within the group that holds it; nothing else of the step crosses devices.
 * Every rank creates its context over its LOCAL slices of the tensors (adagc_shard_plan computes them for
 * flat equal shards; ADAGC_ALLOW_EMPTY lets a rank list tensors it holds nothing of) and runs, per step:
 *
 *   1. adagc_shard_sumsq        phase 1 on the local gradient slice; d_sumsq_out[i] = sum of squares of this
 *                               rank's part of tensor i, float64, n_tensors entries, device memory;
 *   2. the caller sums d_sumsq_out over the ranks (one all-reduce of 8 * n_tensors bytes, e.g. NCCL);
 *   3. adagc_step_presummed /   phase 2 from the summed vector `d_sumsq` (decisions, gamma, statistics:
 *      adagc_clip_presummed     identical on every rank, since every rank sees the same sums) and phase 3
 *                               on the local slices.
 *
 * gamma (d_ema, n_tensors floats) is replicated: every rank holds and updates the full vector.  The other
 * arguments are those of adagc_step / adagc_clip.  d_sumsq is read only and must not be the same buffer the
 * next adagc_shard_sumsq writes before this call's kernels have run (same stream: always fine).
 * With one rank the three calls compute exactly what adagc_step computes.
 */
int adagc_shard_sumsq(adagc_ctx* ctx, const void* d_grads, double* d_sumsq_out, void* cuda_stream);
int adagc_step_presummed(adagc_ctx* ctx, void* d_params, const void* d_grads, void* d_m, void* d_v,
                         float* d_ema, const double* d_sumsq, int64_t step, double lr, double beta1,
                         double beta2, double eps, double wd, double lambda_rel, double beta, int64_t warmup,
                         void* cuda_stream);
int adagc_clip_presummed(adagc_ctx* ctx, const void* d_grads_in, void* d_grads_out, float* d_ema,
                         const double* d_sumsq, int64_t step, double lambda_rel, double beta, int64_t warmup,
                         void* cuda_stream);

/*
 * Flat equal shards: the arena [0, arena_elems) of `full` (arena_elems = max offset + numel) is cut into
 * `world` consecutive ranges of shard_elems = ceil(arena_elems / world) rounded up to a multiple of 8
 * elements; rank r owns [r * shard_elems, min((r + 1) * shard_elems, arena_elems)).  Writes, for every
 * tensor i of `full`, this rank's slice into local[i] (n_tensors entries, host memory): numel = elements of
 * tensor i inside the range (possibly 0), offset = where the slice starts, counted from the start of the
 * range (so the rank's arenas are the sub-arrays of the full arenas that begin at *elem_begin), ndim = 0.
 * *elem_begin / *elem_end receive the range; a rank whose range would start at or beyond arena_elems holds
 * nothing and gets the empty range [0, 0); the three sharded entry points ignore the arena pointers of a
 * context that holds no element (they may be NULL).  Host-only, no CUDA call.  Returns ADAGC_E_INVALID_ARG for
 * world < 1 or rank outside [0, world), or the descriptor's own validation error.
 */
int adagc_shard_plan(const adagc_desc* full, int32_t rank, int32_t world, adagc_tensor* local,
                     int64_t* elem_begin, int64_t* elem_end);

/*
 * adagc_step fed from HOST memory: copies the gradient arena `h_grads` (arena_elems elements of the grad
 * dtype; pinned memory recommended) into `d_grads`, runs the step, copies the per-tensor statistics of this
 * step back into the host arrays (any may be NULL) and synchronises the stream.
 * On AdaGC steps (step > warmup) the work is pipelined: the tensors are taken in groups (arena order), the
 * copies run on a stream owned by the context, and each group goes through norm, finalize and update on
 * `cuda_stream` as soon as its gradients have arrived, so the kernels hide behind the host-to-device copy.
 * Results are identical to adagc_step's.  Warm-up steps need the global norm first and are not pipelined.
 */
int adagc_step_host(adagc_ctx* ctx, void* d_params, void* d_grads, void* d_m, void* d_v,
                    float* d_ema, const void* h_grads, int64_t step, double lr, double beta1,
                    double beta2, double eps, double wd, double lambda_rel, double beta,
                    int64_t warmup, float* h_norm, float* h_clipfactor, uint8_t* h_flag,
                    void* cuda_stream);

/*
 * Statistics of the most recent step, copied to host arrays of n_tensors entries (any pointer may
 * be NULL): gradient norm, clip factor h, clip flag, cumulative clip count; plus the number of
 * steps executed and the device status word.  Synchronises the stream.
 */
int adagc_get_stats(adagc_ctx* ctx, float* h_norm, float* h_clipfactor, uint8_t* h_flag,
                    uint64_t* h_clip_count, uint64_t* h_steps_done, int32_t* h_device_status,
                    void* cuda_stream);

/* Per-tensor sums of squares of the most recent step in float64 (n_tensors entries).
 * Synchronises the stream. */
int adagc_get_sumsq(adagc_ctx* ctx, double* h_sumsq, void* cuda_stream);

/*
 * "Thresholded initialization", variant 3 of the paper's EMA-initialization ablation (Section 5: gamma_t,i =
 * min(||g_t,i||, 0.1)).  With cap > 0, every place where the default seeds gamma (step 1) or takes the running
 * minimum (warm-up steps) sets gamma_t,i = min(||hat(g)_t,i||, cap) instead: the constant stands where
 * gamma_t-1,i stands in Algorithm 1's warm-up line, so after warm-up gamma is the last warm-up step's clipped
 * norm, capped.  With T_start = 0 the seed of step 1 is min(||g_1,i||, cap) and Eq. 3 applies to it at once.
 * AdaGC steps after the first are unchanged.  cap = 0 (the default) switches the variant off.  Host-only; takes
 * effect from the next step.  Returns ADAGC_E_INVALID_ARG for a negative or non-finite cap.
 */
int adagc_set_ema_cap(adagc_ctx* ctx, double cap);

/*
 * How bfloat16-stored moments (state_dtype = ADAGC_BF16) are rounded where they are stored.
 *   ADAGC_ROUND_NEAREST     to the nearest bfloat16, ties to even (the default);
 *   ADAGC_ROUND_STOCHASTIC  to the neighbour of larger magnitude with probability (distance to the smaller neighbour) /
 *                           spacing, otherwise to the smaller one: unbiased, so a slow average (beta2 = 0.999) keeps
 *                           moving where rounding to nearest stalls.  The single-precision value of "Optimizer state
 *                           stored as bfloat16" above has the 16-bit random integer r added to the low half of its bit
 *                           pattern, and that half is dropped.  r comes from the counter-based generator Philox4x32-10
 *                           (Salmon et al., SC 2011): the four elements 4q .. 4q+3 of the arenas share one call with
 *                           counter (lo q, hi q, lo step, hi step) and key (lo seed, hi seed); element 4q + l takes
 *                           output word l, its low half for m, its high half for v.  The result therefore depends on
 *                           (seed, step, element position) only: reruns and restarts reproduce it bit for bit.
 *                           In this mode (and only in it, and only for eps >= 1e-30) theta's increment
 *                           m_hat / (sqrt(v_hat) + eps) is taken with the approximate square root and reciprocal
 *                           (relative error of a few 1e-7, subnormal v_hat flushed to zero) instead of the correctly
 *                           rounded ones: the random numbers make the kernel instruction-bound otherwise, and the
 *                           moments already carry a random relative error of 2^-9.  The stored moments are unaffected.
 * Host-only; takes effect from the next step.  ADAGC_E_DTYPE if the context's state is fp32.  adagc_step_capturable
 * returns ADAGC_E_INVALID_ARG while stochastic rounding is on (its step number lives on the device).
 */
#define ADAGC_ROUND_NEAREST 0
#define ADAGC_ROUND_STOCHASTIC 1
int adagc_set_state_rounding(adagc_ctx* ctx, int32_t mode, uint64_t seed);

/* The update path this context uses: ADAGC_UPDATE_PATH_REGISTERS or ADAGC_UPDATE_PATH_BULK. */
int adagc_update_path(const adagc_ctx* ctx);

/* Thread blocks that this context launches for its norm / scale kernels (*norm_grid: eight per SM, fewer when the
 * layout has fewer chunks) and for its update kernel (*update_grid: one per SM on the bulk-async path, two on the
 * register path).  The kernels' memory behaviour was tuned for exactly these residencies (the paper has no counterpart;
 * the tests use this to notice a kernel whose register count no longer admits its grid).  Either pointer may be NULL.
 * Returns ADAGC_OK or ADAGC_E_INVALID_ARG (NULL context). */
int adagc_launch_grids(const adagc_ctx* ctx, int32_t* norm_grid, int32_t* update_grid);

/* Elements spanned by the arenas: max over tensors of offset + numel. */
int64_t adagc_arena_elems(const adagc_ctx* ctx);

/* Kernels launched by this context so far. */
uint64_t adagc_launch_count(const adagc_ctx* ctx);

/*
 * Optional per-phase timing.  When enabled, adagc_step / adagc_clip record CUDA events on the
 * caller's stream around the three phases (norm, finalize, update-or-scale).
 * adagc_get_phase_times synchronises on the last event and returns the durations in
 * milliseconds of the most recent step: ms[0] norm, ms[1] finalize, ms[2] update / scale.  (On AdaGC steps the
 * decisions are taken inside the norm kernel unless ADAGC_SEPARATE_FINALIZE is set: ms[0] then covers both and
 * ms[1] is the empty interval between two events.)
 */
int adagc_set_phase_timing(adagc_ctx* ctx, int enabled);
int adagc_get_phase_times(adagc_ctx* ctx, float ms[3]);

/*
 * Sum of squares (squared L2 norm) of one contiguous gradient buffer, for callers that cannot
 * allocate.  (The paper has no counterpart of this entry point: it is a convenience of this library.)
 *
 * Who needs it: code that must take a gradient norm at a point where it cannot get device memory --
 * it runs while the framework's allocator is locked or out of memory, it is a plug-in that is handed
 * only its input and output buffers, or its memory budget was fixed before start-up.  Everything else
 * in this header works on a caller-provided workspace; this call needs none.  Its per-chunk partial
 * sums live in a fixed 512 KiB array inside the library's device image, so every GPU that loads the
 * library holds those 512 KiB until the process exits.
 *
 *   d_grads      device buffer of `numel` elements of `grad_dtype` (ADAGC_F32 or ADAGC_BF16),
 *                16-byte aligned, read only
 *   numel        1 .. 2^30 (1 073 741 824) elements; more returns ADAGC_E_TOO_LARGE and enqueues nothing
 *   d_sumsq_out  device pointer to one double (8-byte aligned), overwritten with sum_j g_j^2 in
 *                float64; same chunking and summation order as the norm phase of adagc_step
 *
 * The call enqueues two kernels on `cuda_stream`, does not synchronise, and calls no allocating
 * routine.  The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call outside any stream capture.
 * That lookup is safe against several host threads making their first call at once (one does it, the
 * others wait).  Device ordinals 0..63 are supported; on a higher ordinal, or if the lookup fails, the
 * call returns ADAGC_E_CUDA and enqueues nothing.  If a launch itself fails the return value is
 * ADAGC_E_CUDA as well, and the first kernel may already be enqueued.
 * All calls share the one array and it keeps the previous call's contents; every entry a call reads
 * it has first rewritten, so nothing needs clearing, but two calls whose kernels overlap on the GPU
 * (different streams, or several host threads) race on it: serialise them on one stream or with events.
 */
int adagc_sumsq_noalloc(const void* d_grads, int32_t grad_dtype, int64_t numel, double* d_sumsq_out,
                        void* cuda_stream);

/*
 * Test aid for the bounded device-side waits (the bulk-async update kernel waits on shared-memory
 * barriers; every such wait gives up after a time limit instead of spinning forever).  Launches one
 * small block that waits, with the same routine, on a barrier that nothing ever signals; after
 * `limit_ms` (0 < limit_ms <= 1000) it gives up, sets ADAGC_E_TIMEOUT in the device status word and
 * returns normally, leaving the context usable.  Enqueues only.
 */
int adagc_debug_wait_timeout(adagc_ctx* ctx, double limit_ms, void* cuda_stream);

/*
 * Debugging aids for the chunk tables (host-only, no CUDA call).  adagc_create cuts every tensor into chunks of 16384
 * elements (the last one shorter; one partial sum per chunk) and hands the chunks to thread blocks through three
 * tables; adagc_debug_chunk_tables rebuilds one of them for `grid` blocks:
 *   which = 0  original order, block b owns the consecutive entries [block_begin[b], block_begin[b+1]) (norm kernel
 *              with the decisions in its tail);
 *   which = 1  balanced over the blocks of the norm / scale grid, a block's entries contiguous;
 *   which = 2  balanced over the blocks of the update grid; a block's full chunks come first:
 *              [block_begin[b], block_mid[b]) are full, [block_mid[b], block_begin[b+1]) partial.
 * Output arrays (host memory): adagc_num_chunks(desc) entries each of h_start (element offset into the arenas),
 * h_count, h_tensor, h_partial; grid + 1 entries of h_block_begin; grid entries of h_block_mid (which = 2 only).
 * adagc_debug_chunk_entry_ok is the predicate a library built with -DADAGC_BOUNDS_CHECK applies, on the device, to
 * every table entry a block is about to walk (such a build sets ADAGC_E_BOUNDS in the status word and skips the block
 * instead of accessing memory); adagc_debug_bounds_checked_build tells whether this library is such a build.
 */
int adagc_debug_chunk_tables(const adagc_desc* desc, int32_t which, int32_t grid, int64_t* h_start, int32_t* h_count,
                             int32_t* h_tensor, int32_t* h_partial, int32_t* h_block_begin, int32_t* h_block_mid);
int adagc_debug_chunk_entry_ok(int64_t start, int32_t count, int32_t tensor, int32_t partial, int64_t arena_elems,
                               int32_t n_chunks, int32_t n_tensors);
int adagc_debug_bounds_checked_build(void);

/* Test aid: feeds `device_status` to the same host-side latch that adagc_get_stats applies to the status word it reads
 * (a context created with ADAGC_FUSED_SMALL refuses further steps once ADAGC_E_TIMEOUT has been seen).  Host-only. */
int adagc_debug_latch_status(adagc_ctx* ctx, int32_t device_status);

/* Static string for a status code. */
const char* adagc_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ADAGC_H_ */
