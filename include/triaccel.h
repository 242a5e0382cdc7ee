/*
 * triaccel.h -- C ABI of the Tri-Accel fused optimizer pass for NVIDIA B200 (sm_100a).
 *
 * One call of ta_step() runs, over every parameter tensor ("layer", a segment of one flat
 * buffer), the per-step control-and-update pass of Tri-Accel (arXiv 2508.16905):
 *   - per-layer gradient mean / variance and their exponential moving averages (Sec. 3.1),
 *   - the sparse second-order signal: a Hutchinson diagonal estimate z*(Hz) from Rademacher
 *     probes with a per-layer top-k magnitude mask (Abstract, Sec. 1, Sec. 3.2),
 *   - the per-layer precision code FP16/BF16/FP32 from the variance EMA, with curvature
 *     promotion, and the curvature-scaled step size (Sec. 3.1, Sec. 3.2, Sec. 3.4),
 *   - the FP32 master-weight update fused with the cast into the layer's 16-bit copy
 *     (Sec. 2 master-copy principle, Sec. 3.2 step size, Sec. 4.1 SGD).
 * ta_batch_next() is the host-only memory-elastic batch rule (Sec. 3.3).
 *
 * Conventions
 *   - Every function returns an int: TA_OK or a negative TA_ERR_* code.  Nothing throws.
 *     ta_last_error() gives a static, human-readable string for the last failure of a handle.
 *   - "device" pointers are CUDA device pointers of the handle's device; "host" pointers are
 *     ordinary host memory.  The caller owns every buffer it passes.  The library owns the
 *     handle, its per-layer state, its workspace and the mask bits; ta_destroy() frees them.
 *   - All device work is enqueued on the stream passed in (a cudaStream_t cast to void*, NULL =
 *     the default stream) and is asynchronous.  Only ta_stats(), ta_precision_codes(),
 *     ta_step_host() and the state save/load calls wait for it.
 *   - One handle belongs to one device (the device current at ta_create) and is not thread-safe.
 *   - There is no CPU fallback: without a usable CUDA device ta_create fails with TA_ERR_CUDA.
 *   - Flat-buffer layout: element i of layer l lives at flat index offset_l + i.  All flat
 *     buffers (w, g, c, each probe of Hz, z_out) have n_total elements and use the same index.
 *     Elements outside every segment ("gaps") are never used or written (a 16-byte vector that straddles the
 *     edge of a segment may be fetched whole; the elements outside are masked out).
 */
#ifndef TRIACCEL_H
#define TRIACCEL_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TA_OK          0
#define TA_ERR_ARG    (-1)   /* NULL / out-of-range argument, invalid table or hyper-parameter      */
#define TA_ERR_ALIGN  (-2)   /* a device pointer is not 16-byte aligned                             */
#define TA_ERR_STATE  (-3)   /* call order: step did not increase, handle destroyed, size mismatch  */
#define TA_ERR_CUDA   (-4)   /* a CUDA runtime call failed; ta_last_error() names it                */
#define TA_ERR_NOMEM  (-5)   /* host or device allocation failed                                    */

/* precision codes, in the order of the paper's case table (Sec. 3.1) */
#define TA_CODE_FP16 0
#define TA_CODE_BF16 1
#define TA_CODE_FP32 2

/* gradient element types */
#define TA_GRAD_F32  0
#define TA_GRAD_BF16 1

#define TA_MAX_PROBES 8

typedef struct ta_handle ta_handle;

/* One layer: [offset, offset + length) in elements of the flat buffer. */
typedef struct {
    uint64_t offset;
    uint64_t length;
} ta_segment;

/*
 * Hyper-parameters.  struct_size must be sizeof(ta_hparams) of the header the caller compiled
 * against (ABI growth).  Symbols follow the paper.
 */
typedef struct {
    uint32_t struct_size;
    float beta;          /* EMA smoothing, [0,1)                         Sec. 3.1 */
    float tau_low;       /* v_l <  tau_low            -> FP16            Sec. 3.1 */
    float tau_high;      /* v_l >= tau_high           -> FP32            Sec. 3.1 */
    float tau_curv;      /* lambda_l > tau_curv  -> one level up         Sec. 3.2 */
    float alpha;         /* eta_l = eta0 / (1 + alpha * lambda_l)        Sec. 3.2 */
    float eta0;          /* base learning rate (see ta_set_lr)           Sec. 3.2 */
    uint32_t topk_ppm;   /* mask keeps ceil(n_l * ppm / 1e6) (>= 1) largest |S|; 1000000 = dense */
    uint32_t num_probes; /* P, one of 1, 2, 4, 8 */
    uint32_t t_ctrl;     /* decisions are taken at steps with step % t_ctrl == 0   Sec. 3.4 */
    uint32_t grad_dtype; /* TA_GRAD_F32 or TA_GRAD_BF16 */
    float momentum;      /* SGD momentum mu in [0,1); 0 = plain SGD               Sec. 4.1 */
    float weight_decay;  /* L2 coefficient wd >= 0 added to the gradient; 0 = none       */
    uint32_t flags;      /* 0 or TA_FLAG_* bits */
} ta_hparams;

/*
 * TA_FLAG_INPUTS_FINITE -- the caller vouches that g and Hz hold no inf / NaN inside the segments (a mixed-precision
 * loop knows this from its own overflow check when it unscales the gradients).  Without the flag, one non-finite value
 * anywhere makes the whole step change nothing, so no layer can be updated before every layer has been read once, and
 * the gradient is read from memory twice.  With the flag the pass no longer holds the update back:
 *   - at a step with decisions (step % t_ctrl == 0) every layer is updated as soon as its own statistics are complete
 *     (Sec. 3.1, 3.2: all decisions are per layer), while its gradient is still in the L2 cache;
 *   - at a step without decisions (Sec. 3.4) the step size and the code of every layer are known beforehand, and the
 *     statistics, the update and the cast run as a single pass that reads every input once.
 * On finite inputs the results are those of the default pass.  Non-finite values are still counted
 * (ta_step_status.nonfinite_count) but no longer stop the step: skipped stays 0 and the layers that held them carry
 * non-finite statistics and weights.  Used by large dense models (no top-k mask, no momentum, beyond the size of the
 * one-launch path); other handles accept the flag and run the default pass.
 */
#define TA_FLAG_INPUTS_FINITE 1u
/*
 * TA_FLAG_NO_ONE_LAUNCH -- small dense models normally run the whole pass as one cooperative launch; with this flag
 * the handle uses the kernels of large models instead (separate sweep / decide / update launches, or the pipelined
 * launch together with TA_FLAG_INPUTS_FINITE).  Results are the same; meant for diagnostics and for exercising those
 * kernels on small tables.
 */
#define TA_FLAG_NO_ONE_LAUNCH 2u
/*
 * TA_FLAG_GUARD_WORKSPACES -- a test aid: every device buffer that ta_create allocates for the handle (plans, per-item
 * and per-layer sums, candidate lists, masks, counters) gets 256 guard bytes on either side, and
 * ta_test_check_guards() tells whether any kernel of the pass has written there (TA_ERR_STATE, with the buffer's
 * number in ta_last_error).  Results and speed of the pass are unchanged.
 */
#define TA_FLAG_GUARD_WORKSPACES 4u
/*
 * TA_FLAG_COOPERATIVE_LAUNCH -- small dense models run the pass as two dependent launches over one plan (statistics;
 * decisions and update), the second waiting for the first in hardware and the first launch of the next step free to
 * start beside the second of this one.  With this flag they run as ONE cooperative launch around a grid-wide barrier
 * instead, which keeps weights and gradients in shared memory between the two halves (models whose tensors fit).
 * Same results.
 */
#define TA_FLAG_COOPERATIVE_LAUNCH 8u

/* Per-layer statistics as of the last ta_step (host side, filled by ta_stats). */
typedef struct {
    float grad_mean;        /* mean of this step's gradient over the layer                      */
    float grad_var;         /* population variance of this step's gradient over the layer       */
    float ema_mean;         /* m_l                                                               */
    float ema_var;          /* v_l                                                               */
    float lambda_max;       /* max_i |S_i| / P, the curvature summary lambda_l                   */
    float topk_threshold;   /* k-th largest |S_i| of the layer (S is the probe SUM, not the mean) */
    float topk_mass;        /* sum of masked |S| / sum of all |S| (diagnostic)                   */
    float eta_scale;        /* s_l = 1 / (1 + alpha * lambda_l), as of the last control step     */
    uint64_t k;             /* mask population k_l                                               */
    uint32_t code;          /* TA_CODE_*                                                         */
    uint32_t near_threshold;/* 1 when v_l or lambda_l was within 1e-5 relative of a threshold at the last decision */
} ta_layer_stats;

typedef struct {
    uint64_t step;                 /* step of the last ta_step                                  */
    uint64_t nonfinite_count;      /* non-finite values seen in g and Hz at that step           */
    uint32_t skipped;              /* 1: that step changed nothing because of non-finite input  */
    uint32_t near_threshold_count; /* layers flagged near_threshold at the last decision        */
} ta_step_status;

/*
 * ta_create -- validates the segment table and hyper-parameters, plans the sweep and allocates
 * the library-owned device state on the current device.
 *   table    host, L entries, ascending and non-overlapping, every length in [1, 2^32 - 2];
 *            gaps between segments are allowed.  Offsets that are multiples of 4 elements give
 *            fully vectorised access; any offset is handled correctly.
 *   n_total  elements of every flat buffer; >= last offset + length; a multiple of 4.
 *   hp       host; see ta_hparams.
 *   out      receives the handle.
 * Initial state (Sec. 3.1): m_l = v_l = 0, lambda_l = 0, s_l = 1, code BF16 (the default mode),
 * mask empty.  Errors: TA_ERR_ARG, TA_ERR_NOMEM, TA_ERR_CUDA; *out is NULL on error.
 */
int ta_create(const ta_segment *table, uint32_t L, uint64_t n_total, const ta_hparams *hp, ta_handle **out);

/* Frees the handle and everything it owns.  NULL is allowed. */
int ta_destroy(ta_handle *h);

/*
 * ta_step -- one optimizer pass (asynchronous).
 *   w      device float[n_total], FP32 master weights, updated in place:
 *          w_i <- fl32(w_i - eta_l * b_i), eta_l = fl32(eta0 * s_l)                  (Sec. 3.2, 4.1)
 *          with b_i = g_i for plain SGD; with weight decay d_i = fl32(g_i + wd * w_i); with momentum
 *          b_i <- fl32(mu * b_i + d_i) in a library-owned buffer that starts at zero (no dampening,
 *          no Nesterov step: the rule of the paper's SGD baselines)
 *   g      device, float[n_total] or bfloat16[n_total] per hp.grad_dtype; read only
 *   Hz     device float[P][n_total] (probe p at Hz + p * n_total), the caller's products
 *          H z^(p) with z^(p) = the probe ta_probe() writes for (probe_seed, step, p); or NULL,
 *          in which case lambda_l, the threshold and the mask of the last step with Hz are kept
 *          (Sec. 3.2: curvature only every T iterations)
 *   c      device uint16[n_total], the 16-bit working copy: for layers coded FP16 / BF16 the
 *          round-to-nearest-even cast of the new w (IEEE binary16 with subnormals and overflow to
 *          inf / bfloat16); layers coded FP32 are left untouched                       (Sec. 2)
 *   probe_seed, step   key the Rademacher generator; step must be larger than at the previous
 *          call and below 2^32; decisions are taken when step % t_ctrl == 0, held otherwise.
 * If any gradient or Hz value inside a segment is not finite, the whole step changes nothing
 * (weights, copies, per-layer state) and ta_stats reports skipped = 1.
 * Errors: TA_ERR_ARG (NULL w/g/c), TA_ERR_ALIGN (a pointer not 16-byte aligned), TA_ERR_STATE
 * (step not increasing), TA_ERR_CUDA.  On error nothing is enqueued.
 */
int ta_step(ta_handle *h, float *w, const void *g, const float *Hz, uint16_t *c,
            uint64_t probe_seed, uint64_t step, void *stream);

/*
 * ta_step_host -- the same pass for callers whose tensors live in HOST memory (ideally pinned).
 * Copies w, g and Hz to library-owned device staging buffers (allocated at the first call, kept
 * until ta_destroy), runs ta_step, waits, then copies back the new w of every layer and the new c
 * of the layers coded FP16 / BF16 (c_host of FP32-coded layers and of gaps is left untouched; a
 * skipped step copies nothing back).  Returns after the stream has drained.
 * Arguments as for ta_step, but all four buffers are host pointers.  Errors as ta_step, plus
 * TA_ERR_NOMEM when the staging buffers cannot be allocated.
 */
int ta_step_host(ta_handle *h, float *w_host, const void *g_host, const float *Hz_host, uint16_t *c_host,
                 uint64_t probe_seed, uint64_t step, void *stream);

/* Sets eta0 for the following steps; the caller owns warm-up and decay schedules (Sec. 4.3). */
int ta_set_lr(ta_handle *h, float eta0);

/*
 * ta_probe -- writes the Rademacher probe z^(p) of (probe_seed, step), +1.0f / -1.0f, for all
 * n_total flat elements to z_out (device float[n_total], 16-byte aligned).  These are the signs
 * the sweep regenerates in registers.  The generator is Philox-4x32 with 10 rounds (Salmon et al.,
 * SC'11): for flat element i, with block = i / 4096, r = i % 4096, row = r / 128,
 * slot = (r / 4) % 32, comp = r % 4, the sign bit is bit (4*row + comp) of the 128-bit output of
 * Philox(counter = (q_lo, q_hi, step, p), key = (seed_lo, seed_hi)), q = 32*block + slot;
 * z = +1 for a 0 bit, -1 for a 1 bit.  p < num_probes.
 */
int ta_probe(ta_handle *h, uint64_t probe_seed, uint64_t step, uint32_t p, float *z_out, void *stream);

/*
 * ta_stats -- waits for the stream of the last ta_step, then fills out_host[L] and *status
 * (either may be NULL).  Step (1) of the control loop of Sec. 3.4.
 */
int ta_stats(ta_handle *h, ta_layer_stats *out_host, ta_step_status *status);

/* ta_precision_codes -- waits like ta_stats, then writes the L current codes (TA_CODE_*). Sec. 3.1 */
int ta_precision_codes(ta_handle *h, uint8_t *out_host);

/*
 * ta_masks -- the top-k mask of the last step with Hz: bit (i & 31) of word i >> 5 is set when
 * flat element i is among the k_l largest |S| of its layer (ties: lower index first); bits of
 * gaps are 0.  *dev_bits is library-owned device memory, valid until the next ta_step with Hz or
 * ta_destroy; read it on the stream used for ta_step.  The library keeps two mask buffers that swap roles
 * whenever a step with Hz commits, so call ta_masks again after such a step; the call waits for the stream of
 * the last ta_step.  With topk_ppm == 1000000 every element is in the mask, nothing is stored, and
 * *dev_bits = NULL, *num_words = 0.
 */
int ta_masks(ta_handle *h, const uint32_t **dev_bits, uint64_t *num_words);

/*
 * ta_power_iterate -- one step of the per-layer power iteration of Sec. 3.2,
 *     u <- H_l u / ||H_l u||,   lambda ~ (u^T H_l u) / (u^T u),
 * for all layers at once, on the same flat layout.  The caller supplies the products Hu (per layer, the
 * block H_l applied to u_l; e.g. from autograd).  To find the top-k eigenvalues one after the other (the
 * paper uses k = 5), eigenvectors already found are deflated:  Hu' = Hu - sum_j lambda_j (v_j . u) v_j.
 *   u, Hu      device float[n_total]
 *   V          device float[m][n_total], unit eigenvectors found so far (NULL when m = 0)
 *   lambda_V   device float[m][L], their eigenvalues per layer (NULL when m = 0)
 *   m          number of deflated vectors, <= TA_MAX_EIGS
 *   u_next     device float[n_total] (output; may be u itself): Hu' / ||Hu'|| per layer, 0 where ||Hu'|| = 0
 *   lambda_out device float[L] (output): Rayleigh quotient u . Hu' / u . u per layer (0 where u = 0)
 *   norm_out   device float[L] (output) or NULL: ||Hu'|| per layer
 * Sums are double, combined in a fixed order (bit-reproducible).  Asynchronous on `stream`.
 * Errors: TA_ERR_ARG, TA_ERR_ALIGN, TA_ERR_NOMEM (workspace, allocated at the first call), TA_ERR_CUDA.
 */
#define TA_MAX_EIGS 8
int ta_power_iterate(ta_handle *h, const float *u, const float *Hu, const float *V, const float *lambda_V, uint32_t m,
                     float *u_next, float *lambda_out, float *norm_out, void *stream);

/*
 * ta_set_curvature -- sets lambda_l of every layer from host values (e.g. the largest of the top-k
 * eigenvalues found by ta_power_iterate: max_{i<=k} lambda_i(H_l), Sec. 3.2).  The following ta_step calls
 * with Hz = NULL use them for the step size and the precision promotion.  Waits for the stream.
 * Errors: TA_ERR_ARG (NULL, negative or non-finite value), TA_ERR_CUDA.
 */
int ta_set_curvature(ta_handle *h, const float *lambda_max_host);

/*
 * A model spread over several GPUs by flat ranges (the paper leaves multi-GPU training as future work, Sec. 4.5; this
 * is the optimizer pass's side of it).  Rank r holds the elements [range_lo, range_hi) of every flat buffer, which may
 * cut layers anywhere on a multiple of 128 elements.  All decisions of the pass are per layer and need only the
 * layer's sums (Sec. 3.1: mean and variance; Sec. 3.2: the largest |S|), so one small exchange per step is enough:
 *
 *   ta_shard_sweep   statistics of the local part of every layer, one ta_layer_record per layer (device memory)
 *   (the caller gathers the records of all ranks, in rank order: world * L records; e.g. an NCCL all-gather)
 *   ta_shard_apply   combines the records in rank order (every rank arrives at identical numbers), takes the
 *                    decisions, screens the step (a non-finite value on any rank skips the step on every rank) and
 *                    updates the local weights and copies
 *
 * ta_create_shard takes the table and n_total of the WHOLE model plus this rank's range; the buffers passed to the two
 * calls hold only the range (element i of the model at index i - range_lo; Hz_local is [P][range_hi - range_lo]).
 * The probes are those of the whole model (they depend on the flat index, not on the cut).  Results equal those of
 * one handle over the whole model: codes, step sizes, weights and copies bit for bit, the double-precision moments up
 * to the order of summation.  Dense curvature only (topk_ppm == 1000000), no momentum buffer; ta_stats, ta_set_lr,
 * ta_precision_codes and the state calls work as usual (every rank holds the state of all layers); ta_step returns
 * TA_ERR_STATE on such a handle.
 */
typedef struct ta_layer_record {
    double s1, s2;        /* sums of (g - pivot) and (g - pivot)^2 over the local elements of the layer */
    double n;             /* their number (0: the layer has no element on this rank)                     */
    float pivot;          /* the first local gradient value of the layer                                 */
    uint32_t amax, amin;  /* largest / smallest |S| (bit patterns)                                       */
    uint32_t bad;         /* non-finite inputs                                                           */
} ta_layer_record;
int ta_create_shard(const ta_segment *table, uint32_t L, uint64_t n_total, const ta_hparams *hp, uint64_t range_lo,
                    uint64_t range_hi, ta_handle **out);
int ta_shard_sweep(ta_handle *h, const void *g_local, const float *Hz_local, uint64_t probe_seed, uint64_t step,
                   ta_layer_record *records_out /* device, L records */, void *stream);
int ta_shard_apply(ta_handle *h, float *w_local, const void *g_local, uint16_t *c_local,
                   const ta_layer_record *records_all /* device, world * L records, rank-major */, uint32_t world, void *stream);

/* How this handle runs the pass, in words (static string): "separate kernels", "two dependent launches", ... */
const char *ta_path(const ta_handle *h);

/* Number of kernels the library launched on behalf of this handle so far (for benchmarks). */
int ta_launch_count(ta_handle *h, uint64_t *count);

/*
 * Per-phase device timing (a measurement aid).  After ta_timing_begin(h, n) the next n calls of
 * ta_step record CUDA events on their stream before the sweep, after it, after the decisions
 * (including the top-k selection) and after the update.  ta_timing_end waits for the stream and
 * returns the summed milliseconds of the three phases and the number of steps they cover.
 */
int ta_timing_begin(ta_handle *h, uint32_t max_steps);
int ta_timing_end(ta_handle *h, double *ms_sweep, double *ms_decide, double *ms_update, uint32_t *steps);

/*
 * Failure detection.  With TA_FLAG_COOPERATIVE_LAUNCH small dense models run as one cooperative launch whose blocks
 * meet at a grid-wide barrier.  Every such wait is bounded (a few hundred milliseconds): a block that gives up
 * records it and returns, the step then changes neither weights, copies nor per-layer state, and the
 * next ta_stats / ta_precision_codes returns TA_ERR_CUDA once ("a bounded device-side wait ran out"),
 * after which the handle is usable again.  ta_test_expire_next_wait is a test aid: it makes the waits of
 * the next ta_step of this handle expect arrivals that never come, so that the path above can be
 * exercised without hanging or faulting the GPU.  TA_ERR_STATE if the handle does not use that path.
 */
int ta_test_expire_next_wait(ta_handle *h);
/* Waits for the stream, then checks the guard bytes around the handle's workspaces (see TA_FLAG_GUARD_WORKSPACES). */
int ta_test_check_guards(ta_handle *h);

/*
 * The work plan of the one-launch path, for inspection (host only, no GPU needed).  Small dense models
 * run the whole pass of Sec. 3.1 - 3.2 in one launch; its plan cuts every layer into "runs" (contiguous
 * pieces, cut on the grid of 128-element rows of the flat buffer, so that only the first and last row
 * of a layer can be partial) and gives each of at most `warps` warps a list of consecutive runs of
 * about equal cost (elements plus a constant per run), which is what keeps a table of thousands of
 * tiny tensors beside a few large ones from starving warps.  Writes the runs in buffer order to
 * out[0 .. *n_runs) (at most cap; TA_ERR_ARG if there are more), the number of warps that got work to
 * *warps_used and the largest number of rows one warp walks to *max_rows.  ta_create builds the same
 * plan with warps = resident warps of the device.  Table rules as for ta_create.
 */
typedef struct ta_run {
    uint64_t begin;      /* first element */
    uint32_t length;     /* elements, all inside one layer */
    uint32_t layer;
    uint32_t warp;       /* the warp of the grid that handles the run */
    uint32_t reserved;
} ta_run;
int ta_plan_one_launch(const ta_segment *table, uint32_t L, uint32_t warps, ta_run *out, uint32_t cap,
                       uint32_t *n_runs, uint32_t *warps_used, uint32_t *max_rows);

/*
 * The work items of the multi-kernel pass (models too large for the one-launch path, top-k masks, momentum), for
 * inspection (host only, no GPU needed).  Every layer is cut on a global grid of *item_elems elements (512 ... 16384,
 * chosen from the parameter count so that every warp slot of a GPU with sm_count SMs gets several items); one warp
 * handles one item, eight consecutive items make the batch of one block.  topk != 0: a layer of at least eight items
 * starts on a batch boundary (empty padding items, length 0, before it), so that its batches hold one layer only and
 * count the histogram of Sec. 3.2's selection in shared memory.  Writes the items in buffer order to
 * out[0 .. *n_items) (at most cap; TA_ERR_ARG if there are more): `warp` is the item's place in its batch, `reserved`
 * is 1 when all items of that batch lie in one layer.  ta_create builds the same plan with the device's SM count.
 * Table rules as for ta_create.
 */
int ta_plan_items(const ta_segment *table, uint32_t L, uint32_t sm_count, uint32_t topk, ta_run *out, uint64_t cap,
                  uint64_t *n_items, uint32_t *item_elems);

/*
 * The task queues of the pipelined pass (TA_FLAG_INPUTS_FINITE on a large dense model), for inspection (host only,
 * no GPU needed).  Every task covers one batch: up to 14336 consecutive elements of one layer.  With
 * with_decisions != 0, the two queues of a step that takes decisions (Sec. 3.4), one after the other: the sweep tasks
 * (TA_TASK_SWEEP, statistics) in buffer order, then the update tasks (TA_TASK_APPLY) layer by layer, within a layer
 * the last batch first.  Blocks draw from both queues; an update task is handed out once its layer is decided, and
 * until then the block goes on sweeping.  Otherwise the queue of a step between decisions, one single-pass task
 * (TA_TASK_BOTH) per batch.  Writes at most cap tasks; *n_tasks is their number (TA_ERR_ARG if cap is smaller).
 * Table rules as for ta_create.
 */
#define TA_TASK_SWEEP 0u
#define TA_TASK_APPLY 1u
#define TA_TASK_BOTH  2u
typedef struct ta_task {
    uint64_t begin;      /* first element of the batch */
    uint32_t length;     /* elements, all inside one layer */
    uint32_t layer;
    uint32_t kind;       /* TA_TASK_* */
    uint32_t reserved;
} ta_task;
int ta_plan_pipeline(const ta_segment *table, uint32_t L, uint32_t with_decisions, ta_task *out, uint64_t cap, uint64_t *n_tasks);

/* Static description of the last error of this handle ("" if none).  h may be NULL: then the
 * last ta_create failure of the calling thread. */
const char *ta_last_error(const ta_handle *h);

/*
 * Per-layer state checkpoint: EMAs, lambda, threshold, codes, step scale, mask bits, last step.
 * ta_state_size gives the byte count; ta_state_save writes it to a host buffer (waits for the
 * stream); ta_state_load restores it into a handle created with the same table and
 * hyper-parameters (TA_ERR_STATE otherwise).  The next step after a load is bit-identical to
 * the one the saved handle would have taken.
 */
int ta_state_size(ta_handle *h, uint64_t *bytes);
int ta_state_save(ta_handle *h, void *buf_host, uint64_t bytes);
int ta_state_load(ta_handle *h, const void *buf_host, uint64_t bytes);

/*
 * Memory-elastic batch rule (Sec. 3.3), host only:
 *   B <- B + delta_up    if MemUsage <  rho_low  * MemMax
 *   B <- B - delta_down  if MemUsage >  rho_high * MemMax
 *   B unchanged otherwise; the result is clamped to [B_min, B_max] and stored back in bc->B.
 * mem_reader(user, &free_bytes, &total_bytes) returns 0 on success; NULL selects cudaMemGetInfo
 * of the current device.  MemUsage = total - free; MemMax = mem_budget_bytes if non-zero, else
 * total.  Errors: TA_ERR_ARG (NULL, rho_low > rho_high, B_min > B_max, negative deltas),
 * TA_ERR_CUDA (the reader failed; B is left unchanged).
 */
typedef int (*ta_mem_reader)(void *user, uint64_t *free_bytes, uint64_t *total_bytes);

typedef struct {
    int64_t B;
    int64_t delta_up, delta_down;
    int64_t B_min, B_max;
    double rho_low, rho_high;
    uint64_t mem_budget_bytes;
    ta_mem_reader mem_reader;
    void *user;
} ta_batch_ctrl;

int ta_batch_next(ta_batch_ctrl *bc, int64_t *B_next);

/*
 * ta_grad_moments_static -- per-layer gradient mean and population variance, computed without
 * allocating anything.  (The paper has no counterpart: this entry point exists for the callers
 * described next, not for a step of the method.)
 *
 * Who it is for: code that is not allowed to call cudaMalloc at the point where it needs the
 * statistics -- a plug-in running inside a host application that owns all device memory and has
 * handed out every byte of it, a callback that runs while an allocator lock is held, a process
 * whose memory pool was sized up front and must not grow.  ta_create / ta_step allocate their
 * workspace with cudaMalloc; this call never calls cudaMalloc, cudaFree or any allocating routine.
 *
 * How: the scratch (per tile of TA_STATIC_TILE_ELEMS gradient elements: two partial sums, the tile's
 * pivot value and a non-finite count) lives in a fixed array inside the library's device image, about
 * 770 KB.  A GPU holds it from the moment the CUDA runtime loads this library's device code there until
 * the process exits.  The layer table travels as a kernel argument.
 *
 * The first call on each device is a warm-up: with the CUDA runtime's default lazy loading it is that
 * call which loads the device code (kernels and the array) onto the device, which takes device memory
 * once and can fail when none is left, and it looks up the array's device address (cudaGetSymbolAddress,
 * with that device current).  Make it at start-up, while memory is still free, outside any stream
 * capture and outside allocator locks (or run with CUDA_MODULE_LOADING=EAGER, which moves the loading
 * to context creation).  Every later call on that device allocates nothing at all: free device memory
 * is the same before and after it.
 *
 *   table      host, L <= TA_STATIC_MAX_LAYERS segments, same rules as ta_create
 *   g          device, float or bfloat16 per grad_dtype, 16-byte aligned, indexed by flat element
 *   mean_var   device double[2 * L] (output): mean of layer l at [2l], variance at [2l + 1]
 *   nonfinite  device uint32[L] (output, 4-byte aligned) or NULL: non-finite gradient values per layer
 *   stream     cudaStream_t as void*; the call is asynchronous
 *
 * Limits: the layers must fit in TA_STATIC_MAX_TILES tiles (tiles are cut on a global grid of
 * TA_STATIC_TILE_ELEMS elements, so a layer of n elements needs about n / TA_STATIC_TILE_ELEMS + 1);
 * that is roughly 536 million parameters.  A larger table is rejected with TA_ERR_ARG and a message
 * (ta_static_last_error) and nothing is launched.
 * All calls on one device share the one array and it keeps the previous call's contents.  Every
 * slot a call reads is written earlier in the same call, so nothing needs clearing; but two calls
 * whose kernels overlap on the GPU (different streams, no ordering between them) race on it and
 * give wrong results.  Order them on one stream or with events.
 * Results equal ta_stats().grad_mean / grad_var of a ta_step on the same gradient up to rounding
 * (both accumulate in double).  Errors: TA_ERR_ARG, TA_ERR_ALIGN, TA_ERR_CUDA.
 */
#define TA_STATIC_TILE_ELEMS 16384u
#define TA_STATIC_MAX_TILES  32768u
#define TA_STATIC_MAX_LAYERS 128u
int ta_grad_moments_static(const ta_segment *table, uint32_t L, const void *g, uint32_t grad_dtype,
                           double *mean_var, uint32_t *nonfinite, void *stream);
/* Message of the calling thread's last ta_grad_moments_static failure ("" if none). */
const char *ta_static_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TRIACCEL_H */
