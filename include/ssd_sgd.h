/*
 * ssd_sgd.h - C ABI of the SSD-SGD update path on one NVIDIA B200 (sm_100a).
 *
 * SSD-SGD ("Several Steps Delay SGD", arXiv 2012.05396) trains with a
 * parameter server that applies a synchronous momentum-SGD update from the
 * gradients of K workers at every iteration, while each worker pulls the global
 * weight only once every k iterations and, in between, advances a local copy of
 * the weights with the GLU rule ("global gradient for local update").  This
 * library is the per-iteration parameter-update arithmetic of that method over
 * the flattened model state.  The K workers are K sets of buffers in one GPU's
 * memory: a "push" is the server kernel reading worker i's gradient buffer, a
 * "pull" is a store of the global weight into worker i's local weight.
 *
 * Conventions
 *  - Every pointer in ssd_buffers and every gradient pointer is DEVICE memory
 *    owned by the caller, 16-byte aligned (32-byte alignment of every buffer
 *    enables the 256-bit access path; buffers that start on 4 KB boundaries are
 *    measurably faster still, about 3 % on B200, because a thread block reads
 *    4 KB of every buffer per trip), holding at least ssd_arena_numel()
 *    elements.  The library never allocates, frees or retains device memory of
 *    its own; a context holds host-side metadata only.  Pointer *tables*
 *    (w_loc, pre, w_dev, grads) are HOST arrays of K device pointers and are
 *    copied when passed.
 *  - State is float32.  Gradients are float32 or bfloat16 (widened exactly).
 *  - Arithmetic: IEEE-754 binary32, round to nearest even, every multiply and
 *    add rounded separately (no fused multiply-add), operands in the order
 *    written below, the K gradients summed left to right (worker 0 first).
 *    Results are therefore unique and reproducible bit for bit.
 *  - Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as void*,
 *    NULL = the legacy default stream) and return without waiting for the GPU.
 *    Work of successive calls on the same stream is ordered by the stream.
 *    Three calls copy a small table out of ordinary (pageable) host memory of
 *    the context: ssd_set_tensor_scales, ssd_set_lr while per-tensor scales are
 *    set, and ssd_server_sync_update_static.  The CUDA runtime stages such a
 *    copy before the call returns, which can wait for earlier copies on that
 *    stream; nothing else in the library blocks the host.
 *  - Every call returns an ssd_status.  Arguments are validated before any
 *    launch: on an argument, alignment, layout or state error nothing was
 *    enqueued and no counter moved.  SSD_ERR_CUDA reports a failure of the CUDA
 *    runtime itself (ssd_last_cuda_error has its text); no counter moved, but
 *    work enqueued before the failing call stays enqueued.
 *  - A context is not thread-safe; use one per host thread or lock around it.
 *    It works on the CUDA device that is current when its first launching call is
 *    made (the device its buffers live on); keep that device current for every
 *    later call on the context.
 *
 * Arena layout.  A parameter layout is an ordered list of T tensors given by
 * their element counts.  Tensor t lives at element offset ssd_tensor_offset(t)
 * of every buffer; offsets are multiples of 4 elements (16 bytes in float32),
 * the gaps are padding that the update treats like any other element (keep
 * them zero).  All kernels sweep the arena as one flat stream.
 *
 * Schedule (Algorithm 1 and Algorithm 2 of the paper).  Iteration n = 0,1,...
 *   warm-up   n < W, or delay_k == 0: plain synchronous SGD; workers compute on
 *             the global weight.  On the last warm-up iteration (n == W-1) each
 *             worker keeps a copy of the new global weight as its local weight
 *             (SSD_FLAG_COPY).  W counts iterations: the paper's loop
 *             "while num <= wp" runs W = wp+1 times.
 *   delay     d = n - W >= 0.  Every iteration: server update, then one GLU
 *             update per worker.  SSD_FLAG_FIRST on d == 0 (pre_weight is
 *             initialised with the local weight), SSD_FLAG_REFRESH when d > 0
 *             and d % k == 0 (pre_weight is overwritten, Algorithm 2),
 *             SSD_FLAG_PULL when d % k == k-1 (Algorithm 1).  These tests equal
 *             the printed ones, num % k == k-1 and loc_update % k == 0, whenever
 *             the paper's own constraint (1+wp) % k == 0 holds, and stay well
 *             defined when it does not.
 */
#ifndef SSD_SGD_H
#define SSD_SGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ssd_ctx ssd_ctx;

typedef enum {
    SSD_OK = 0,
    SSD_ERR_ARG = 1,      /* NULL pointer, value out of range, unknown enum   */
    SSD_ERR_ALIGN = 2,    /* a device pointer is not 16-byte aligned          */
    SSD_ERR_LAYOUT = 3,   /* empty or oversized layout, negative element count */
    SSD_ERR_STATE = 4,    /* call not valid in the context's current stage    */
    SSD_ERR_CUDA = 5,     /* the CUDA runtime reported an error on launch     */
    SSD_ERR_NOMEM = 6,    /* host allocation of the context failed            */
    SSD_ERR_TOO_LARGE = 7 /* more tensors than the static per-tensor table holds */
} ssd_status;

typedef enum { SSD_F32 = 0, SSD_BF16 = 1 } ssd_dtype;

/* Local updater of the workers in the delay stage.  The paper's is GLU; its Section
 * 4.4 compares it with plain SGD, Eq. 5 (with the descent sign):
 *     w_loc_i[j] = w_loc_i[j] - lr_local * (g_i[j] + wd * w_loc_i[j])
 * which has no grad_sync: pre_weight is neither read nor written (the FIRST and
 * REFRESH flags have no effect) and alpha and beta are not used.  Pulls work the same. */
typedef enum { SSD_LOCAL_GLU = 0, SSD_LOCAL_SGD = 1 } ssd_local_updater;

enum { SSD_STAGE_WARMUP = 0, SSD_STAGE_DELAY = 1 };
enum { SSD_FLAG_FIRST = 1, SSD_FLAG_REFRESH = 2, SSD_FLAG_PULL = 4, SSD_FLAG_COPY = 8 };
enum { SSD_VIEW_GLOBAL = 0, SSD_VIEW_LOCAL = 1, SSD_VIEW_DEVICE = 2 };

#define SSD_MAX_WORKERS 32

/* Parameter layout: element counts of the T tensors (host array, copied). */
typedef struct {
    int32_t num_tensors;          /* T >= 1                                    */
    const int64_t *numel;         /* numel[t] >= 0; sum of padded counts < 2^40 */
} ssd_layout;

/* Hyper-parameters (Table 1 of the paper) and the schedule inputs of Algorithm 1. */
typedef struct {
    int32_t K;                    /* workers, 1..SSD_MAX_WORKERS                */
    float lr;                     /* server learning rate, > 0                  */
    float momentum;               /* m, 0 <= m < 1                              */
    float wd;                     /* weight decay, used by server and GLU       */
    int32_t warmup_iters;         /* W >= 0, number of SSGD iterations (wp + 1) */
    int32_t delay_k;              /* k >= 0; 0 = synchronous SGD forever        */
    float lr_local;               /* GLU learning rate; NaN = 4 * lr (Section 4.1) */
    float alpha;                  /* weight of the local gradient; NaN = 2.0    */
    float beta;                   /* weight of grad_sync; NaN = 0.5             */
    float rescale;                /* factor on the K-sum; NaN = 1/K (average)   */
    int32_t grad_dtype;           /* ssd_dtype of every gradient buffer         */
    int32_t local_updater;        /* ssd_local_updater; 0 = GLU                  */
} ssd_hparams;

/* Caller-owned device state.  w_loc, pre, w_dev: host arrays of K device pointers.
 * The K*3+2 buffers must not overlap each other or any gradient buffer: ssd_init
 * compares their byte ranges and every call that takes gradients compares those
 * with the state (SSD_ERR_ARG).  With delay_k == 0 (synchronous SGD only) no
 * worker state is ever touched and the three tables may be NULL.
 * `pre` alone may be NULL when pre_weight is not to live in device memory: see
 * ssd_set_host_pre_weight (or the plain-SGD local updater, which has none).
 * Shared pre_weight: the K pre_weight buffers always hold equal values (each worker
 * sets its own from the same pulled global weight: "the same pre_weight", Section
 * 3.3), so all K entries of `pre` may point at ONE buffer.  ssd_step then reads it
 * once per element instead of K times and writes it once (K-1 arenas less memory,
 * 4(K-1) bytes per parameter less traffic); results are unchanged.  The per-worker
 * calls (ssd_worker_glu_update, ssd_worker_local_step in the delay stage) would
 * overwrite it between workers and return SSD_ERR_STATE for such a context.
 * Merged device weights: w_dev[i] == w_loc[i] for every worker (all of them or none:
 * SSD_ERR_ARG otherwise) declares that the caller keeps no separate device weights.
 * Algorithm 1 hands the local update's result to the devices on a pull iteration and
 * then overwrites the local weight with the pulled global weight; with one buffer for
 * both, that result is overwritten before anyone could read it, so on pull iterations
 * the local update is skipped altogether: w_loc[i] = w (after pre_weight = old
 * w_loc[i], where the iteration writes pre_weight), and the next gradient is computed
 * on the pulled weight.  w, mom, w_loc and pre_weight are, bit for bit, what the
 * separate-buffer form gives, on every iteration; only the device-weight output of
 * pull iterations is not produced.  K arenas less memory; a fused pull iteration
 * moves K*(sg+4)+16 bytes per parameter instead of K*(sg+16)+16 (sg = bytes per
 * gradient element). */
typedef struct {
    float *w;                     /* global weight w_t (server)                 */
    float *mom;                   /* server momentum mom_t                      */
    float *const *w_loc;          /* local weight w'_{t,i} of each worker       */
    float *const *pre;            /* pre_weight of each worker                  */
    float *const *w_dev;          /* device weights of each worker; written only
                                     on pull iterations (see ssd_worker_weights) */
} ssd_buffers;

/* Arena length in elements for a layout: the sum of the element counts, each
 * rounded up to a multiple of 4.  Needs no context.  Errors: SSD_ERR_ARG (NULL),
 * SSD_ERR_LAYOUT. */
ssd_status ssd_arena_numel(const ssd_layout *layout, int64_t *padded_numel);

/* Creates a context.  Copies the layout, resolves NaN hyper-parameters to the
 * paper's defaults and derives, in double precision from the float-typed
 * hyper-parameters with one final rounding to float,
 *     c       = (1 - m) / (lr * k)      the grad_sync scale of Section 3.3
 *     rescale = 1 / K                   when averaging.
 * Does not touch any buffer.  Before the first step the caller sets w = w_0,
 * mom = 0 and, when warmup_iters == 0, also w_loc[i] = w_0 for every worker
 * (Algorithm 1 starts by pulling w_0); ssd_broadcast_weights does the latter.
 * Needs no CUDA device: the current device is looked up at the first launch,
 * and launching calls return SSD_ERR_CUDA when none is usable.
 * Errors: SSD_ERR_ARG, SSD_ERR_ALIGN, SSD_ERR_LAYOUT, SSD_ERR_NOMEM.  *out is
 * NULL on error. */
ssd_status ssd_init(ssd_ctx **out, const ssd_layout *layout, const ssd_hparams *hp,
                    const ssd_buffers *buffers);

/* Releases the context (host memory only).  NULL is accepted. */
void ssd_destroy(ssd_ctx *ctx);

/* Element offset of tensor `tensor` in every arena. */
ssd_status ssd_tensor_offset(const ssd_ctx *ctx, int32_t tensor, int64_t *elem_offset);

/* Stage and flags of iteration `iter` under the context's W and k (pure function
 * of its arguments and the two schedule inputs; see "Schedule" above). */
ssd_status ssd_schedule(const ssd_ctx *ctx, int64_t iter, int32_t *stage, int32_t *flags);

/* Server side of one iteration (Eq. 6 with momentum, Section 3.2.1): for every
 * arena element j
 *     s    = ((g_0[j] + g_1[j]) + g_2[j]) + ... + g_{K-1}[j]
 *     grad = s * rescale
 *     mom[j] = m * mom[j] - lr * (grad + wd * w[j])
 *     w[j]   = w[j] + mom[j]
 * `grads`: host array of K device pointers (dtype = grad_dtype), read only.
 * Does not read or move the context's counters: it is the whole of synchronous
 * SGD when used alone.  One kernel launch. */
ssd_status ssd_server_sync_update(ssd_ctx *ctx, const void *const *grads, void *cuda_stream);

/* ssd_server_sync_update with per-tensor hyper-parameters for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this is a packaging of the
 * server update above, not a step of the method.)
 *
 * Per-tensor scales normally need a device table that the caller allocates and
 * hands to ssd_set_tensor_scales.  Some callers have no way to do that: a plugin
 * that runs inside a host program whose memory pool has already claimed the whole
 * GPU, a service with a fixed device-memory budget, or a section of code in which
 * cudaMalloc is off limits because it synchronises the device.  For them the table
 * lives in a fixed array inside this library's device image (24 KB on every GPU
 * that loads the library, for as long as the process lives), and this call fills
 * it and runs the server update in one go.  It calls no cudaMalloc, cudaFree or
 * any other allocating routine.
 *
 * lr_mult, wd_mult: HOST arrays of num_tensors floats, as for
 * ssd_set_tensor_scales (NULL = all 1; lr_mult > 0); they are read before the call
 * returns.  grads, w and mom as for ssd_server_sync_update.  The result equals,
 * bit for bit, ssd_set_tensor_scales followed by ssd_server_sync_update.  The
 * context's own table (if any) is neither used nor changed.
 *  - Layouts with more than SSD_STATIC_TABLE_MAX_TENSORS tensors are rejected with
 *    SSD_ERR_TOO_LARGE before anything is enqueued.
 *  - The first call on each device looks up the array's device address (with that
 *    device current).  Make that first call before starting any stream capture.
 *    The context's device must be the current one (SSD_ERR_STATE otherwise).
 *  - The array is shared by every context and every call in the process and keeps
 *    what the last call wrote; each call overwrites the entries it uses.  Two calls
 *    whose work can overlap on the GPU (different streams, or different contexts on
 *    different streams) race on it: keep such calls on one stream or order them
 *    with events. */
#define SSD_STATIC_TABLE_MAX_TENSORS 1024
ssd_status ssd_server_sync_update_static(ssd_ctx *ctx, const void *const *grads, const float *lr_mult,
                                         const float *wd_mult, void *cuda_stream);

/* One GLU call of worker `worker` (Algorithm 2 and the GLU rule of Section
 * 3.2.1, with the descent sign that the server rule and grad_sync imply):
 *     if FIRST:   pre_i[j] = w_loc_i[j]
 *     gs = (pre_i[j] - w_loc_i[j]) * c
 *     if REFRESH: pre_i[j] = w_loc_i[j]                (value before the update)
 *     r  = w_loc_i[j] - lr_local * ((alpha * g_i[j] + wd * w_loc_i[j]) + beta * gs)
 *     if PULL:    w_dev_i[j] = r ; w_loc_i[j] = w[j]   (Algorithm 1: the devices keep
 *                 the GLU result, the local weight takes the pulled global weight)
 *     else:       w_loc_i[j] = r
 * `flags` is any combination of SSD_FLAG_FIRST / REFRESH / PULL.  With PULL, `w`
 * must already hold this iteration's server result (enqueue the server update
 * first on the same stream).  For a context with merged device weights a PULL call
 * reduces to: if FIRST or REFRESH: pre_i[j] = w_loc_i[j]; then w_loc_i[j] = w[j].
 * Does not read or move the counters.  Errors:
 * SSD_ERR_ARG (worker out of range, unknown flag, NULL grad), SSD_ERR_STATE
 * (delay_k == 0: there is no delay stage), SSD_ERR_ALIGN.  One kernel launch. */
ssd_status ssd_worker_glu_update(ssd_ctx *ctx, int32_t worker, const void *grad, int32_t flags,
                                 void *cuda_stream);

/* Body of Algorithm 1 for one worker at the context's current iteration, to be
 * enqueued after ssd_server_sync_update of the same iteration: in the warm-up
 * stage it stores w into w_loc_i on the last warm-up iteration and does nothing
 * otherwise (`grad` may be NULL there); in the delay stage it is
 * ssd_worker_glu_update with the flags of ssd_schedule.  Does not move the
 * counters: call ssd_advance once all K workers are enqueued. */
ssd_status ssd_worker_local_step(ssd_ctx *ctx, int32_t worker, const void *grad, void *cuda_stream);

/* Ends an iteration assembled from the two calls above: iter += 1 and, in the
 * delay stage, loc_update += 1. */
ssd_status ssd_advance(ssd_ctx *ctx);

/* One whole iteration for the server and all K workers, then ssd_advance.  Same
 * results, bit for bit, as ssd_server_sync_update + K * ssd_worker_local_step,
 * but as ONE fused kernel in which every gradient element is read once and
 * feeds both the server sum and its own worker's GLU update (the paper notes
 * that push and local update only read the gradient, Section 2.2).
 * CUDA graphs: the call is one kernel launch plus host bookkeeping, so it can be made
 * while `cuda_stream` is being captured.  The launch is recorded with the buffers and
 * the flags of the iteration at capture time; the flags of the delay stage repeat
 * with period k from its second iteration on, so a captured run of k consecutive
 * delay-stage iterations (not containing the first GLU call) can be replayed for any
 * later period, with the gradients written into the same buffers before each replay.
 * The counters move only when the call is made, not when the graph is replayed:
 * after each replay set them with ssd_set_counters(iter + k, loc_update + k).  Run
 * one period outside capture first (the first launch of each kernel variant asks the
 * runtime for its occupancy).  For arenas of a few MB, where a step lasts
 * microseconds, replaying a period takes the launch latency out (ResNet-20 layout,
 * K = 4: 4.1 instead of 9.5 us per step on B200). */
ssd_status ssd_step(ssd_ctx *ctx, const void *const *grads, void *cuda_stream);

/* ssd_step restricted to the tensors [first_tensor, first_tensor + num_tensors) of the
 * layout (their arena range, padding included), at the context's current
 * iteration, WITHOUT moving the counters.  The paper's training pipeline pushes and
 * updates layer by layer while the backward pass is still producing the gradients
 * of earlier layers (Section 2.1); this is the call for that: enqueue one group of
 * layers as soon as their gradients are ready, in any order, each tensor exactly
 * once per iteration, then call ssd_advance.  The update is elementwise, so the
 * result equals one ssd_step over the whole arena, bit for bit.  `grads` are the K
 * whole gradient arenas, as for ssd_step.  One kernel launch per call (none when
 * the tensors are all empty).  Errors: SSD_ERR_ARG (range outside the layout). */
ssd_status ssd_step_tensors(ssd_ctx *ctx, const void *const *grads, int32_t first_tensor,
                            int32_t num_tensors, void *cuda_stream);

/* ssd_step for gradients that arrive in HOST memory (as they would from a
 * network push).  `host_grads`: K host pointers (pinned memory, or the copies are
 * not asynchronous); `staging`: K device buffers of arena size (gradient dtype) that
 * receive them; `host_w_out`: optional host buffer that receives the new global
 * weight w (NULL = no read-back).  The arena is processed in chunks of 2^24
 * elements (ssd_set_host_chunk): the host-to-device copies of one chunk, the update of the previous one
 * and the device-to-host copy of the one before overlap, on two side streams that
 * the context creates at the first call (driver objects, no device memory).  All of
 * it is ordered after the work already on `cuda_stream`, and `cuda_stream` ends
 * behind the last copy: the caller synchronises `cuda_stream` before reading
 * host_w_out or reusing host_grads.  One kernel launch per chunk.  Errors:
 * SSD_ERR_ARG, SSD_ERR_ALIGN, SSD_ERR_STATE (delay stage of a context without
 * pre_weight buffers and without ssd_set_host_pre_weight), SSD_ERR_CUDA. */
ssd_status ssd_step_host(ssd_ctx *ctx, const void *const *host_grads, void *const *staging,
                         float *host_w_out, void *cuda_stream);

/* Elements per chunk of ssd_step_host: a multiple of 1024, at most 2^30; 0 = the
 * default 2^24.  Results do not depend on it.  SSD_ERR_STATE while a host-resident
 * pre_weight is set (its device slices were sized for the current chunk). */
ssd_status ssd_set_host_chunk(ssd_ctx *ctx, int64_t chunk_elems);

/* pre_weight in HOST memory.  The paper keeps the backup of the pulled weights
 * (pre_weight) in CPU-side memory so that it does not occupy the accelerator
 * (Section 3.5, "Embedding in Framework").  For a context created with
 * ssd_buffers.pre == NULL this call names where it lives instead:
 *   host_pre       ONE host arena of ssd_arena_numel() floats (pinned memory, or the
 *                  copies are not asynchronous), 16-byte aligned.  One arena serves
 *                  all K workers, whose pre_weights always hold equal values (see
 *                  "Shared pre_weight" above).  The library reads and writes it;
 *                  its content is part of the state (keep it across a checkpoint).
 *   device_slices  device memory of slots * min(chunk, ssd_arena_numel()) floats
 *                  (chunk = the ssd_step_host chunk, 2^24 unless changed), 16-byte
 *                  aligned (32 for the 256-bit path), not overlapping any state buffer;
 *   slots          1..8 slices; 2 or more let the copy of one chunk's slice overlap
 *                  the update of the previous chunk.
 * ssd_step_host then streams pre_weight with the gradients: per chunk, the slice is
 * copied host-to-device next to the K gradient slices (except on the first GLU
 * call, which does not read pre_weight), the fused step runs on the chunk with the
 * slice as the one pre_weight of all workers, and on the iterations that overwrite
 * pre_weight (first GLU call, refresh) the slice is copied back device-to-host on
 * the side stream that also returns w.  Per step that is 4 bytes per parameter more
 * host-to-device traffic (1/K of the gradients' when they are float32), 4 more
 * device-to-host on one iteration in k, and K arenas of device memory less than
 * private pre_weights (one less than a shared one).  Results equal the
 * device-resident forms bit for bit.
 * ssd_step_host also accepts host_grads == NULL in every mode: the gradients are
 * then taken to be in `staging` already (device memory) and only pre_weight and w
 * cross the bus.
 * All other delay-stage calls (ssd_step, ssd_step_tensors, the per-worker calls)
 * need pre_weight in device memory and return SSD_ERR_STATE for such a context.
 * (NULL, NULL, 0) switches it off again.  Errors: SSD_ERR_ARG, SSD_ERR_ALIGN,
 * SSD_ERR_STATE (the context has device pre_weight buffers, no worker state, or
 * delay_k == 0). */
ssd_status ssd_set_host_pre_weight(ssd_ctx *ctx, float *host_pre, float *device_slices, int32_t slots);

/* w_loc[i] = w for every worker (the initial pull of Algorithm 1).  Needed before
 * the first step only when warmup_iters == 0.  One kernel launch.  SSD_ERR_STATE
 * when the context was created without worker state. */
ssd_status ssd_broadcast_weights(ssd_ctx *ctx, void *cuda_stream);

/* Where worker `worker` finds the weights for its next forward/backward pass
 * after the iterations done so far: the global w in the warm-up stage, w_loc_i
 * after a GLU step without pull, w_dev_i after a pull iteration (w_loc_i, which
 * then holds the pulled weight, for a context with merged device weights).  `view`
 * receives the SSD_VIEW_* code; either output may be NULL. */
ssd_status ssd_worker_weights(const ssd_ctx *ctx, int32_t worker, const float **weights,
                              int32_t *view);

/* Counters: iterations done (Algorithm 1's num) and GLU calls done per worker
 * (Algorithm 2's loc_update); stage and flags of the NEXT iteration.  Outputs
 * may be NULL.  ssd_set_counters restores them (resume from a checkpoint whose
 * buffers the caller has restored); loc_update must equal max(0, iter - W) when
 * delay_k > 0 and 0 otherwise, else SSD_ERR_STATE. */
ssd_status ssd_get_counters(const ssd_ctx *ctx, int64_t *iter, int64_t *loc_update,
                            int32_t *next_stage, int32_t *next_flags);
ssd_status ssd_set_counters(ssd_ctx *ctx, int64_t iter, int64_t loc_update);

/* Changes the learning rates between iterations and re-derives c.  NaN keeps a
 * value.  (The geometric-series argument behind grad_sync assumes a constant lr;
 * after a change grad_sync is an estimate under the new lr.)  When per-tensor
 * scales are set, the table is rebuilt and its upload enqueued on `cuda_stream`,
 * so the change is ordered with the steps enqueued on that stream. */
ssd_status ssd_set_lr(ssd_ctx *ctx, float lr, float lr_local, void *cuda_stream);

/* Per-tensor hyper-parameters.  The paper uses one lr and one wd for the whole
 * model; this is the usual refinement (e.g. no weight decay on BN and bias).
 * Tensor t, padding up to the next tensor included, then uses
 *     lr_t = lr * lr_mult[t],  lr_local_t = lr_local * lr_mult[t],  wd_t = wd * wd_mult[t]
 * (one float multiplication each) and c_t = (1 - m) / (lr_t * k), in place of the
 * uniform values, in the server rule and in the GLU rule alike.
 * lr_mult, wd_mult: HOST arrays of num_tensors floats (NULL = all 1; lr_mult > 0).
 * device_table: caller-owned DEVICE memory of ssd_tensor_table_bytes() bytes,
 * 16-byte aligned, which the kernels read from then on and which must stay
 * valid until it is replaced; the library fills it by a copy enqueued on
 * `cuda_stream`.  device_table == NULL returns to uniform hyper-parameters.
 * Errors: SSD_ERR_ARG, SSD_ERR_ALIGN, SSD_ERR_CUDA. */
ssd_status ssd_tensor_table_bytes(const ssd_ctx *ctx, int64_t *bytes);
ssd_status ssd_set_tensor_scales(ssd_ctx *ctx, const float *lr_mult, const float *wd_mult,
                                 void *device_table, void *cuda_stream);

/* Resolved hyper-parameters as the kernels use them, and the derived c. */
ssd_status ssd_get_hparams(const ssd_ctx *ctx, ssd_hparams *resolved, float *sync_scale);

/* Launch shape of every kernel of this context: threads per block (multiple of
 * 32, 64..512) and resident blocks per SM (1..32, capped at what fits).  Each call
 * sets both; 0 for either returns that one to the per-kernel default, which depends
 * on the kernel, K, the gradient type and the iteration's flags.  Results do not
 * depend on it. */
ssd_status ssd_set_launch(ssd_ctx *ctx, int32_t threads_per_block, int32_t blocks_per_sm);

/* Shape of the kernels' inner loop.  vector_elems: elements each thread owns per
 * trip: 16 (two 256-bit accesses to float32 data, one to bfloat16 gradients), 8
 * (one 256-bit access to float32 data, 128 bits of bfloat16) or 4 (128-bit); the
 * wide forms are used only when every buffer involved is 32-byte aligned, else
 * the next narrower one is taken.  batch: workers whose loads a thread issues
 * together, 1, 2, 4 or 8 (the fused step uses at most 4, and at most 2 with
 * vectors of 8 or 16, beyond which registers would spill; kernels with vectors of
 * 16 run at most 256 threads per block).  0 = the default for the kernel, K,
 * gradient type and alignment.  Results do not depend on either. */
ssd_status ssd_set_kernel_shape(ssd_ctx *ctx, int32_t vector_elems, int32_t batch);

/* The overrides as last set by ssd_set_launch and ssd_set_kernel_shape (0 = default).
 * Outputs may be NULL. */
ssd_status ssd_get_launch(const ssd_ctx *ctx, int32_t *threads_per_block, int32_t *blocks_per_sm,
                          int32_t *vector_elems, int32_t *batch);

/* Shared-memory staging for the fused step.  stages = 2..8 makes ssd_step (and its
 * range forms) in the delay stage use a kernel in which one thread per block streams
 * the inputs into a ring of `stages` shared-memory buffers with bulk asynchronous
 * copies and 256 threads consume them; 0 (the default) is the register path.  On
 * B200 the register path is the faster one; the staged kernel is kept for comparison
 * and gives the same bits.  Contexts with a shared pre_weight or the plain-SGD
 * updater, and bfloat16 ranges that do not start and end on multiples of 8 elements,
 * stay on the register path.  Every wait inside the staged kernel is bounded; if one
 * ever runs out, the launch ends early with its results incomplete and
 * ssd_staging_error reports 1 (process-wide, sticky; the call synchronises the
 * device). */
ssd_status ssd_set_staging(ssd_ctx *ctx, int32_t stages);
ssd_status ssd_staging_error(ssd_ctx *ctx, int32_t *flag);

/* Number of kernels this context has launched so far. */
int64_t ssd_kernel_launches(const ssd_ctx *ctx);

/* Text for a status code (static storage). */
const char *ssd_status_str(ssd_status status);

/* Text of the last CUDA runtime error a call on this context returned as
 * SSD_ERR_CUDA (static or context storage; empty string if none). */
const char *ssd_last_cuda_error(const ssd_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SSD_SGD_H */
