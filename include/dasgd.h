/*
 * libdasgd -- DaSGD (Local SGD with Delayed Averaging) hot path for NVIDIA B200 (sm_100a).
 *
 * K worker replicas of a P-element model live as rows of [K][ld] arrays in one GPU's memory
 * (ld >= P is the row stride in elements).  The library applies, with hand-written CUDA kernels,
 *   - the local step of every worker          (Eq. 2, "otherwise" branch, Section III-C-1),
 *   - the snapshot of the just-stepped weights (the bracketed term of Eq. 2's second branch),
 *   - the mean over the worker axis            (the (1/M)*sum_j of Eq. 2; "J" in the Appendix),
 *   - the delayed merge                        (Eq. 2, second branch),
 * and schedules the mean on a side stream so that it runs while the next local steps proceed
 * (the overlap of Section III, Fig. 2, and of Eq. 6's condition t_c < d*t_p).
 *
 * Conventions
 *   - Every pointer named "device" is a CUDA device pointer on the context's device; every
 *     pointer named "host" is ordinary (preferably page-locked) host memory.
 *   - All device buffers and both streams are owned by the caller and must stay valid until
 *     dasgd_destroy().  The library owns only its host-side context, its CUDA events and, when
 *     gradient staging is configured, one copy stream.
 *   - All calls are asynchronous with respect to the host except dasgd_sync, dasgd_get_timing
 *     and dasgd_destroy.  A context is not thread-safe; different contexts are independent.
 *   - Every call returns a dasgd_status and never aborts.  After a non-OK status
 *     dasgd_last_error() gives a one-line explanation.
 *   - Step counting: t = number of completed local steps.  Snapshots are taken when t is a
 *     positive multiple of tau; the snapshot taken at t = s is merged when t = s + d
 *     (Appendix form of the condition, (k+1-d) mod tau = 0; Fig. 2 for the indexing).
 */
#ifndef DASGD_H
#define DASGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dasgd_ctx dasgd_ctx;

typedef enum {
  DASGD_OK = 0,
  DASGD_ERR_INVALID_ARG = 1,   /* bad configuration or NULL / misaligned pointer            */
  DASGD_ERR_BAD_STATE = 2,     /* call out of order (nothing to average, nothing to merge)   */
  DASGD_ERR_NO_SLOT = 3,       /* snapshot requested while every slot holds a pending average */
  DASGD_ERR_CUDA = 4,          /* a CUDA runtime call failed; see dasgd_last_error            */
  DASGD_ERR_TIMEOUT = 5,       /* dasgd_sync gave up waiting                                  */
  DASGD_ERR_UNSUPPORTED = 6    /* valid request this library cannot serve                     */
} dasgd_status;

typedef enum {
  DASGD_F32 = 0,            /* gradients, weights, momentum: float32                                   */
  DASGD_BF16_MASTER_F32 = 1 /* gradients bfloat16; float32 master weights + momentum; a bfloat16 copy
                               of the weights (w_lp) is rewritten, round-to-nearest-even, with every
                               write of the master                                                    */
} dasgd_dtype;

typedef enum {
  DASGD_MERGE_XI = 0,   /* w_k <- xi*w_k + (1-xi)*mean          (Eq. 2, second branch)                 */
  DASGD_MERGE_DELTA = 1 /* w_k <- w_k + (mean - snapshot_k)     (not in the paper; keeps local progress) */
} dasgd_merge_mode;

/* flags */
#define DASGD_FLAG_TIMING 0x1u        /* record CUDA events around every average and every wait for it */
#define DASGD_FLAG_FUSE_SNAPSHOT 0x2u /* dasgd_step: store the snapshot from the kernel that last writes
                                         w in that step instead of running a separate copy             */
#define DASGD_FLAG_FUSE_MERGE 0x4u    /* dasgd_step: blend the mean inside the local-step kernel of the step
                                         the merge lands on (Eq. 2's second branch as one assignment).
                                         Applies when d >= 2, and when d == 1 if n_chunks > 1 or
                                         DASGD_FLAG_FUSE_MERGE_D1 is set                                */

#define DASGD_FLAG_ROTATE_SNAPSHOT 0x8u /* snapshots cost no copy: w and the n_slots arrays of snap form a
                                         pool of n_slots+1 weight arrays; a snapshot freezes the array that
                                         holds the current weights and the next kernel that writes weights
                                         writes them into a free array.  The current weights then move
                                         between arrays: ask dasgd_get_weights where they are.  Results are
                                         the same as without the flag.  FUSE_SNAPSHOT has no effect.        */

#define DASGD_FLAG_INLINE_MEAN 0x10u   /* dasgd_step runs ONE kernel per iteration: each thread walks the K rows
                                         of its parameters, does the local step and the merge that lands, and,
                                         when a snapshot is due, writes the mean of the K results directly.  No
                                         snapshot array is read or written (cfg.snap may be NULL) and the side
                                         stream stays idle: fastest schedule on one GPU, same results, but the
                                         mean is no longer computed asynchronously.  xi-blend merge only.  The
                                         explicit snapshot/average/merge calls keep working if snap is given. */

#define DASGD_FLAG_FUSE_MERGE_D1 0x80u /* with DASGD_FLAG_FUSE_MERGE and n_chunks <= 1: fold the merge into the
                                         step kernel also when d == 1.  The kernel of step s+1 then cannot start
                                         before the mean of step s is complete, so this pays off only when the
                                         caller's own work between two steps (forward/backward) gives the mean
                                         its window (the condition t_c < d*t_p of Eq. 6); with back-to-back steps
                                         use n_chunks instead                                                   */

#define DASGD_FLAG_TWO_LANES 0x100u    /* with n_chunks > 1: the step kernels of odd column ranges run on a second
                                         stream owned by the library, forked from the main stream at the start of
                                         the dasgd_step call and joined to it at its end, so that consecutive
                                         ranges overlap at their boundaries.  Work the caller enqueues on the
                                         main stream before / after the call is still ordered before / after all
                                         of it.  Results are unchanged.                                        */

#define DASGD_FLAG_GRAPH 0x200u        /* with n_chunks > 1: every chunked iteration is recorded once as a CUDA graph
                                         (stream capture of the very launches the library would issue) and then
                                         replayed, which removes most of the host's per-launch cost and lets more,
                                         smaller column ranges pay off.  The recorded kernels read the gradients
                                         pointer and the learning rate from a 16-byte device block that the library
                                         allocates at dasgd_init and frees at dasgd_destroy (its only device
                                         allocation).  A replay finishes when its last mean is complete, so the
                                         means of one iteration overlap the step kernels of the SAME iteration only.
                                         Ignored with DASGD_FLAG_TIMING (which times the same dependency structure
                                         with direct launches) and with a sharded worker axis.  Results unchanged. */

#define DASGD_FLAG_TWO_SIDE_STREAMS 0x400u /* with n_chunks > 1: the means of odd column ranges run on a second side
                                         stream owned by the library (same priority as side_stream), so that the mean
                                         of one range does not queue behind the mean of the range before it.  The two
                                         meet again at the end of every group of ranges and at the end of the
                                         dasgd_step call: whatever the caller orders after side_stream still comes
                                         after all means.  The best number of ranges becomes much less critical.
                                         Has no effect on a sharded worker axis.  Results unchanged.              */

/* Variants of the local step.  Section IV-A states only the values of momentum and weight decay used on the
 * paper's platform and gives no formula, so the common forms are all offered; the default is the plain one. */
#define DASGD_FLAG_NESTEROV 0x20u      /* w <- w - lr*(g' + mu*m) with the freshly updated m (needs momentum > 0) */
#define DASGD_FLAG_DECOUPLED_WD 0x40u  /* g' = g, and w <- w - lr*lambda*w - lr*(step direction): the decay acts
                                          on the weights directly instead of entering the momentum            */

typedef struct dasgd_config {
  int32_t K;            /* workers (the paper's M), >= 1                                              */
  int32_t tau;          /* local steps between snapshots, >= 1                                        */
  int32_t d;            /* delay in local steps between snapshot and merge, >= 0 (0 = Local SGD)      */
  int32_t dtype;        /* dasgd_dtype                                                                */
  int32_t merge_mode;   /* dasgd_merge_mode                                                           */
  int32_t n_slots;      /* snapshot/mean slots provided; must be >= max(1, ceil(d/tau))               */
  uint32_t flags;       /* DASGD_FLAG_*                                                               */
  int32_t device;       /* CUDA device ordinal that owns every buffer and both streams                */
  int64_t P;            /* parameters per worker, >= 1                                                */
  int64_t ld;           /* row stride in elements of every [K][ld] array; 0 means P.  Rows start on
                           16-byte boundaries (full-speed path) when ld % 8 == 0                      */
  float xi;             /* local proportion in the merge, 0 <= xi <= 1                                */
  float momentum;       /* mu; 0 disables the momentum buffer (m may then be NULL)                    */
  float weight_decay;   /* lambda, coupled L2: g' = g + lambda*w                                      */
  uint32_t sync_timeout_ms; /* dasgd_sync gives up after this long; 0 means 60000                     */
  int32_t n_stage;      /* gradient staging arrays behind g_stage: 0 (none), 1, or 2 (the copy of the
                           next step's gradients then overlaps this step's kernels)                   */
  int32_t n_chunks;     /* 0 or 1: off.  C > 1 (at most 1024; needs d >= 1, DASGD_FLAG_ROTATE_SNAPSHOT and
                           DASGD_FLAG_FUSE_MERGE): dasgd_step cuts the parameter axis into C column ranges
                           and pipelines them: the step kernel of range c (which blends the mean of range c
                           that lands) is followed on the side stream by the mean of range c of the new
                           snapshot, which runs beside the step kernels of ranges c+1, ...  With d == 1 the
                           merge then costs no pass of its own although the mean of step s is consumed by
                           step s+1; with any d >= 1 the mean of a range starts while much of the range is
                           still in the L2 cache.  Results are the same as without chunks.               */
  void *w;              /* device, [K][ld] float32, in/out: weights (master weights in bf16 mode); with
                           DASGD_FLAG_ROTATE_SNAPSHOT: where the weights START (see dasgd_get_weights)  */
  void *m;              /* device, [K][ld] float32, in/out: momentum buffers (start them at 0)        */
  void *w_lp;           /* device, [K][ld] bfloat16, out: low-precision weights; bf16 mode only       */
  void *snap;           /* device, [n_slots][K][ld] float32, scratch: snapshots (ROTATE: weight arrays) */
  void *mean;           /* device, [n_slots][ld] float32, scratch: worker-axis means                  */
  void *g_stage;        /* device, [n_stage][K][ld] gradient dtype, scratch for dasgd_step_host; may be NULL */
  void *main_stream;    /* cudaStream_t carrying local steps, snapshots and merges                    */
  void *side_stream;    /* cudaStream_t carrying the averages; must differ from main_stream           */
} dasgd_config;

/* Validates cfg, copies it, creates the events.  No kernel is launched.  *out is NULL on error
 * (the error text is then available from dasgd_last_error(NULL)). */
dasgd_status dasgd_init(dasgd_ctx **out, const dasgd_config *cfg);

/* Local step for all K workers on the main stream (Eq. 2 first branch; momentum / weight decay in
 * the usual form of Section IV-A's hyper-parameters):
 *     g' = g + lambda*w;   m <- mu*m + g';   w <- w - lr*m        (mu == 0: w <- w - lr*g')
 * grads: device, [K][ld], float32 or bfloat16 according to dtype; read only; must stay untouched
 * until the main stream has passed this call.  Increments t. */
dasgd_status dasgd_local_step(dasgd_ctx *ctx, const void *grads_device, float lr);

/* Main stream: copy w into a free slot (Eq. 2: the quantity that is averaged).  DASGD_ERR_NO_SLOT if
 * every slot still holds a pending average. */
dasgd_status dasgd_snapshot(dasgd_ctx *ctx);

/* Side stream: mean over the K rows of the oldest snapshot that has none yet.  Returns at once;
 * the main stream is not blocked.  DASGD_ERR_BAD_STATE if no such snapshot exists. */
dasgd_status dasgd_average_async(dasgd_ctx *ctx);

/* Main stream: wait (on the device) for the OLDEST pending average, blend it into every worker's
 * current weights according to merge_mode, release the slot.  DASGD_ERR_BAD_STATE if no average is
 * pending.  This wait is the only point where averaging can delay local work. */
dasgd_status dasgd_merge(dasgd_ctx *ctx);

/* Host waits (bounded by sync_timeout_ms) until both streams have drained; reports CUDA errors
 * raised by earlier asynchronous work.  Pending averages stay pending; nothing is applied. */
dasgd_status dasgd_sync(dasgd_ctx *ctx);

/* One iteration of the schedule, all asynchronous:
 *     local step;  if a snapshot from t-d is due, merge it;  if t % tau == 0, snapshot + average
 * (d == 0: snapshot, average and merge in the same iteration, i.e. Local SGD).  Honors the
 * FUSE flags; results are the same with and without them. */
dasgd_status dasgd_step(dasgd_ctx *ctx, const void *grads_device, float lr);

/* dasgd_step for callers whose gradients are in HOST memory: copies grads_host ([K][ld], gradient
 * dtype) into the next staging array of cfg.g_stage on a copy stream owned by the library, makes the
 * main stream wait for that copy, runs dasgd_step on it and, if probe_host != NULL, copies the first
 * probe_elems float32 weights of worker 0 back into probe_host on the main stream.  With n_stage = 2
 * the copy for call i+1 runs while the kernels of call i do.  Both host buffers must stay valid until
 * dasgd_sync returns (page-locked memory keeps the copies asynchronous).  DASGD_ERR_BAD_STATE if
 * cfg.g_stage was NULL or n_stage < 1. */
dasgd_status dasgd_step_host(dasgd_ctx *ctx, const void *grads_host, float lr, float *probe_host,
                             int64_t probe_elems);

/* Device pointer of the [K][ld] float32 array that holds the current weights: cfg.w, unless
 * DASGD_FLAG_ROTATE_SNAPSHOT is set, in which case it can be cfg.w or any of the n_slots arrays of
 * cfg.snap and is valid until the next call that writes weights (local_step, merge, step). */
dasgd_status dasgd_get_weights(const dasgd_ctx *ctx, void **w_device);

/* t, the number of completed local steps, and the number of snapshots awaiting their merge. */
dasgd_status dasgd_get_step(const dasgd_ctx *ctx, int64_t *t, int32_t *pending);

/* Device pointers of the i-th oldest pending slot (0 = oldest) and the step it was taken at.
 * *snap_device is NULL for a slot made by the DASGD_FLAG_INLINE_MEAN schedule (it has a mean but no
 * snapshot array). */
dasgd_status dasgd_get_pending(const dasgd_ctx *ctx, int32_t i, int64_t *s, void **snap_device,
                               void **mean_device);

/* Requires DASGD_FLAG_TIMING.  Synchronises, then returns sums over all averages completed since
 * the last dasgd_reset_timing: n_avg mean launches, ms_avg = time the mean kernels took on the side stream,
 * ms_stall = time streams spent blocked on them.  The stall of one wait is measured between two CUDA events
 * on the device clock: "the waiting stream has finished everything queued before the wait" and "the mean
 * kernel is complete"; it counts when the second comes after the first, else it is 0.  The fraction of
 * averaging hidden behind local work is 1 - ms_stall/ms_avg (Section V, Eq. 6). */
dasgd_status dasgd_get_timing(dasgd_ctx *ctx, int64_t *n_avg, double *ms_avg, double *ms_stall);

/* Requires DASGD_FLAG_TIMING.  Synchronises, then returns the number of launches and the summed
 * device time (CUDA events on the launching stream) of one kind of work since the last
 * dasgd_reset_timing: which = 0 local-step kernels (fused variants included), 1 snapshot copies,
 * 2 worker-axis means, 3 merge kernels, 4 the waits for a mean (n = waits issued, ms = time blocked). */
dasgd_status dasgd_get_kernel_timing(dasgd_ctx *ctx, int32_t which, int64_t *n, double *ms);

/* Synchronises and zeroes every timing counter. */
dasgd_status dasgd_reset_timing(dasgd_ctx *ctx);

/* Checkpointing.  The schedule state of a context (step counter, which array of the pool holds the
 * current weights, the pending snapshots and their slots) as an opaque blob of at most 4096 bytes.
 * dasgd_export_state synchronises both streams, then writes the blob to host_buf (*len receives its
 * size; DASGD_ERR_INVALID_ARG if buf_len is too small).  To checkpoint, save the blob together with the
 * contents of w, m, w_lp, snap and mean.  To resume, create a context with the same configuration
 * over buffers holding the saved contents and call dasgd_import_state before any other call; the run
 * then continues exactly as the original would have (the paper has no counterpart of these calls). */
dasgd_status dasgd_export_state(dasgd_ctx *ctx, void *host_buf, int64_t buf_len, int64_t *len);
dasgd_status dasgd_import_state(dasgd_ctx *ctx, const void *host_buf, int64_t len);

/* Delay guideline of Section III-D (Eq. 3) and Section VI-C/VI-D: the averaging is fully hidden when
 * t_c < d * t_p (t_c: time of one averaging, t_p: time of one local update, same unit), so *d is the
 * smallest positive integer with that property and *tau = *d + 1.  Pure host arithmetic.
 * DASGD_ERR_INVALID_ARG unless t_c >= 0, t_p > 0 and both outputs are non-NULL. */
dasgd_status dasgd_delay_guideline(double t_c, double t_p, int32_t *d, int32_t *tau);

/* The guideline applied to this context's own measurements.  Requires DASGD_FLAG_TIMING and at least
 * one timed local step and one timed mean.  t_c = average device time of the mean kernel; t_p = average
 * device time of the local-step kernel + extra_tp_ms (the caller's forward/backward time per step,
 * 0 if the gradients are precomputed).  Synchronises.  Outputs: *d, *tau, and (if non-NULL) the two
 * times in milliseconds. */
dasgd_status dasgd_advise_delay(dasgd_ctx *ctx, double extra_tp_ms, int32_t *d, int32_t *tau, double *t_c_ms,
                                double *t_p_ms);

/* Requires DASGD_FLAG_TIMING.  Synchronises, then returns how many replica-parameters (K times the columns
 * of each launch) the timed launches of one kind have processed since the last dasgd_reset_timing; `which`
 * as in dasgd_get_kernel_timing (4, the waits, always gives 0).  With n_chunks > 1 one step is several
 * launches, so bytes per second follow from units and time, not from the launch count. */
dasgd_status dasgd_get_kernel_units(dasgd_ctx *ctx, int32_t which, int64_t *units);

/* bf16 mode: rewrites the bfloat16 copy w_lp from the float32 master weights (round to nearest even) with
 * the library's own conversion, on the main stream.  Call it after writing initial weights into w, so that
 * no rounding of the method's state happens outside the library.  DASGD_ERR_BAD_STATE in float32 mode. */
dasgd_status dasgd_refresh_lp(dasgd_ctx *ctx);

/* ---- Momentum averaging (a variant; the paper has no counterpart: Section III averages the weights only and
 * Section IV-A says nothing about the momentum buffers at a merge, so by default they stay local).
 *
 * After this call the momentum buffers go through the same three operations as the weights, at the same moments:
 * every snapshot also copies m into the slot's [K][ld] array of m_snap (main stream), every mean is followed by the
 * worker-axis mean of that copy into the slot's [ld] vector of m_mean (side stream), and every merge also blends
 * the buffers, m_k <- xi*m_k + (1-xi)*mean_m (DASGD_MERGE_DELTA: m_k <- m_k + (mean_m - copy_k)), after the kernels
 * of that step have updated them.  These are passes of their own (8 + 4 + 4/K + 8 + 4/K bytes per
 * replica-parameter and cycle, 4 more for the delta form): the variant is for studying the method, not for speed.
 * m_snap: device, [n_slots][K][ld] float32; m_mean: device, [n_slots][ld] float32; both caller-owned, 16-byte
 * aligned, on cfg.device, borrowed until dasgd_destroy.  Call it right after dasgd_init (DASGD_ERR_BAD_STATE once
 * the context has been used).  Needs momentum > 0.  DASGD_ERR_UNSUPPORTED with DASGD_FLAG_INLINE_MEAN and on a
 * sharded worker axis; DASGD_FLAG_GRAPH is ignored.  dasgd_get_pending_momentum: the copy and the mean of the i-th
 * oldest pending snapshot (either pointer may be NULL). */
dasgd_status dasgd_set_momentum_averaging(dasgd_ctx *ctx, void *m_snap_device, void *m_mean_device);
dasgd_status dasgd_get_pending_momentum(const dasgd_ctx *ctx, int32_t i, void **m_snap_device, void **m_mean_device);

/* ---- Sharded worker axis (the data-parallel setting of Section II-B: the M workers live on several GPUs
 * and an all-reduce adds their contributions; Section III: the averaging runs while the local steps go on).
 *
 * A context then holds cfg.K of K_total workers.  Where the other entry points form the mean, such a
 * context (1) writes the plain float32 SUM of its own rows into the mean slot (skipped when cfg.K == 1: the
 * row is its own sum), (2) calls `exchange`, which must leave in recv_device the element-wise sum of
 * send_device over ALL shards, ordered on side_stream (an all-reduce enqueued on that stream), and
 * (3) divides by K_total, correctly rounded, where the merge reads the result.  The mean slots (and
 * dasgd_get_pending) therefore hold sums, not means.  Every shard must issue the same sequence of calls.
 * Call dasgd_set_shard right after dasgd_init.  Not available with DASGD_FLAG_INLINE_MEAN. */
typedef dasgd_status (*dasgd_exchange_fn)(void *user, const void *send_device, void *recv_device, int64_t count,
                                          void *side_stream);
dasgd_status dasgd_set_shard(dasgd_ctx *ctx, int32_t K_total, dasgd_exchange_fn exchange, void *user);

/* The exchange over NCCL: ncclAllReduce(sum, float32) on the side stream.  The NCCL library (libnccl.so.2) is
 * loaded on first use; DASGD_ERR_UNSUPPORTED if it cannot be.  Rank 0 makes an id (128 bytes, host) and hands
 * it to the other ranks by any means; every rank then creates its communicator with the device current that
 * owns its context, and passes it to dasgd_set_shard_nccl.  The communicator stays the caller's: destroy it
 * after the context. */
dasgd_status dasgd_nccl_unique_id(void *id128_host);
dasgd_status dasgd_nccl_comm_init(void **comm, const void *id128_host, int32_t nranks, int32_t rank, int32_t device);
dasgd_status dasgd_nccl_comm_destroy(void *comm);
dasgd_status dasgd_set_shard_nccl(dasgd_ctx *ctx, int32_t K_total, void *comm);

/* Number of kernels this context has launched so far. */
dasgd_status dasgd_get_launches(const dasgd_ctx *ctx, int64_t *launches);

const char *dasgd_strerror(dasgd_status s);
const char *dasgd_last_error(const dasgd_ctx *ctx); /* ctx may be NULL: last dasgd_init failure */
dasgd_status dasgd_destroy(dasgd_ctx *ctx);         /* synchronises both streams, frees the context */

/* Largest P that dasgd_average_merge_noalloc accepts (its built-in mean vector: 4 MiB). */
#define DASGD_NOALLOC_MAX_P 1048576

/* Averages K replicas and blends the mean back, in one call, WITHOUT any device buffer beyond w:
 *     mean[p] = (1/K) * sum_k w[k][p];    w[k][p] <- xi*w[k][p] + (1-xi)*mean[p]
 * i.e. what dasgd_snapshot + dasgd_average_async + dasgd_merge do with d = 0, for callers that
 * cannot allocate: a serving loop whose device memory pool is frozen once it is warm, a plug-in
 * that is handed a fixed arena by its host application, a process whose device allocator belongs to
 * another runtime and must not be bypassed.  (The paper has no counterpart of this call; it is a convenience of this library.)
 *
 * w_device: device, [K][ld] float32, in/out (ld = 0 means P).  stream: the cudaStream_t the two kernels
 * are enqueued on; the call does not wait for them.  device: ordinal of the GPU that holds w.
 * errbuf (may be NULL): receives a one-line explanation when the status is not DASGD_OK.
 *
 * The mean vector is kept in an array built into the library (DASGD_NOALLOC_MAX_P float32 = 4 MiB on
 * every GPU that loads the library, held until the process exits).  P > DASGD_NOALLOC_MAX_P is refused
 * with DASGD_ERR_UNSUPPORTED.  The call performs no cudaMalloc/cudaFree and calls no allocating routine.
 * The first call on each device looks up the array's device address; make that first call outside any
 * stream capture.  All calls on a device share the array: it keeps the previous call's contents, needs no
 * clearing (every element that is read is overwritten first), and two calls whose kernels can overlap
 * on the GPU (different streams without ordering between them) race on it -- order them. */
dasgd_status dasgd_average_merge_noalloc(void *w_device, int32_t K, int64_t P, int64_t ld, float xi,
                                         int32_t device, void *stream, char *errbuf, int64_t errbuf_len);

/* Library version, "major.minor". */
const char *dasgd_version(void);

#ifdef __cplusplus
}
#endif
#endif
