/* softsync_ps.h — C ABI of the n-softsync parameter server (one GPU).
 *
 * The calls follow the protocol of "Staleness-aware Async-SGD for Distributed
 * Deep Learning" (arXiv 1511.05950), Section 2.1: a learner pulls the weights
 * together with the server's scalar timestamp, computes a gradient, and pushes
 * it back tagged with that timestamp; the server sums c = floor(lambda / n)
 * gradients (Section 2.2, Eq. 2), scales each by a learning rate that depends
 * on its staleness (Section 2.4, Eq. 3) and advances the timestamp by one.
 *
 * Conventions
 *   - Pointers named *_dev are device pointers on the GPU that was current when
 *     ps_create ran (later calls may be made with any device current: the library switches to
 *     the server's GPU and back); *_host are host pointers.  The library allocates no device
 *     memory: weights, momentum and staging slots are bound by the caller.
 *   - All device work is enqueued on one stream (PS_OPT_STREAM, default: the
 *     legacy default stream).  Calls return once the work is enqueued unless
 *     stated otherwise.
 *   - Every function returns a ps_status; negative values are errors and leave
 *     the server state unchanged.  Nothing aborts or throws.
 *   - A handle is not thread-safe: the paper's server handles one blocking call
 *     at a time (Section 2.3) and so does this one.
 */
#ifndef SOFTSYNC_PS_H
#define SOFTSYNC_PS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ps_ctx ps_t;               /* opaque; created by ps_create, freed by ps_destroy */

enum ps_modulation {
    PS_MOD_CONSTANT = 0,                  /* alpha = alpha0 for every gradient (Section 4.3, case (a)) */
    PS_MOD_INV_STALENESS = 1,             /* alpha = alpha0 / max(tau, 1)       (Eq. 3; alpha0 at tau = 0) */
    PS_MOD_EXP_STALENESS = 2              /* alpha = alpha0 * rho^tau: the exponential penalty of the earlier work
                                           * that Section 1 compares Eq. 3 with; rho: ps_set_penalty_base */
};

enum ps_status {
    PS_OK = 0,
    PS_READY = 1,                         /* ps_push_gradient: this push completed a group of c */
    PS_ERR_INVALID_ARG = -1,
    PS_ERR_BAD_LEARNER = -2,              /* learner id outside [0, lambda) */
    PS_ERR_BAD_TIMESTAMP = -3,            /* ts < 0 or ts > server timestamp: staleness would be negative (Section 2.1) */
    PS_ERR_NOT_READY = -4,                /* ps_apply_update: no complete group is pending */
    PS_ERR_QUEUE_FULL = -5,               /* too many unapplied groups, or no free staging slot */
    PS_ERR_CUDA = -6,                     /* a CUDA call failed; see ps_last_cuda_error */
    PS_ERR_NOMEM = -7,                    /* host allocation failed */
    PS_ERR_NO_STATE = -8,                 /* weights/momentum (or staging slots) not bound yet */
    PS_ERR_LOG_EVICTED = -9,              /* requested log range is no longer (or not yet) held */
    PS_ERR_BARRIER = -10,                 /* hardsync: this learner has already contributed to the current round */
    PS_ERR_DEVICE_WAIT = -11,             /* a bounded wait inside an update kernel ran out (PS_KERNEL_BULK); theta and v
                                           * are partly updated and must be re-initialised; see ps_kernel_status */
    PS_ERR_STATIC_LIMIT = -12             /* ps_fused_update_static: more blocks than PS_STATIC_MAX_BLOCKS or more
                                           * gradients than PS_STATIC_MAX_GRADS: the fixed status area cannot hold it */
};

enum ps_grad_dtype { PS_GRAD_FP32 = 0, PS_GRAD_BF16 = 1 };

enum ps_option {
    PS_OPT_GRAD_DTYPE = 1,                /* ps_grad_dtype of every pushed gradient; only while nothing is pending */
    PS_OPT_FUSE_T = 2,                    /* max groups applied by one kernel pass, 1..PS_MAX_FUSE_T (default 1) */
    PS_OPT_STREAM = 3,                    /* cudaStream_t as an integer (default 0); only while nothing is pending.
                                           * Work already enqueued on the old stream is ordered before the new one. */
    PS_OPT_QUEUE_GROUPS = 4,              /* max complete-but-unapplied groups (default 64) */
    PS_OPT_LOG_UPDATES = 5,               /* how many most recent updates the log keeps (default max(1024, 2^20 / c)) */
    PS_OPT_TIMING = 6,                    /* 1: bracket every update kernel with CUDA events (ps_kernel_time) */
    PS_OPT_KERNEL = 7,                    /* ps_kernel_choice (default PS_KERNEL_AUTO) */
    PS_OPT_BLOCK_THREADS = 8,             /* threads per block: 128, 256 or 512; 0 = default (128; 512 for PS_KERNEL_BULK) */
    PS_OPT_OVERLAP_LAUNCH = 9,            /* 1: update kernels are launched as programmatic dependents (see below); default 0 */
    PS_OPT_PROTOCOL = 10,                 /* ps_protocol (default PS_PROTOCOL_SOFTSYNC); only while nothing is pending */
    PS_OPT_GROUP_SIZE = 11,               /* read-only: c = floor(lambda / n) of Eq. 2 */
    PS_OPT_LAST_KERNEL = 12,              /* read-only: ps_kernel_choice the most recent update launch took (0: none yet) */
    PS_OPT_LAUNCHES_SCALAR = 13,          /* read-only: update launches so far that took the scalar kernel, */
    PS_OPT_LAUNCHES_VECTOR = 14,          /*            the vector kernel, */
    PS_OPT_LAUNCHES_BULK = 15,            /*            the bulk-copy kernel */
    PS_OPT_BULK_TILE = 16,                /* PS_KERNEL_BULK: elements per shared-memory tile, a power of two in
                                           * [256, 8192] (halved until the stages of one block fit 200 KB of an SM's
                                           * shared memory); 0 = the largest that fits (default) */
    PS_OPT_BULK_STAGES = 17,              /* PS_KERNEL_BULK: tiles in flight per block, 2..8 (default 2) */
    PS_OPT_BULK_WAIT_LIMIT = 18,          /* PS_KERNEL_BULK: polls of a copy barrier before the kernel gives up
                                           * (default 2^20, about a second; at least 16) */
    PS_OPT_BULK_SELFTEST = 19,            /* PS_KERNEL_BULK, diagnostics: 1 makes block 0 of the NEXT launch announce 16
                                           * bytes more than it copies for its first tile, so that tile's wait runs out;
                                           * the launch then ends with PS_ERR_DEVICE_WAIT recorded.  Resets to 0. */
    PS_OPT_ZIGZAG = 20                    /* 1 (default): successive update launches walk the vector in opposite directions,
                                           * so a launch starts on the part of theta and v the previous one left in
                                           * the L2; 0: every launch walks forward.  Same bits either way. */
};

/* PS_OPT_OVERLAP_LAUNCH = 1 lets an update kernel start while the previous kernel on the stream is still
 * draining: it fetches its gradients at once and waits for the previous kernel only before it reads
 * theta and v.  The caller promises in return that no gradient buffer is produced by the kernel that
 * directly precedes a ps_apply_update on the server's stream and may still be running (gradients written
 * by earlier kernels, by kernels the host has already synchronised with, by copies, or on other streams
 * with proper ordering are fine).  Results are bit-identical either way. */

/* Section 2.2 describes two protocols.  n-softsync (the default): an update after c = floor(lambda/n)
 * gradients from any learners, stale gradients welcome.  Hardsync (Eq. 1, synchronous SGD): one update per
 * round from exactly one gradient of every learner, all computed on the current weights.  In hardsync mode
 * (needs n = 1, so c = lambda) ps_push_gradient enforces the barrier: a gradient whose timestamp is not the
 * server's current one is refused with PS_ERR_BAD_TIMESTAMP (staleness must be 0), a second gradient from a
 * learner within one round with PS_ERR_BARRIER.  The update itself is the same kernel: Eq. 2 with all
 * staleness 0 is Eq. 1. */
enum ps_protocol { PS_PROTOCOL_SOFTSYNC = 0, PS_PROTOCOL_HARDSYNC = 1 };

enum ps_kernel_choice {
    PS_KERNEL_AUTO = 0,                   /* vector kernel when the pointers are aligned for it, else scalar */
    PS_KERNEL_SCALAR = 1,                 /* one element per thread */
    PS_KERNEL_VECTOR = 2,                 /* four elements per thread, streamed through registers: 16-byte accesses to
                                           * theta, v and fp32 gradients, 8-byte ones to bf16 gradients and the bf16
                                           * mirror; needs exactly those alignments */
    PS_KERNEL_BULK = 3                    /* persistent blocks that stage tiles of theta, v and the gradients in shared
                                           * memory with bulk asynchronous copies (cp.async.bulk + mbarrier, one block per
                                           * cluster, no multicast).  Needs every pointer 16-byte aligned and at most 16
                                           * gradients per launch (T * c <= 16), else PS_ERR_INVALID_ARG.  Same bits as the
                                           * other kernels.  Never chosen by PS_KERNEL_AUTO: on this element-wise, touch-once
                                           * pass it measures level with the register kernel at best (large tiles, two
                                           * stages) and is the more restricted of the two; it exists so that the
                                           * comparison can be repeated.  Every barrier wait in it is bounded
                                           * (PS_OPT_BULK_WAIT_LIMIT).  Its first launch allocates 64 bytes of pinned host
                                           * memory for the status record. */
};

#define PS_MAX_GROUP 256                  /* largest c = floor(lambda / n) */
#define PS_MAX_FUSE_T 16                  /* largest temporal-fusion depth */
#define PS_MAX_ENTRIES 512                /* largest T * c one kernel pass takes; T is clamped to fit */
#define PS_MAX_LAYERS 64                  /* largest layer table of ps_set_layer_multipliers */
#define PS_MAX_REPLICAS 8                 /* most weight replicas of ps_bind_weight_replicas */

/* One gradient's part in one weight update; what the server decided, for checking
 * against Section 2.1 (timestamp, staleness) and Eq. 2-3 (grouping, scale). */
typedef struct ps_log_entry {
    int64_t update;                       /* timestamp i the update started from (it produced i + 1) */
    int64_t push_index;                   /* how many gradients this learner had pushed before */
    int64_t ts_grad;                      /* j: timestamp of the weights the gradient was computed on */
    int64_t tau;                          /* staleness i - j >= 0 */
    int64_t sigma;                        /* staleness used in the learning rate: max(tau, 1) for PS_MOD_INV_STALENESS,
                                           * 1 for PS_MOD_CONSTANT, tau for PS_MOD_EXP_STALENESS */
    int32_t learner;
    int32_t position;                     /* place in the summation order of the group, 0 .. c-1 */
    float scale;                          /* s = alpha0 / (c * sigma) (alpha0 * rho^tau / c for the exponential penalty),
                                           * rounded to fp32 once */
    float decay;                          /* d = weight_decay * sum of the group's scales (fp32) */
} ps_log_entry;

/* Section 2.1-2.2.  Creates a server for `num_params` fp32 weights, `lambda` learners and
 * splitting parameter n (1 <= n <= lambda; c = floor(lambda / n) <= PS_MAX_GROUP).
 * alpha0: base learning rate; momentum, weight_decay: see ps_apply_update; modulation:
 * ps_modulation.  Timestamp starts at 0.  The handle is owned by the library. */
int ps_create(ps_t **out, int64_t num_params, int lambda, int n,
              float alpha0, float momentum, float weight_decay, int modulation);

/* Frees the handle (not the caller's device buffers).  Waits for enqueued work first. */
int ps_destroy(ps_t *ps);

/* Binds caller-owned device buffers of num_params fp32 each: weights theta and momentum v.
 * They must stay valid until ps_destroy and must not overlap.  4-byte alignment is enough; 16-byte
 * alignment enables the vector kernel.  Does not touch their contents (a bf16 mirror bound earlier is
 * refilled from the new weights). */
int ps_bind_state(ps_t *ps, float *w_dev, float *v_dev);

/* The starting point of Section 2.1: sets theta_0 (copied from w_src, host memory if src_is_host != 0,
 * else device), zeroes the momentum, resets the timestamp to 0 (the clock of Section 2.1 starts at
 * 0 and gains one per weight update), and drops pending gradients, the log and a recorded
 * PS_ERR_DEVICE_WAIT. */
int ps_init_weights(ps_t *ps, const float *w_src, int src_is_host);

/* Binds a caller-owned device buffer of num_params bf16 values (2-byte aligned; 8-byte aligned keeps the
 * vector kernel) that from now on always holds theta rounded to nearest-even bf16: it is filled at once
 * (and by ps_init_weights), and every ps_apply_update rewrites it in the same pass that updates theta
 * (2 more bytes per element instead of a separate conversion pass).  Learners that compute in bf16 can
 * read it in place after the update, or take a copy with ps_pull_weights_bf16.  NULL unbinds.
 * Not in the paper (its weights are 4-byte, Section 4.1). */
int ps_bind_weight_mirror(ps_t *ps, void *mirror_bf16_dev);

/* Weight broadcast fused into the update.  Section 2.2 has the server send the updated weights to the learners;
 * Section 2.3 shards the server.  Binds up to PS_MAX_REPLICAS further fp32 buffers of num_params elements that
 * from now on always hold theta as well: they are filled at once (and by ps_init_weights), and every
 * ps_apply_update stores the new theta there in the same pass that computes it (4 more bytes written per element
 * and replica, nothing more read).  A replica may be memory of ANOTHER GPU that this GPU can address (a peer
 * mapping; the caller obtains it): the kernel only ever stores to a replica, so the data crosses NVLink once, as
 * remote writes, while the update runs.  With one shard per GPU and, on every GPU, a full-length buffer into
 * whose range [lo_g, hi_g) shard g writes, a learner's weight pull is a read of its own GPU's buffer: the
 * all-gather has already happened, tile by tile, inside the update kernels.  The caller orders a learner's read
 * after the update (ps_synchronize on the owning servers, then its own cross-GPU barrier).
 * replicas_dev: HOST array of `count` device pointers, copied; 4-byte aligned (16 keeps the vector kernel);
 * must not overlap theta, v, the bf16 mirror or one another.  count = 0 unbinds.  Only while no complete group is pending. */
int ps_bind_weight_replicas(ps_t *ps, int count, float *const *replicas_dev);

/* Binds `num_slots` caller-owned device slots of `slot_bytes` each (a multiple of 16, at least
 * num_params * gradient size; base 16-byte aligned) that ps_push_gradient_host copies into. */
int ps_bind_staging(ps_t *ps, void *slots_dev, int64_t slot_bytes, int num_slots);

/* Sets / reads one ps_option (the paper fixes none of them; they configure this implementation).
 * Unknown keys, values out of range and changes that are only allowed while no gradient is pending
 * return PS_ERR_INVALID_ARG and change nothing. */
int ps_set_option(ps_t *ps, int key, int64_t value);
int ps_get_option(ps_t *ps, int key, int64_t *value);

/* Learning-rate schedule (Section 4.3 lowers alpha0 in steps during training): sets the base rate for
 * gradients pushed from now on.  Gradients already pushed keep the rate that was in force when they
 * arrived (the rate of Section 2.4, Eq. 3 is fixed per gradient as it comes in). */
int ps_set_alpha0(ps_t *ps, float alpha0);

/* Base rho of the exponential staleness penalty, alpha = alpha0 * rho^tau, used by PS_MOD_EXP_STALENESS
 * (Section 1 discusses that rule as the earlier proposal and gives no formula; this form gives a fresh
 * gradient, tau = 0, the full alpha0).  0 < rho <= 1, default 0.5; rho = 1 is the constant rate.  Only
 * while no gradient is pending. */
int ps_set_penalty_base(ps_t *ps, float rho);

/* Per-layer multipliers.  The small network of Section 4.1 follows a Caffe model, in which every layer
 * carries a learning-rate and a weight-decay multiplier (commonly 2 and 0 for biases).  Layer q covers
 * elements [bounds_host[q], bounds_host[q+1]) with bounds_host[0] = 0, bounds_host[num_layers] = num_params,
 * ascending; its elements are updated with
 *     v = momentum * v + lr_mult[q] * (acc + (wd_mult[q] * d) * theta)
 * (each product and sum rounded once), i.e. rate alpha * lr_mult[q] and decay weight_decay * wd_mult[q].
 * Multipliers of 1 give exactly the bits of a server without a table.  num_layers = 0 removes the table;
 * at most PS_MAX_LAYERS.  The three arrays are host memory and are copied.  Only while no gradient is
 * pending. */
int ps_set_layer_multipliers(ps_t *ps, int num_layers, const int64_t *bounds_host,
                             const float *lr_mult_host, const float *wd_mult_host);

/* pullWeights (Section 2.1): *ts receives the server timestamp i a gradient computed on these
 * weights must carry.  If out_dev != NULL, every complete pending group is applied first and
 * theta_i (num_params fp32) is copied to out_dev on the stream, so the weights always belong to
 * the returned timestamp.  out_dev == NULL returns the timestamp only. */
int ps_pull_weights(ps_t *ps, float *out_dev, int64_t *ts);

/* pullWeights for bf16 learners: like ps_pull_weights with out_dev != NULL, but copies the bf16 mirror
 * (num_params * 2 bytes).  Needs ps_bind_weight_mirror. */
int ps_pull_weights_bf16(ps_t *ps, void *out_bf16_dev, int64_t *ts);

/* Same, into host memory; returns after the copy has completed. */
int ps_pull_weights_host(ps_t *ps, float *out_host, int64_t *ts);

/* Same, but returns as soon as the copy is enqueued on a second, library-owned stream, so that it
 * overlaps host-to-device gradient copies issued afterwards (full-duplex PCIe).  The copy waits for
 * the updates enqueued so far; later updates wait for the copy before they overwrite theta.
 * out_host should be pinned memory and must not be read before ps_synchronize (or a later
 * ps_pull_weights_host) has returned.  The paper's learners block in pullWeights (Section 2.3);
 * this is the non-blocking form of the same call. */
int ps_pull_weights_host_async(ps_t *ps, float *out_host, int64_t *ts);

/* pushGradient + the bookkeeping half of sumGradients (Section 2.1, 2.2).  grad_dev: num_params
 * values of the configured dtype, BORROWED: it must stay valid and unchanged until the
 * ps_apply_update that consumes it has finished on the stream.  ts: the timestamp the learner
 * pulled.  Staleness tau = i - ts is taken against the server timestamp i at this call (the
 * number of complete groups so far).  Returns PS_READY if the gradient completed a group of c,
 * else PS_OK. */
int ps_push_gradient(ps_t *ps, int learner, const void *grad_dev, int64_t ts);

/* Same for a gradient in host memory: it is copied (cudaMemcpyAsync on the stream) into a free
 * staging slot, which is released when the update that consumes it has been enqueued.  The host
 * buffer may be reused when the call returns only if it is pageable; pinned buffers must stay
 * unchanged until the stream has passed the copy. */
int ps_push_gradient_host(ps_t *ps, int learner, const void *grad_host, int64_t ts);

/* Receive buffers for learners on the same GPU (the counterpart of the server-side receive buffer of the
 * paper's MPI transport, Section 2.3): ps_acquire_slot lends one free staging slot (bound with
 * ps_bind_staging); the learner writes its gradient there with its own kernels or copies and hands it over
 * with ps_push_slot, which behaves like ps_push_gradient and returns the slot to the pool once the update
 * that consumes it is enqueued.  A slot that will not be pushed goes back with ps_release_slot.
 * PS_ERR_QUEUE_FULL when every slot is in use.
 *
 * Two orderings are the learner's to keep, because a recycled slot may still be read by the update kernel
 * that consumed its previous gradient, and the next update must not start before the new gradient is there:
 *   (1) the write into the slot comes AFTER the slot's previous consumer: true for work enqueued on the
 *       server's stream; a learner writing on another stream first calls ps_slot_wait(ps, id, its stream);
 *   (2) the write comes BEFORE the update that consumes it: true for work enqueued on the server's stream
 *       before ps_apply_update; a learner writing on another stream calls ps_slot_written(ps, id, its
 *       stream) after enqueuing the write and before ps_push_slot, which makes the server's stream wait.
 * A launch that consumes a gradient pushed with ps_push_slot is never started early by
 * PS_OPT_OVERLAP_LAUNCH (its producer may be the kernel directly before it). */
int ps_acquire_slot(ps_t *ps, void **slot_dev, int *slot_id);
int ps_push_slot(ps_t *ps, int learner, int slot_id, int64_t ts);
int ps_release_slot(ps_t *ps, int slot_id);
/* stream: a cudaStream_t.  Both need a slot currently lent by ps_acquire_slot. */
int ps_slot_wait(ps_t *ps, int slot_id, void *stream);      /* `stream` waits until the slot's last consumer has finished */
int ps_slot_written(ps_t *ps, int slot_id, void *stream);   /* the server's stream waits for what `stream` holds so far */

/* applyUpdate fused with sumGradients (Section 2.1; Eq. 2 with the learning rate of Eq. 3):
 * takes up to PS_OPT_FUSE_T complete groups, oldest first, and applies them in ONE kernel pass
 * that reads theta and v once, reads every gradient of those groups once, and writes theta and
 * v once.  Per element and per group, in fp32 with separately rounded multiplies and adds:
 *     acc = s_1 g_1 + s_2 g_2 + ... + s_c g_c     (ascending learner id, then push index)
 *     v   = momentum * v + (acc + d * theta)
 *     theta = theta - v
 * with s_l = alpha0 / (c * sigma_l), alpha0 as it was when gradient l was pushed, and
 * d = weight_decay * sum_l s_l.  Advances the applied
 * timestamp by the number of groups and appends to the log.  Returns that number (>= 1) or
 * PS_ERR_NOT_READY. */
int ps_apply_update(ps_t *ps);

/* Applies every complete pending group (repeated ps_apply_update: Section 2.1's applyUpdate for each group
 * of Eq. 2 that is waiting).  Returns the number applied (>= 0). */
int ps_flush(ps_t *ps);

/* Blocks until everything this handle enqueued (main stream and read-back stream) has finished.
 * Returns PS_ERR_DEVICE_WAIT if an update kernel has given up on a bounded wait since ps_init_weights. */
int ps_synchronize(ps_t *ps);

/* Waits for the stream, then reports the status record of the bulk-copy kernel: *code 0 = no wait has run
 * out; else 1, with the block, the block's tile counter and the stage whose copy barrier did not complete.
 * Any output pointer may be NULL. */
int ps_kernel_status(ps_t *ps, int *code, int *block, int64_t *tile, int *stage);

/* The server's record of what Section 2.1 defines per gradient (its timestamp j, the server timestamp i it
 * met, the staleness i - j: the quantity whose distribution Fig. 1 shows) and of Eq. 2-3 (group membership,
 * summation order, scale).  Copies the entries of updates [first_update, first_update + count) to out_host
 * (count * c entries, update-major, in summation order). */
int ps_get_update_log(ps_t *ps, int64_t first_update, int64_t count, ps_log_entry *out_host);

/* Device pointers of the bound state and both readings of the timestamp of Section 2.1: ts_applied
 * counts updates whose kernel has been enqueued; ts_logical = ts_applied + complete pending groups (what
 * ps_pull_weights returns: a complete group has already advanced the clock the learners see, whether or
 * not its kernel has been launched).  Any output pointer may be NULL. */
int ps_peek_state(ps_t *ps, const float **w_dev, const float **v_dev,
                  int64_t *ts_applied, int64_t *ts_logical);

/* Checkpoint of the protocol state (the paper describes none; long trainings need one): timestamp,
 * current alpha0 and every learner's push count, as PS_STATE_WORDS(lambda) 64-bit words in host memory.
 * Theta and v are the caller's buffers and are saved by the caller.  Pending gradients are borrowed
 * device buffers and cannot be saved: both calls return PS_ERR_NOT_READY unless no gradient is waiting
 * (checkpoint on a group boundary, after ps_flush).  ps_export_state returns the number of words written;
 * ps_import_state needs a handle created with the same num_params, lambda and n, restarts the log at the
 * imported timestamp, and leaves theta and v alone. */
#define PS_STATE_WORDS(lambda) (8 + (lambda))
int ps_export_state(ps_t *ps, int64_t *out_host, int64_t capacity_words);
int ps_import_state(ps_t *ps, const int64_t *in_host, int64_t words);

/* With PS_OPT_TIMING = 1: waits for the stream, then returns the summed CUDA-event duration of the
 * update kernels launched since the last call and their number.  Either pointer may be NULL. */
int ps_kernel_time(ps_t *ps, double *total_ms, int64_t *launches);

/* cudaError_t of the most recent failed CUDA call made for this handle (0 if none). */
int ps_last_cuda_error(ps_t *ps);

const char *ps_status_string(int status);

/* One fused update without any allocation.  The paper has no counterpart: this entry point exists for
 * callers that must not allocate while they run.  Examples: a learner framework whose caching allocator owns
 * all device memory, so that a cudaMalloc or cudaHostAlloc made behind its back can fail or fragment its
 * pool; a training loop whose steady state has to stay free of calls that synchronise the device, which
 * allocation calls do; code that runs where allocation is not permitted at all.  The ordinary path cannot
 * promise that: ps_create allocates host memory, and the first PS_KERNEL_BULK launch of a handle calls
 * cudaHostAlloc for the status record its kernel reports through.
 *
 * What it does: one weight update (Eq. 2 with momentum and decay, the arithmetic of ps_apply_update for one
 * group) by the shared-memory staged kernel of PS_KERNEL_BULK, with no handle and no protocol state:
 *     acc = scales[0] g_0 + ... + scales[c-1] g_{c-1};  v = momentum * v + (acc + decay * theta);  theta -= v
 * w_dev, v_dev: num_params fp32 each, device memory, read and written.  grads_dev: HOST array of c DEVICE
 * pointers to num_params values of grad_dtype (ps_grad_dtype) each, read only.  scales_host: HOST array of c
 * fp32 scales (the caller applies Eq. 3 and the 1/c of Eq. 2 itself).  Every device pointer must be 16-byte
 * aligned and belong to the current device.  The caller owns every buffer; nothing is kept after the call.
 * blocks: 0 lets the library choose (as many as fit the SMs, fewer for short vectors); a positive value caps the grid,
 * for a server that shares its GPU with learners' kernels.  stream: a cudaStream_t; the work is enqueued
 * there and the call returns at once unless blocks_gave_up != NULL.
 *
 * Scratch memory: the kernel reports a copy wait that ran out in a status record, one per block.  Here the
 * records are a fixed array of PS_STATIC_MAX_BLOCKS entries (16 KiB) in the library's static device memory,
 * which every GPU that loads the library holds until the process exits.  A launch that would need more
 * blocks, or c > PS_STATIC_MAX_GRADS, is refused with PS_ERR_STATIC_LIMIT and does nothing.  All calls on
 * one device share the array and it keeps the previous call's contents: every call clears the records it
 * is about to use (a memset enqueued on `stream` before the kernel), so calls whose device work overlaps,
 * on different streams or from different threads, race on the records and must be serialised by the caller.
 *
 * blocks_gave_up != NULL: the call waits for `stream`, reads the records back and stores how many blocks
 * gave up (0: the update is complete; otherwise theta and v are partly updated).  NULL: nothing is read.
 *
 * The first call on each device looks the array's device address up and raises the kernel's shared-memory
 * limit; make that first call outside any stream capture.  No call of this function uses cudaMalloc,
 * cudaFree, cudaHostAlloc or any other allocating routine.
 * Returns PS_OK, PS_ERR_INVALID_ARG, PS_ERR_STATIC_LIMIT or PS_ERR_CUDA. */
#define PS_STATIC_MAX_BLOCKS 1024
#define PS_STATIC_MAX_GRADS 16
int ps_fused_update_static(float *w_dev, float *v_dev, int64_t num_params,
                           const void *const *grads_dev, const float *scales_host, int c,
                           float decay, float momentum, int grad_dtype,
                           int blocks, void *stream, int *blocks_gave_up);

#ifdef __cplusplus
}
#endif
#endif /* SOFTSYNC_PS_H */
