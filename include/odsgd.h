/*
 * odsgd.h - C ABI of the OD-SGD parameter-update library for NVIDIA B200 (sm_100a).
 *
 * The library runs the per-iteration parameter-update pass of One-step Delay SGD
 * (OD-SGD) and of the two rules the paper compares it with (SSGD, ASGD) as fused
 * one-pass CUDA kernels over a flat fp32 parameter arena:
 *
 *   - the GLOBAL update, the parameter-server role (paper: Algorithm 1, "Update w_t
 *     with aggregated gradient" once all M workers have delivered):
 *         gbar = (g_0 + g_1 + ... + g_{M-1}) * (1/M)     workers added in this order
 *         d    = gbar + wd * w
 *         v'   = momentum * v - lr * d
 *         w'   = w + v'
 *   - the LOCAL update, the worker role (paper: Algorithm 2, repeat-loop, "w_bak = w_t"
 *     then "Update w_bak with g_m"; Section 3.3 "Local Updater"):
 *         x_m  = w_bak - local_lr * g_m
 *     where w_bak is the global weight vector from BEFORE this iteration's global
 *     update (the worker has not pulled the new one yet); x_m are the weights worker
 *     m trains on next.  Delay-compensated flavours: Eq. 4 and Eq. 5/6.
 *   - the SSGD server step (Section 3.1: the server side is the same as OD-SGD's) and
 *     the ASGD server step (Section 1: each arriving gradient is applied at once).
 *
 * Conventions
 *   - Every function returns an int: ODSGD_OK (0) or a negative ODSGD_ERR_* code.
 *     Nothing throws across this boundary.  odsgd_last_error() gives a text for the
 *     most recent failure on a context.
 *   - "device pointer" = address in the memory of the CUDA device that was current
 *     when odsgd_create() ran; "host pointer" = ordinary process memory.
 *   - The caller owns every device buffer for the whole life of the context; the
 *     context only borrows them.  The library allocates no parameter-sized memory.
 *   - All update calls are asynchronous: they enqueue work on `stream` (a
 *     cudaStream_t passed as void*; NULL = the legacy default stream) and return.
 *     The library never synchronises.  Buffers must stay valid until that work is done.
 *   - Arena layout: all parameter tensors concatenated into one float array of
 *     `n_params` elements; `tensor_offsets` (n_tensors + 1 ascending element offsets,
 *     first 0, last n_params) marks where each tensor starts.  Gradient arenas, the
 *     momentum arena and the local-weight arenas use the same layout.  Padding
 *     elements between tensors are updated like any other element (zeros stay zeros).
 *   - Alignment: the fast path needs every device pointer 16-byte aligned.  Without
 *     ODSGD_FLAG_ALLOW_UNALIGNED a misaligned pointer is rejected with ODSGD_ERR_ALIGN;
 *     with it, a scalar (4-byte) kernel is used for that call.
 *   - Arithmetic is IEEE-754 binary32, round-to-nearest-even, subnormals kept.  By
 *     default every operator written above rounds on its own, so results are
 *     reproducible bit for bit against a plain scalar CPU evaluation in the same order
 *     (the kernels are bound by memory bandwidth, so this costs no time).  With
 *     ODSGD_FLAG_ALLOW_FMA the compiler may fuse a multiply with the following add (one
 *     rounding instead of two); results then differ from the default in the last bits.
 */
#ifndef ODSGD_H_
#define ODSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ODSGD_VERSION_MAJOR 0
#define ODSGD_VERSION_MINOR 1

/* Largest number of workers (gradient buffers) one context can take. */
#define ODSGD_MAX_WORKERS 64

#define ODSGD_OK 0
#define ODSGD_ERR_ARG (-1)         /* NULL where a pointer is needed, size or index out of range */
#define ODSGD_ERR_ALIGN (-2)       /* a device pointer is not 16-byte aligned (4-byte for the scalar path) */
#define ODSGD_ERR_OVERLAP (-3)     /* two buffers that must be distinct overlap */
#define ODSGD_ERR_STATE (-4)       /* call not valid in the context's current state */
#define ODSGD_ERR_CUDA (-5)        /* a CUDA runtime call or the launch failed; text in odsgd_last_error */
#define ODSGD_ERR_UNSUPPORTED (-6) /* valid request this build does not implement */

#define ODSGD_FLAG_DETERMINISTIC 0x1u   /* one rounding per operator; this is the default, the bit only states it */
#define ODSGD_FLAG_ALLOW_UNALIGNED 0x2u /* accept 4-byte aligned pointers (slower scalar kernel) */
#define ODSGD_FLAG_ALLOW_FMA 0x4u       /* let multiply-add pairs fuse (excludes ODSGD_FLAG_DETERMINISTIC) */
#define ODSGD_FLAG_WORKER_ONLY 0x8u     /* worker-role context: v may be NULL; only odsgd_worker_local_update runs */

/* Largest number of weight mirrors per weight arena (odsgd_set_weight_mirrors). */
#define ODSGD_MAX_MIRRORS 15

/* Gradient tables one context can keep bound at a time (odsgd_bind_grads). */
#define ODSGD_MAX_BINDINGS 16

/* Local update rules (Section 3.3, "Local Updater"). */
#define ODSGD_LOCAL_SGD 0  /* x = w_bak - local_lr * g */
#define ODSGD_LOCAL_DC_C 1 /* Eq. 4 */
#define ODSGD_LOCAL_DC_A 2 /* Eq. 5 with the running mean square of Eq. 6 */
#define ODSGD_LOCAL_MOMENTUM 3 /* the server's own rule run by the worker: SGD with momentum (and decay) */

typedef struct odsgd_ctx odsgd_ctx;

/*
 * Description of one training job's parameter state.  Plain data, copied by
 * odsgd_create(); the arrays it points to (local, tensor_offsets) are host arrays
 * read during the call only.
 *
 * Weight storage, two layouts:
 *   ping-pong  (w_b != NULL): each global update reads the current half and writes
 *              the other one, then the halves swap roles.  The half just read still
 *              holds the old weights, which are exactly the w_bak the workers need,
 *              so keeping them costs no extra traffic.  w_delayed must be NULL.
 *   in place   (w_b == NULL): the global update overwrites w_a.  If w_delayed != NULL
 *              the old weights are also written there (one extra store stream) so
 *              that odsgd_local_update() can run later; if it is NULL only the fused
 *              call can produce local weights.
 */
typedef struct odsgd_desc {
    float* w_a;                   /* device, n_params floats: global weights w_0 at create time */
    float* w_b;                   /* device, n_params floats, or NULL */
    float* w_delayed;             /* device, n_params floats, or NULL (in-place layout only) */
    float* v;                     /* device, n_params floats: momentum state (caller zero-fills for a fresh run);
                                     may be NULL only with ODSGD_FLAG_WORKER_ONLY */
    float* const* local;          /* host array of n_workers device pointers (entries may be NULL), or NULL */
    size_t n_params;              /* elements in each arena, > 0 */
    const size_t* tensor_offsets; /* host, n_tensors + 1 ascending offsets, [0] = 0, [n_tensors] = n_params */
    size_t n_tensors;             /* >= 1 */
    int n_workers;                /* M, 1 .. ODSGD_MAX_WORKERS */
    float lr;                     /* global learning rate */
    float local_lr;               /* local learning rate */
    float momentum;
    float wd;                     /* weight decay (L2 coefficient) */
    uint32_t flags;               /* ODSGD_FLAG_* */
} odsgd_desc;

/* Library version as major * 1000 + minor. */
int odsgd_version(void);

/* Text for an ODSGD_ERR_* code (static storage). */
const char* odsgd_strerror(int code);

/*
 * Validates `desc` and builds a context on the current CUDA device.  No kernel is
 * launched and nothing is written to the caller's buffers.
 * Errors: ERR_ARG (NULL/zero/out-of-range field, offsets not ascending or not ending
 * at n_params, w_delayed given together with w_b), ERR_ALIGN, ERR_OVERLAP (any two of
 * w_a, w_b, w_delayed, v, local[m] overlap), ERR_CUDA (no usable device).
 * On error *out is set to NULL; odsgd_last_error(NULL) describes the failure.
 */
int odsgd_create(odsgd_ctx** out, const odsgd_desc* desc);

/* Frees the context (host memory and its small device tables).  Caller buffers are untouched. */
int odsgd_destroy(odsgd_ctx* ctx);

/*
 * Global update (Algorithm 1).  `worker_grads` is a HOST array of n_workers DEVICE
 * pointers, each an arena of n_params floats; they are read only and summed in index
 * order.  Advances the step counter; in the ping-pong layout swaps the halves.  The
 * gradient pointers are remembered as "this iteration's gradients" so that
 * odsgd_local_update() can follow.
 * Errors: ERR_ARG (NULL table or entry), ERR_ALIGN, ERR_OVERLAP (a gradient buffer
 * overlaps a state buffer), ERR_CUDA.
 */
int odsgd_global_update(odsgd_ctx* ctx, const float* const* worker_grads, void* stream);

/*
 * Local update of worker `worker_id` (Algorithm 2, "Update w_bak with g_m"):
 * local[worker_id] = w_bak (-) local_lr * g_worker_id, with w_bak the weights from
 * before the latest odsgd_global_update() and g the gradient bound by that call
 * (the gradient buffer must still hold the same data).
 * Errors: ERR_STATE (no global update since create or since the last SSGD/ASGD step,
 * or in-place layout without w_delayed), ERR_ARG (worker_id out of range, or no local
 * buffer for that worker).
 */
int odsgd_local_update(odsgd_ctx* ctx, int worker_id, void* stream);

/*
 * Fused global + local update: the global update and the local update of one worker
 * (worker_id >= 0) or of every worker that has a local buffer (worker_id == -1) in a
 * single pass; the weights and each gradient are read once.  Results are bit-identical
 * to odsgd_global_update() followed by odsgd_local_update().  Same state effects and
 * errors as those two calls.
 */
int odsgd_fused_update(odsgd_ctx* ctx, const float* const* worker_grads, int worker_id, void* stream);

/*
 * Same as odsgd_fused_update() for gradients that arrive in HOST memory (as they do at
 * a parameter server fed by a network).  `host_grads`: host array of n_workers host
 * pointers (page-locked memory for real asynchrony), n_params floats each.
 * `dev_staging`: host array of n_workers device pointers the gradients are copied
 * into (caller-owned, n_params floats each).  If `host_local_out` is not NULL and
 * worker_id >= 0, local[worker_id] is copied back to it after the update.  The uploads and
 * the kernel are enqueued on `stream` in order; nothing is synchronised.
 * `copy_stream`: NULL (or equal to `stream`) puts the copy-back on `stream` too.  A different
 * stream makes the copy-back run there, ordered after the kernel by an event, so that it
 * overlaps the NEXT call's uploads (the bus is full duplex); the next call's kernel waits for
 * that copy before it overwrites local[worker_id].  The caller synchronises `copy_stream`
 * before reading `host_local_out`.  (The context creates two CUDA events on first use of a
 * separate copy stream.)  Every check that can refuse the call runs before the first copy is
 * enqueued, so a failed call leaves `dev_staging` untouched; and every later kernel this
 * context launches that may write a local arena, on whatever stream, first waits for a
 * copy-back that is still pending.
 */
int odsgd_fused_update_host(odsgd_ctx* ctx, const float* const* host_grads, float* const* dev_staging,
                            int worker_id, float* host_local_out, void* stream, void* copy_stream);

/*
 * SSGD server step (Section 3.1): the same arithmetic as the global update, applied
 * in place to the current weights; no backup weights are kept and no local update may
 * follow (workers pull the new weights instead).
 */
int odsgd_ssgd_step(odsgd_ctx* ctx, const float* const* worker_grads, void* stream);

/*
 * ASGD server step (Section 1): one worker's gradient `grad` (device pointer) is
 * applied at once, without sum or 1/M: d = g + wd*w; v' = momentum*v - lr*d; w' = w + v'.
 * In place on the current weights.  `worker_id` (0 .. n_workers-1) is recorded only;
 * the order of application is the order of the calls.
 */
int odsgd_asgd_step(odsgd_ctx* ctx, int worker_id, const float* grad, void* stream);

/*
 * The same three server calls on a gradient table that was checked once.  A training loop
 * hands the library the same M gradient buffers every iteration; odsgd_bind_grads() validates
 * such a table (NULL entries, overlap with every state buffer, alignment) and keeps a copy of
 * its pointers in one of ODSGD_MAX_BINDINGS slots of the context, and the *_bound calls then
 * skip that validation: their per-call host work is filling the kernel's argument block and the
 * launch.  (Algorithm 1 and Algorithm 2 run once per iteration on the same buffers; on small
 * parameter sets the host side of a call, not the kernel, is what bounds the iteration rate.)
 * Results are bit-identical to the unbound calls.
 *   odsgd_bind_grads    worker_grads as in odsgd_global_update; *slot receives the slot index.
 *                       Errors: ERR_ARG, ERR_OVERLAP, ERR_ALIGN as that call would report them,
 *                       ERR_UNSUPPORTED when all slots are taken; *slot is then -1.
 *   odsgd_unbind_grads  frees a slot.
 *   *_bound             ERR_ARG for a slot that holds no table; ERR_STATE when the context's set
 *                       of state buffers changed after the bind (odsgd_set_local_rule,
 *                       odsgd_set_server_mean_square): the table must be bound again, which
 *                       repeats the overlap check against the new buffers.  Otherwise the errors
 *                       of the unbound call.
 * The bound buffers must stay valid, and must keep not overlapping the state, for as long as the
 * slot is used; the library cannot see a buffer being freed and reallocated elsewhere.
 */
int odsgd_bind_grads(odsgd_ctx* ctx, const float* const* worker_grads, int* slot);
int odsgd_unbind_grads(odsgd_ctx* ctx, int slot);
int odsgd_global_update_bound(odsgd_ctx* ctx, int slot, void* stream);
int odsgd_fused_update_bound(odsgd_ctx* ctx, int slot, int worker_id, void* stream);
int odsgd_ssgd_step_bound(odsgd_ctx* ctx, int slot, void* stream);

/*
 * The worker's half of an iteration when the server's half runs elsewhere (Algorithm 2,
 * repeat-loop: "w_bak = w_t", then "Update w_bak with g_m", while the gradient is on its way to
 * the server; Section 3.1: push and local update overlap because both only read the gradient).
 * Applies the context's local rule to explicit inputs:
 *     local[worker_id] = LocalRule(w_bak, grad)        (x = w_bak - local_lr * grad by default)
 * `w_bak`: device, n_params floats, the global weights this worker pulled last; it may be one of
 * the context's own weight arenas (w_a / w_b), but not an arena the call writes.  `grad`: device,
 * n_params floats, this worker's gradient, outside every state buffer.  `no_delay` != 0 says
 * that `grad` was computed on `w_bak` itself (the last warm-up iteration of Algorithm 2), so the
 * delay-compensated rules of Eq. 4 / Eq. 5 see a zero delay; it is ignored by the other rules.
 * Works in any context; a context created with ODSGD_FLAG_WORKER_ONLY (no momentum arena) can
 * run nothing else: its server calls fail with ERR_STATE.  Does not touch the step counter or
 * the weights.
 * Errors: ERR_ARG, ERR_OVERLAP, ERR_ALIGN, ERR_STATE (rule needs a state arena the worker lacks).
 */
int odsgd_worker_local_update(odsgd_ctx* ctx, int worker_id, const float* w_bak, const float* grad,
                              int no_delay, void* stream);

/*
 * Which slice of the arena rank `rank` of `n_ranks` owns when the server role is spread over
 * several GPUs (Section 2.2: gradients are reduced, pushed to the server and the new weights
 * pulled back; every element is updated independently, so the server's work shards by index).
 * All slices have the same nominal length, ceil(n_params / n_ranks) rounded up to 4 elements
 * (16 bytes, so every slice start keeps the arena's alignment); slice r is
 * [r * len, min((r + 1) * len, n_params)).  The slices are disjoint, ascending and cover
 * [0, n_params) exactly; the last non-empty one may be short, and with more ranks than
 * 4-element groups the trailing ranks get empty slices (begin == end == n_params).
 * Host arithmetic only.  Errors: ERR_ARG (NULL output, n_ranks < 1, rank out of range).
 */
int odsgd_shard_range(size_t n_params, int n_ranks, int rank, size_t* begin, size_t* end);

/*
 * Weight mirrors: further device buffers that receive every weight the server pass writes, by
 * the kernel's own stores.  With the server role spread over R GPUs (odsgd_shard_range), each
 * rank updates the slice it owns, and every rank needs the whole new vector before its workers
 * can use it: Section 2.2's pull (Fig. 3), which Section 3.1 overlaps with the next iteration.
 * A context over the owned slice whose mirrors are that same slice inside the other R - 1 ranks'
 * replicas (their memory mapped into this process: CUDA IPC or symmetric memory, with peer
 * access enabled) delivers the new weights while it computes them; no all-gather follows the
 * kernel.  The same holds on the read side without any call: entries of `worker_grads` may be
 * peer-mapped memory of another GPU, so that the push needs no staging copy.  The kernels touch
 * all of these with ordinary 128-bit loads and stores only (no bulk-copy engine, no multicast).
 *   mirrors_a, mirrors_b  HOST arrays of n_mirrors DEVICE pointers, n_params floats each:
 *                         mirrors_a[i] shadows w_a, mirrors_b[i] shadows w_b (ping-pong layout:
 *                         both tables; in-place layout: mirrors_b must be NULL).  A call that
 *                         writes weight half h also writes h's mirrors, same offsets, same bits.
 *   n_mirrors             0 .. ODSGD_MAX_MIRRORS; 0 switches the feature off (tables ignored).
 * While mirrors are set only odsgd_global_update / odsgd_ssgd_step and their *_bound forms run
 * (they carry no local update; workers use odsgd_worker_local_update on their own replica); the
 * fused, scheduled, ASGD and DC-ASGD calls fail with ERR_STATE because they would leave the
 * mirrors stale.  The library never reads a mirror and does not initialise it: the caller fills
 * each with w_0.  Mirrors count as state buffers: they must not overlap one another, the
 * context's arenas or a gradient buffer (ERR_OVERLAP, here or in the update call), and setting
 * them invalidates bound gradient tables like any other change of the state buffers.  Ordering
 * between GPUs is the caller's: the peers' gradients must be complete before the call's kernel
 * starts, and a peer may read its replica only after that kernel has finished (for instance a
 * stream-ordered collective on either side).  The library cannot tell a peer-mapped address
 * from a local one and cannot check that peer access is enabled.
 * Errors: ERR_ARG (NULL table or entry, count out of range, mirrors_b against the layout),
 * ERR_ALIGN, ERR_OVERLAP, ERR_STATE (worker-only context).
 */
int odsgd_set_weight_mirrors(odsgd_ctx* ctx, float* const* mirrors_a, float* const* mirrors_b, int n_mirrors);

/*
 * Hyper-parameters are kernel arguments, never compiled in: the paper's runs change the
 * learning rates during training (Section 4: division by 10 at fixed epochs, the linear ramp
 * from 0.1 to 0.8 over the first epochs, polynomial decay; global and local rates are chosen
 * separately, Section 4.2), so a setter may be called before any update call and takes effect
 * from the next launch on.  Momentum and weight decay are the server rule's (Section 4.1:
 * momentum 0.9 for SSGD and OD-SGD, 0 for ASGD).
 */
int odsgd_set_lr(odsgd_ctx* ctx, float lr);
int odsgd_set_local_lr(odsgd_ctx* ctx, float local_lr);
int odsgd_set_momentum(odsgd_ctx* ctx, float momentum);
int odsgd_set_wd(odsgd_ctx* ctx, float wd);

/*
 * Chooses the local update rule (Section 3.3).  ODSGD_LOCAL_SGD ignores the other
 * arguments.  ODSGD_LOCAL_DC_C uses `lambda` (Eq. 4).  ODSGD_LOCAL_DC_A uses `lambda`,
 * the mean-square decay `m` and `eps` (Eq. 5, Eq. 6); a local update under this rule needs
 * one mean-square arena for the worker it updates: `mean_square` is a host array of
 * n_workers device pointers (n_params floats each, caller-owned and caller-initialised,
 * normally zeros; entries may be NULL for workers that are never updated locally, and the
 * whole table may be NULL when the rule is only used by odsgd_dcasgd_step); pass NULL for
 * the other rules.  A local update of a worker without its arena fails with ERR_STATE.
 * ODSGD_LOCAL_MOMENTUM (Section 4.1's MNIST run: local SGD with the server's learning rate and
 * momentum) applies the global update's rule to the worker's backup weights, its own gradient
 * and its own velocity:  d = g + lambda * w_bak;  u <- m * u - local_lr * d;  x = w_bak + u,
 * with `m` the local momentum, `lambda` the local weight decay, `eps` unused, and
 * `mean_square` holding the per-worker velocity arenas u (same rules as above, zero-filled
 * for a fresh run).  In both delay-compensated rules the vector the
 * gradient was computed on (the paper's w_t) is the worker's previous local weights,
 * i.e. the content of local[worker] before the call, which is then overwritten.
 */
int odsgd_set_local_rule(odsgd_ctx* ctx, int rule, float lambda, float m, float eps,
                         float* const* mean_square);

/*
 * Per-tensor multipliers of the stock updater the paper relies on (Section 3.3: the global
 * updater is the framework's own): tensor t is updated with lr * lr_mult[t] and
 * wd * wd_mult[t] (each product rounded once), e.g. wd_mult = 0 for biases and batch-norm
 * scales.  `lr_mult`, `wd_mult`: HOST arrays of n_tensors floats; NULL means all ones; both
 * NULL switches the feature off.  The library keeps a small device table (offsets and the two
 * multiplier arrays, 16 bytes per tensor), allocated by this call with cudaMalloc and filled by
 * a copy enqueued on `stream`; it is freed by odsgd_destroy or when the feature is switched
 * off.  Applies to the global, fused and SSGD calls; the ASGD and local rules are unaffected.
 * The 128-bit kernels need every tensor offset to be a multiple of 4 elements; otherwise the
 * call fails with ERR_ALIGN unless ODSGD_FLAG_ALLOW_UNALIGNED is set (scalar kernel).
 * Call it outside stream capture (ERR_STATE while `stream` is capturing: the call may allocate, and
 * a captured upload would re-read the host copy of the table at every replay); update calls that
 * use the table can be captured afterwards.
 * Errors: ERR_CUDA (allocation or copy failed), ERR_ALIGN, ERR_STATE (wrong current device, capture).
 */
int odsgd_set_tensor_multipliers(odsgd_ctx* ctx, const float* lr_mult, const float* wd_mult, void* stream);

/*
 * Fused global + local update with per-tensor multipliers that never allocates.  (The paper
 * has no counterpart to this call; it exists for deployment reasons only.)
 *
 * odsgd_set_tensor_multipliers() has to cudaMalloc a small device table.  Some callers must
 * not do that: a server loop that runs beside training streams cannot afford cudaMalloc's
 * device-wide synchronisation, and a process that has handed all device memory to its
 * framework's pool may simply be refused.  For them this call does the same work as
 * odsgd_set_tensor_multipliers(ctx, lr_mult, wd_mult, stream) followed by
 * odsgd_fused_update(ctx, worker_grads, worker_id, stream), bit for bit, but keeps the table
 * in a fixed array that is part of the library image: ODSGD_STATIC_TABLE_BYTES of device
 * memory on every GPU that loads the library, held until the process exits.  It calls no
 * cudaMalloc, no cudaFree and no allocating library routine, and does not touch the table of
 * odsgd_set_tensor_multipliers() (which may be on or off; it is ignored here).
 *
 *   lr_mult, wd_mult  HOST arrays of n_tensors floats (NULL = all ones), read during the call
 *   worker_id         0 .. n_workers-1, a worker that has a local buffer
 *
 * Limits: at most ODSGD_STATIC_MAX_TENSORS tensors (more: ERR_UNSUPPORTED, nothing is
 * launched); local rule ODSGD_LOCAL_SGD only (else ERR_UNSUPPORTED); tensor offsets must be
 * multiples of 4 elements unless ODSGD_FLAG_ALLOW_UNALIGNED is set (ERR_ALIGN).
 * Set-up: the first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) with that device current.  The call cannot be recorded into a stream
 * capture: while `stream` is capturing it fails with ERR_STATE and enqueues nothing (a captured
 * upload would re-read, at every replay, whatever table the last eager call left behind).
 * Sharing: every call on a device, from every context, writes the same array, and
 * the array keeps the last call's table.  Each call rewrites all entries it uses before its
 * kernel reads them, in stream order, so calls on ONE stream are safe back to back; calls
 * whose work overlaps on the GPU (different streams, different threads) race on the array
 * and must be serialised by the caller.  On the host the table is staged in one pageable array
 * shared by the whole process; the call holds a process-wide lock while it fills and uploads
 * it, so host threads may call concurrently (also for different devices), at the price of
 * running one at a time.  The upload is an ordinary copy from pageable memory: for a large
 * table it may make the call wait for work enqueued earlier on `stream`.
 */
#define ODSGD_STATIC_MAX_TENSORS 4096
#define ODSGD_STATIC_TABLE_BYTES (16 * ODSGD_STATIC_MAX_TENSORS + 8)
int odsgd_fused_update_mult_static(odsgd_ctx* ctx, const float* const* worker_grads, int worker_id,
                                   const float* lr_mult, const float* wd_mult, void* stream);

/*
 * DC-ASGD at the parameter server (the paper's fourth comparison algorithm, Section 4.1):
 * Eq. 4 or Eq. 5/6 applied to one arriving gradient, with the current global weights in the
 * role of w_{t+tau} and local[worker_id] - the copy worker `worker_id` pulled last - in the
 * role of w_t:
 *     w <- w - lr * (g + lambda' * g*g * (w - local[worker_id]));   local[worker_id] <- w
 * (the worker pulls the new weights).  lambda, m, eps come from odsgd_set_local_rule(), whose
 * rule must be ODSGD_LOCAL_DC_C or ODSGD_LOCAL_DC_A; for DC_A the server's single running mean
 * square lives in the arena given to odsgd_set_server_mean_square().  No momentum, no weight
 * decay (Eq. 4/5 have neither).  In place on the current weights; like the ASGD step it
 * invalidates the backup weights.  local[worker_id] must hold the weights that worker pulled
 * (initially a copy of w_0).
 * Errors: ERR_STATE (rule is SGD, or DC_A without a server mean-square arena), ERR_ARG, ERR_OVERLAP.
 */
int odsgd_dcasgd_step(odsgd_ctx* ctx, int worker_id, const float* grad, void* stream);

/* Device arena (n_params floats, caller-owned, normally zero-filled) for Eq. 6's state at the server. */
int odsgd_set_server_mean_square(odsgd_ctx* ctx, float* mean_square);

/*
 * The worker loop of Algorithm 2 as a state machine.  odsgd_set_warmup() sets wp, the number
 * of warm-up iterations (the paper uses 200 iterations, or 0-5 epochs); it may be called
 * only before the first odsgd_step().  odsgd_step() runs iteration k = 0, 1, 2, ...:
 *   k <  wp : SSGD step (warm-up stage: workers wait for and train on the new weights);
 *   k >= wp : fused global + local update for every worker that has a local buffer (at
 *             k = wp, the last warm-up iteration of Algorithm 2, the gradient was still taken
 *             on the global weights, so the delay-compensated rules see no delay there).
 * The copy "w_bak = w_t" of iteration wp - 1 is implicit: the backup is the weight half the
 * update reads.  odsgd_get_train_weights() tells which arena worker `worker_id` computes its
 * next gradient on: the current global weights while the next iteration index is <= wp, its
 * local arena afterwards.
 */
int odsgd_set_warmup(odsgd_ctx* ctx, uint64_t wp);
int odsgd_step(odsgd_ctx* ctx, const float* const* worker_grads, void* stream);
int odsgd_step_bound(odsgd_ctx* ctx, int slot, void* stream); /* the same on a table bound by odsgd_bind_grads */
int odsgd_get_train_weights(odsgd_ctx* ctx, int worker_id, float** weights);

/*
 * Checkpoint / resume.  Every arena is the caller's, so saving them saves the state; what the
 * context adds is the iteration index of the state machine above and the step counter.  To
 * resume: create a context with the saved current global weights as w_a (plus v, the local
 * arenas and, for ODSGD_LOCAL_DC_A, the mean-square arenas), choose the same rule and warm-up
 * length, then restore the iteration index with odsgd_set_iteration (allowed at any time; it
 * also lifts the "before the first odsgd_step" restriction of odsgd_set_warmup when set to 0).
 */
int odsgd_get_iteration(odsgd_ctx* ctx, uint64_t* iteration);
int odsgd_set_iteration(odsgd_ctx* ctx, uint64_t iteration);

/*
 * Learning-rate schedules the paper's runs use (Section 4): host-side helpers that return the
 * rate for iteration `step`; feed the result to odsgd_set_lr / odsgd_set_local_lr.
 *   step decay : base * factor^(number of boundaries <= step)       (divide by 10 at given epochs)
 *   linear ramp: start + (end - start) * min(step, ramp) / ramp     (the "WP" ramp 0.1 -> 0.8)
 *   polynomial : end + (base - end) * (1 - min(step, total)/total)^power   (power 2 in the paper)
 * Computed in double, rounded once to float.
 */
float odsgd_lr_step_decay(float base_lr, float factor, const uint64_t* boundaries, size_t n_boundaries, uint64_t step);
float odsgd_lr_linear_ramp(float start_lr, float end_lr, uint64_t ramp_steps, uint64_t step);
float odsgd_lr_poly_decay(float base_lr, float end_lr, float power, uint64_t total_steps, uint64_t step);

/* Current and backup (one step old) weight arenas; either output pointer may be NULL.
 * *delayed is NULL when the context keeps no backup or none is valid yet. */
int odsgd_get_weights(odsgd_ctx* ctx, float** current, float** delayed);

/* Number of global updates (OD-SGD or SSGD) plus ASGD / DC-ASGD steps applied so far: the
 * server's counter t of Algorithm 1 ("t <- t + 1" after each update of w_t).  The setter is for
 * resuming from a checkpoint. */
int odsgd_get_step(odsgd_ctx* ctx, uint64_t* step);
int odsgd_set_step(odsgd_ctx* ctx, uint64_t step);

/*
 * Launch shape of the update kernels.  block_threads: 64..1024, multiple of 32 (a block
 * too large for a kernel's register use makes that call fail with ERR_UNSUPPORTED);
 * ctas_per_sm: >= 1, grid = min(tiles, SMs * ctas_per_sm) CTAs striding over the tiles;
 * 0 for either restores the built-in choice.
 */
int odsgd_set_launch_config(odsgd_ctx* ctx, int block_threads, int ctas_per_sm);

/* How many kernels this context has launched since create. */
int odsgd_get_launch_count(odsgd_ctx* ctx, uint64_t* launches);

/* Text describing the last failure on `ctx` (or, for ctx == NULL, of the last failed
 * odsgd_create on this thread).  Never NULL. */
const char* odsgd_last_error(odsgd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* ODSGD_H_ */
