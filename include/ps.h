/*
 * ps.h - C ABI of the B200 parameter-server hot path.
 *
 * Two parts, after the paper "Training Through Failure: Effects of Data
 * Consistency in Parallel Machine Learning Training":
 *
 *   A. the worker step: W logical workers each compute the gradient of the
 *      paper's small CNN (model endnote: conv 16 - ReLU - maxpool, conv 32 -
 *      ReLU - maxpool, flatten, dense 512 - ReLU, dropout 25 %, dense 10) on
 *      their own mini-batch against their own, possibly stale, weight snapshot;
 *   B. the server step: the parameter server applies the queued worker
 *      gradients all at once per iteration (sync), one by one in arrival order
 *      (async), or as one deferred pass over everything that was buffered while
 *      it was down (stateless server), with periodic checkpoints, rollback, and
 *      a chain-replication mirror.
 *
 * Conventions
 *   - Every function returns an int32 status: PS_OK (0) or a negative PS_ERR_*.
 *     Nothing throws, aborts or traps.  ps_last_error() gives a text for the
 *     last failure on the calling thread.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are host memory.
 *     The library allocates no device memory: it carves everything out of the
 *     caller's arena (ps_config.arena) and pinned host block (ps_config.pinned),
 *     whose sizes ps_query_bytes() reports.  The caller owns both blocks and
 *     every input/output buffer, and must keep them alive until ps_destroy().
 *   - All device work is enqueued on ps_config.stream and is asynchronous with
 *     respect to the host unless stated otherwise.  One host thread per context.
 *   - Parameters and gradients are flat fp32 vectors of PS_PARAM_COUNT floats in
 *     the canonical order below; device copies use a row stride of
 *     PS_PARAM_STRIDE floats (padding is zero).
 *
 *       conv1.w [16][1][3][3]  at      0      fc1.w [512][1568] at   4800
 *       conv1.b [16]           at    144      fc1.b [512]       at 807616
 *       conv2.w [32][16][3][3] at    160      fc2.w [10][512]   at 808128
 *       conv2.b [32]           at   4768      fc2.b [10]        at 813248
 *
 *     fc1's input index is c*49 + y*7 + x (channel-major flatten).
 */
#ifndef PS_B200_H
#define PS_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PS_PARAM_COUNT  813258
#define PS_PARAM_STRIDE 813312   /* floats; 3,253,248 bytes, a multiple of 256 */
#define PS_MAX_WORKERS  256
#define PS_MAX_RING     16
#define PS_IMAGE_PIXELS 784      /* 1 x 28 x 28 */
#define PS_NUM_CLASSES  10

enum {
  PS_OK = 0,
  PS_ERR_BAD_ARG = -1,
  PS_ERR_DOWN = -2,             /* the server is down (and, unless the store is external, so are its weights) */
  PS_ERR_QUEUE_FULL = -3,
  PS_ERR_NO_CHECKPOINT = -4,
  PS_ERR_VERSION_EVICTED = -5,  /* the requested weight version is no longer retained */
  PS_ERR_NO_REPLICA = -6,
  PS_ERR_ARENA_TOO_SMALL = -7,
  PS_ERR_CUDA = -8,
  PS_ERR_DEVICE_STATUS = -9     /* a kernel's own input check tripped (e.g. a label outside 0..9) */
};

/* Arithmetic of the dense contractions of part A.  PS_FP32: everything on the FP32 pipes.  PS_BF16: the
 * tensor-core path: BF16 operands (fp32 accumulation) in the products of the second convolution and in the
 * first convolution's filter gradient, TF32 operands in the 512-unit layer; the first convolution's forward
 * pass and the output layer stay FP32.  PS_TF32 is reserved and not built (ps_create refuses it). */
enum { PS_FP32 = 0, PS_TF32 = 1, PS_BF16 = 2 };
typedef enum { PS_SYNC = 0, PS_ASYNC = 1, PS_REPLAY = 2 } ps_mode;

typedef struct ps_ctx ps_ctx;   /* opaque; owned by the library */

typedef struct {
  int32_t  max_workers;      /* 1..PS_MAX_WORKERS logical workers per grad step               */
  int32_t  max_batch;        /* largest per-worker batch                                       */
  int32_t  ring_depth;       /* weight versions retained for stale readers, 1..PS_MAX_RING    */
  int32_t  ckpt_every;       /* checkpoint when version % ckpt_every == 0; 0 = never          */
  int32_t  ckpt_slots;       /* pinned host checkpoint slots (oldest overwritten); >= 0       */
  int32_t  chain_len;        /* servers in the chain; 1 = no replica                           */
  int32_t  replicate_every;  /* R: versions with version % R == 0 are replication events: the next live server
                              * receives that version; each server further down the chain holds what the one
                              * in front of it held one event earlier (the frontend waits for the next server
                              * only: design section on chain replication, relaxed consistency)              */
  int32_t  external_store;   /* 1 = stateless server: weights and queue survive ps_kill()     */
  int32_t  precision;        /* PS_FP32 | PS_TF32 | PS_BF16                                    */
  float    dropout_p;        /* dropout rate of the 512-unit layer, 0 <= p < 1                 */
  int64_t  queue_slots;      /* capacity of the gradient queue, in gradients                   */
  void*    arena;            /* dev, 256-byte aligned, caller-owned                            */
  uint64_t arena_bytes;
  void*    pinned;           /* host, page-locked, caller-owned                                */
  uint64_t pinned_bytes;
  void*    stream;           /* cudaStream_t (NULL = the legacy default stream)                */
} ps_config;

/* Sizes the arena and the pinned block must have for this configuration (arena/pinned/stream
 * fields are ignored).  PS_ERR_BAD_ARG if a field is out of range. */
int32_t ps_query_bytes(const ps_config* cfg, uint64_t* arena_bytes, uint64_t* pinned_bytes);

/* Creates a server at version 0 holding init_params_host (host, PS_PARAM_COUNT floats, canonical
 * order); every replica starts with the same weights.  Must be called with the arena's device
 * current.  Errors: PS_ERR_BAD_ARG, PS_ERR_ARENA_TOO_SMALL, PS_ERR_CUDA. */
int32_t ps_create(const ps_config* cfg, const float* init_params_host, ps_ctx** out);
int32_t ps_destroy(ps_ctx* ctx);   /* synchronises the stream; frees host state only */

/* ---- worker side (paper: the worker loop of the stateless-server pseudo-code figure) -------- */

typedef struct { uint64_t version; const float* dev_ptr; } ps_snapshot;

/* The worker's weight fetch (first step of the worker loop): version head - lag (lag 0 = latest).  No bytes move: dev_ptr is
 * borrowed from the version ring and stays valid until ring_depth further versions have been
 * produced or the server is killed/restored.  While a stateless server is down the stored
 * weights can still be pulled.  Errors: PS_ERR_DOWN, PS_ERR_VERSION_EVICTED, PS_ERR_BAD_ARG. */
int32_t ps_pull_snapshot(ps_ctx* ctx, int32_t worker, int32_t lag, ps_snapshot* out);

/* Reserves the next n queue slots so that the grad step can write gradients in place.
 * slot_ids (host, [n]) receives consecutive ids.  A reservation is dropped by the next
 * ps_queue_reserve, ps_enqueue or ps_apply.  Errors: PS_ERR_QUEUE_FULL, PS_ERR_DOWN. */
int32_t ps_queue_reserve(ps_ctx* ctx, int32_t n, int64_t* slot_ids);

/* Device address of a queue slot (PS_PARAM_STRIDE floats), borrowed. */
int32_t ps_slot_ptr(ps_ctx* ctx, int64_t slot_id, float** dev_ptr_out);

/* The worker's gradient computation (the training call of the pseudo-code figure's worker loop) for W
 * workers of batch b at once.  Worker w uses weights snaps[w].dev_ptr (workers sharing a pointer
 * are processed as one group), images x_dev[w] and labels y_dev[w], and the dropout mask of
 * Philox4x32-10 keyed by (seed, worker_ids[w], step): element (sample i, unit j) uses counter
 * ((i*512+j)/4, worker id, step lo, step hi), key (seed lo, seed hi), output word (i*512+j)%4, and
 * is kept iff that word >= floor(p*2^32); kept activations are scaled by 1/(1-p).
 *   snaps, worker_ids, slot_ids : host arrays [W]
 *   x_dev [W][b][28][28] fp32, y_dev [W][b] int32 in 0..9            (dev, read)
 *   gradient of worker w is written (PS_PARAM_STRIDE floats, padding zero) to queue slot
 *   slot_ids[w] if slot_ids != NULL, else to grads_dev + w*PS_PARAM_STRIDE      (dev, written)
 *   loss_dev [W] mean cross-entropy per worker; argmax_dev [W][b] lowest index of the largest
 *   logit                                                                       (dev, written)
 * On the tensor-core path x_dev must be 16-byte aligned (the images are read by TMA tile copies).
 * Errors: PS_ERR_BAD_ARG (W, b out of range; NULL pointers; slot not reserved; misaligned x_dev). A label outside
 * 0..9 is reported as PS_ERR_DEVICE_STATUS by ps_stats(). */
int32_t workers_grad_step(ps_ctx* ctx, int32_t W, int32_t b, const ps_snapshot* snaps,
                          const int32_t* worker_ids, const float* x_dev, const int32_t* y_dev,
                          uint64_t seed, uint64_t step, const int64_t* slot_ids, float* grads_dev,
                          float* loss_dev, int32_t* argmax_dev);

/* The worker step when the server is up and only the SUM of the workers' gradients is needed (paper, design section on
 * the stateless server: one server step takes all gradients, applies them, stores the result; synchronous training:
 * all updates of an iteration at once).  Every worker must hold the same snapshot (PS_ERR_BAD_ARG otherwise: stale
 * readers and the outage window need the per-worker gradients of workers_grad_step).  Same inputs as
 * workers_grad_step; instead of W gradient vectors one vector, grad_sum_dev (dev, PS_PARAM_STRIDE floats, 16-byte
 * aligned, written, padding zero) = sum over the workers of each worker's gradient of its own mean loss.  The
 * 512-unit layer's weight gradient, which dominates the bytes, is computed over groups of workers at once, so the W
 * vectors of 3.2 MB are never written.  loss_dev / argmax_dev as in workers_grad_step.  Uses the context's reduction
 * scratch: do not run it concurrently with an apply on another stream. */
int32_t workers_grad_step_summed(ps_ctx* ctx, int32_t W, int32_t b, const ps_snapshot* snaps, const int32_t* worker_ids,
                                 const float* x_dev, const int32_t* y_dev, uint64_t seed, uint64_t step,
                                 float* grad_sum_dev, float* loss_dev, int32_t* argmax_dev);

/* Evaluation pass (paper, implementation section: the metric exporter reports accuracy and loss while training):
 * the forward pass only, without dropout (every unit kept, nothing rescaled), of W groups of b samples, group w
 * against weights snaps[w].dev_ptr.  Same inputs and layouts as workers_grad_step.  loss_dev [W] receives the mean
 * cross-entropy of each group, argmax_dev [W][b] the lowest index of the largest logit, correct_dev [W] the number of
 * samples of the group whose argmax equals the label (all dev, written).  No gradient is produced and the queue is
 * not touched.  Errors as workers_grad_step. */
int32_t workers_eval(ps_ctx* ctx, int32_t W, int32_t b, const ps_snapshot* snaps, const float* x_dev,
                     const int32_t* y_dev, float* loss_dev, int32_t* argmax_dev, int32_t* correct_dev);

/* The dropout keep mask (1 = kept) the grad step uses for one worker: same generator, keying and
 * threshold as workers_grad_step (model endnote: 25 % dropout; rate from ps_config.dropout_p).
 * keep_dev (dev, [b][512] bytes) is written on the context's stream. */
int32_t ps_dropout_mask(ps_ctx* ctx, uint64_t seed, int32_t worker_id, uint64_t step, int32_t b,
                        uint8_t* keep_dev);

/* The worker's gradient append (last step of the worker loop): commits n gradients with their metadata.  With slot_ids (the
 * slots of the current reservation, in order) nothing is copied; with slot_ids == NULL the rows
 * of grads_dev ([n][PS_PARAM_STRIDE], dev) are copied into the next n slots.  All enqueue calls
 * between two applies must carry the same n (it is the per-tick worker count that PS_REPLAY
 * divides by).  A stateful server that is down refuses (PS_ERR_DOWN); a stateless one accepts. */
int32_t ps_enqueue(ps_ctx* ctx, int32_t n, const int64_t* slot_ids, const float* grads_dev,
                   const int32_t* worker_ids, const uint64_t* base_versions, uint64_t step);

/* ---- server side ----------------------------------------------------------------------------- */

typedef struct {
  int64_t  applied;       /* gradients consumed                          */
  uint64_t new_version;   /* head version after the call                 */
  int32_t  checkpointed;  /* periodic checkpoints taken during the call  */
  int32_t  replicated;    /* periodic mirror writes during the call      */
} ps_apply_result;

/* One server step over the whole queue (K gradients), which is then emptied.
 *   PS_SYNC   (synchronous training, implementation section): theta <- theta - lr*scale/K * sum g ; version+1
 *   PS_REPLAY (stateless step: get all gradients, apply, put): theta - lr*scale/W_tick * sum g ; version+1
 *             where W_tick is the n of the enqueue calls (one tick's replay equals the sync step)
 *   PS_ASYNC  (asynchronous training: one update per arriving gradient): for k in order: theta <- theta - lr*scale*g_k,
 *             version+1 each; the last ring_depth versions stay readable by stale workers
 * order (host, [K]) is a permutation of the queue positions giving the arrival order for
 * PS_ASYNC (NULL = FIFO); the other modes sum, so they ignore it.  Versions that are multiples of
 * ckpt_every are checkpointed, multiples of replicate_every are mirrored to the replica inside
 * the same pass.  K = 0 is a no-op.  Errors: PS_ERR_DOWN, PS_ERR_BAD_ARG. */
int32_t ps_apply(ps_ctx* ctx, ps_mode mode, float lr, float scale, const int32_t* order,
                 ps_apply_result* out);

/* ps_apply with the treatments of stale gradients that the paper's design section names, in its closing remarks on the
 * stateless server, as alternatives to a smaller learning rate for many pending gradients (gradient clipping, an
 * adaptive learning rate).  Readings taken here:
 *   clip_norm c > 0        every queued gradient g is scaled by min(1, c / ||g||_2) (clipping by global norm, per
 *                          gradient); costs one extra pass over the queue that takes the norms;
 *   staleness_alpha a > 0  gradient k is scaled by 1 / (1 + a * tau_k), tau_k = the version its update is applied to
 *                          (the head for PS_SYNC / PS_REPLAY, head + j for the j-th gradient of PS_ASYNC) minus the
 *                          base_version given at ps_enqueue.  A base version newer than that is PS_ERR_BAD_ARG.
 * 0 switches a treatment off; with both off the call is ps_apply.  Everything else (modes, order, checkpoints,
 * replication, result) is as in ps_apply. */
int32_t ps_apply_stale(ps_ctx* ctx, ps_mode mode, float lr, float scale, const int32_t* order, float clip_norm,
                       float staleness_alpha, ps_apply_result* out);

/* The synchronous server step from the sum that workers_grad_step_summed produces: theta <- theta - lr * scale / n_workers * grad_sum; version + 1;
 * checkpoint and replication as in ps_apply(PS_SYNC), whose result it equals up to rounding when grad_sum is the sum
 * of the n_workers queued gradients.  The queue must be empty (PS_ERR_BAD_ARG).  `applied` reports n_workers. */
int32_t ps_apply_summed(ps_ctx* ctx, const float* grad_sum_dev, int32_t n_workers, float lr, float scale,
                        ps_apply_result* out);

/* The periodic save of the parameters to persistent storage (design section on checkpointing): copies the
 * head weights and version into the next pinned host slot (stream-ordered device-to-host copy); when all slots
 * are in use the oldest checkpoint is overwritten. */
int32_t ps_checkpoint(ps_ctx* ctx, uint64_t* version_out);

/* Resurrects the server.  Stateful (design section on checkpointing: a restarted server resumes from its latest
 * checkpoint): weights and version are the checkpoint's, the queue is empty, only that version
 * is retained.  Stateless: the store survived, nothing is rolled back.  PS_ERR_NO_CHECKPOINT. */
int32_t ps_restore(ps_ctx* ctx, uint64_t* version_out);

/* One replication event on its own: the head's weights go to the next live server, and what each server held
 * moves one server further down the chain (see ps_config.replicate_every). PS_ERR_NO_REPLICA. */
int32_t ps_replicate(ps_ctx* ctx, uint64_t* version_out);

/* Host-side failure injection: server 0 is the current frontend, i >= 1 the i-th LIVE server behind
 * it (a dead server has left the chain).  Killing a stateful frontend loses its weights, retained versions and queue; no device
 * fault is provoked. */
int32_t ps_kill(ps_ctx* ctx, int32_t server);

/* The next live server of the chain becomes the frontend with the weights it already holds in memory (the
 * version it last received); the queue is empty.  PS_ERR_NO_REPLICA. */
int32_t ps_failover(ps_ctx* ctx, uint64_t* version_out);

/* Replaces the head weights (host, canonical order) without changing the version; used to load a
 * given state.  Synchronous. */
int32_t ps_import_params(ps_ctx* ctx, const float* host_in);

/* Copies parameters to the host (PS_PARAM_COUNT floats): which = 0 head, -(i) the i-th replica
 * (i >= 1), 1000+j the j-th most recent checkpoint (0 = latest).  Synchronises the stream. */
int32_t ps_export_params(ps_ctx* ctx, int32_t which, float* host_out, uint64_t* version_out);

typedef struct {
  uint64_t version;          /* head version                          */
  uint64_t oldest_version;   /* oldest version still retained         */
  int64_t  queue_len;        /* committed gradients                   */
  int64_t  applied_total;    /* gradients applied since ps_create     */
  int32_t  up;               /* 1 = the frontend is alive             */
  int32_t  live_replicas;
  int32_t  checkpoints;      /* valid checkpoint slots                */
  uint32_t device_status;    /* 0, or the kernels' input-check flags  */
  uint64_t replica_version;  /* version held by the next server       */
  uint64_t last_ckpt_version;
  int64_t  kernel_launches;  /* kernels launched since ps_create      */
} ps_stats_t;

/* Synchronises the stream and reports counters; returns PS_ERR_DEVICE_STATUS if a kernel's input
 * check tripped (the fields are filled in either way). */
int32_t ps_stats(ps_ctx* ctx, ps_stats_t* out);

/* One whole tick from host buffers: copies x_host/y_host (page-locked memory recommended) to the
 * device, pulls a snapshot per worker (lags host [W] or NULL = 0), runs the grad step into
 * reserved slots, enqueues, applies (apply_mode < 0 skips the apply, e.g. while the server is
 * down) and copies loss (and argmax, if non-NULL) back to the host before returning. */
int32_t ps_tick_host(ps_ctx* ctx, int32_t W, int32_t b, const int32_t* lags, const float* x_host,
                     const int32_t* y_host, uint64_t seed, uint64_t step, int32_t apply_mode,
                     float lr, float scale, const int32_t* order, float* loss_host,
                     int32_t* argmax_host, ps_apply_result* out);

/* The same tick without waiting for it: ps_tick_host_submit enqueues the copies and all the work of a tick and
 * returns; ps_tick_host_wait blocks until the oldest submitted tick has finished (its losses and labels are then in
 * the host buffers given at submit) and returns its apply result.  Up to two ticks may be in flight, so the
 * host-to-device copy of the next tick's inputs (on a copy stream of the library's own) runs while the current
 * tick computes; on the device the ticks still run one after the other: snapshots, versions and the queue are
 * exactly those of back-to-back ps_tick_host calls (the paper's workers likewise fetch their next batch while the
 * server works).  x_host, y_host, loss_host and argmax_host must stay valid and untouched until the matching wait.
 * Errors: PS_ERR_BAD_ARG when two ticks are already in flight (submit) or none is (wait); otherwise as ps_tick_host.
 * Other calls on the context are allowed between submit and wait only if they do not depend on that tick. */
int32_t ps_tick_host_submit(ps_ctx* ctx, int32_t W, int32_t b, const int32_t* lags, const float* x_host,
                            const int32_t* y_host, uint64_t seed, uint64_t step, int32_t apply_mode,
                            float lr, float scale, const int32_t* order, float* loss_host,
                            int32_t* argmax_host);
int32_t ps_tick_host_wait(ps_ctx* ctx, ps_apply_result* out);

/* Exercises the give-up path of the library's bounded waits without disturbing anything (no counterpart in the
 * paper's method; it serves failure detection).  Every wait of the tensor-core kernels on a barrier has a cycle
 * limit; when it runs out the kernel sets bit 1 of the status word, releases what it holds and returns, and
 * ps_stats() then reports PS_ERR_DEVICE_STATUS.  This call launches, on the context's stream, one warp that waits on
 * a barrier of its own at which nobody arrives, for at most limit_cycles SM clock cycles (1..2e9; 20,000 is about
 * 10 microseconds), and then does exactly that.  Nothing else is touched; the context stays usable, but its status
 * word keeps the bit until the context is destroyed. */
int32_t ps_selftest_wait_timeout(ps_ctx* ctx, int64_t limit_cycles);

/* Per-kernel timing for measurement (no counterpart in the paper's method; it serves the roofline
 * report).  ps_profile(ctx, 1) clears the totals and from then on brackets every kernel launch with
 * two CUDA events on the context's stream (and runs the branches of the backward pass one after the
 * other instead of side by side, so that each kernel is timed alone); ps_profile(ctx, 0) stops.
 * ps_profile_read() synchronises
 * the stream and returns, for kernel index 0..n-1, its name (static string), summed device time in
 * milliseconds and launch count; an index past the last kernel returns PS_ERR_BAD_ARG. */
int32_t ps_profile(ps_ctx* ctx, int32_t enable);
int32_t ps_profile_read(ps_ctx* ctx, int32_t kernel, const char** name, double* total_ms, int64_t* launches);

/* Reduce-and-apply without a context and without any allocation.  The paper has no counterpart:
 * this exists for callers that cannot obtain device memory at the time of the call, for example
 * code embedded in an application whose own pool already owns all of the GPU's memory, or a loop
 * that must not stall on the device-wide synchronisation an allocation implies.
 *
 *   theta_out = theta_in - coef * (queue[0] + ... + queue[K-1])
 *
 * queue_dev: K gradients, row stride PS_PARAM_STRIDE floats; theta_in_dev / theta_out_dev:
 * PS_PARAM_STRIDE floats each (may be the same buffer); all dev, 16-byte aligned, caller-owned.
 * 1 <= K <= PS_STATIC_REPLAY_MAX_GRADIENTS, otherwise PS_ERR_BAD_ARG and nothing is launched
 * (apply a longer queue in several calls, feeding theta_out back in as theta_in).  The work is
 * enqueued on `stream` (a cudaStream_t, NULL = legacy default stream) of the current device.
 *
 * The partial sums are kept in a fixed array inside the library image: PS_STATIC_REPLAY_SPLITS
 * vectors of PS_PARAM_STRIDE floats, about 13 MB per GPU, held until the process exits.  The entry
 * point calls no allocator, CUDA's or anyone else's.
 *
 * The first call on each device is a set-up call: it looks up the array's device address, and because
 * CUDA loads a library's device code lazily, that lookup is also the moment the driver sets the array
 * up on that device (13 MB; it can take as long as an allocation would, and on a device whose memory is
 * all taken it fails: PS_ERR_CUDA with a text that says so).  So make one warm-up call per device at
 * start-up, before the application's pool takes the memory and before any stream capture; later calls
 * only launch two kernels.  All calls on a device share the one array and it is not cleared between
 * calls (each call overwrites every element it later reads), so two calls whose kernels may overlap on
 * the GPU, e.g. on different streams, race: serialise them.
 * ps_replay_sum_static_error() returns the text of the calling thread's last failure here. */
#define PS_STATIC_REPLAY_SPLITS 4
#define PS_STATIC_REPLAY_MAX_GRADIENTS 65536
int32_t ps_replay_sum_static(const float* queue_dev, int64_t K, const float* theta_in_dev,
                             float* theta_out_dev, float coef, void* stream);
const char* ps_replay_sum_static_error(void);

const char* ps_last_error(ps_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* PS_B200_H */
