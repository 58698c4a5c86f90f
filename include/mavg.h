/* mavg.h -- C ABI of the M-AVG engine (K-step model averaging with block momentum,
 * Algorithm 1 of Cong & Liu, "Accelerate Distributed Stochastic Descent for Nonconvex
 * Optimization with Momentum").
 *
 * All P learners are held on one GPU as a [P, stride] fp32 replica array.  One round n is
 *   learner level (Algorithm 1, inner loop):  every learner j takes K minibatch-SGD steps
 *       w^j <- w^j - (gamma / B) sum_s grad F(w^j; xi^j_{k,s}),  k = 1..K
 *   meta level (Algorithm 1, last four assignments of the outer loop):
 *       a = (1/P) sum_j w^j;  d = a - w~;  v <- mu v + zeta d;  w~ <- w~ + v
 *   and the start of the next round (Algorithm 1, "set w^j_n = w~_n"):  w^j <- w~  for all j.
 * zeta, the block learning rate, is an extension; zeta = 1 is the paper's update.  mu = 0 with
 * zeta = 1 is K-AVG (Remark after Theorem 1).
 *
 * Conventions
 *   - Every pointer is tagged DEVICE or HOST below.  Device buffers and the CUDA stream belong to
 *     the caller and are borrowed from mavg_create until mavg_destroy; the library calls no
 *     device allocator and frees nothing of the caller's.  The handle is host memory owned by the
 *     library; for the MLP objective it also holds a CUDA graph of one round's local steps
 *     (recorded on a private stream at the first round, replayed on the caller's stream).
 *   - All work is enqueued on the configured stream and returns without waiting, except where a
 *     function hands a value back to HOST memory (then it waits for the stream).
 *   - Errors are status codes; nothing throws, aborts or traps.  Arguments are checked on the
 *     host before anything is launched.  A CUDA error is sticky: the call that meets it and every
 *     later call return MAVG_ERR_CUDA.  mavg_last_error gives a message for the last failure.
 *   - A handle is not thread-safe; distinct handles are independent.
 *   - Counters: rounds n = 1, 2, ...; learners j = 0..P-1; local steps k = 1..K; batch slots
 *     s = 0..B-1.
 *
 * Random numbers (the paper says only "randomly sample a mini-batch"): SplitMix64 used as a
 * counter-based generator.  With mix64 the SplitMix64 output function and G = 0x9E3779B97F4A7C15,
 * fold(s, c) = mix64(s + (c+1) G); the stream of (tag, n, j, k) has key
 * fold(fold(fold(fold(seed, tag), n), j), k) and element i of it is fold(key, i).
 *   tag 1, minibatch indices: learner j owns samples [floor(j S/P), floor((j+1) S/P)); slot s
 *     draws  lo_j + floor(u * len_j / 2^32), u = top 32 bits of element s  (i.i.d. uniform with
 *     replacement inside the learner's shard).
 *   tag 2, synthetic gradients: element i is (sum of the four 16-bit lanes of the 64-bit value
 *     - 131070) * c,  c = fp32(sigma / sqrt(4 (65536^2 - 1) / 12)): an Irwin-Hall(4) variate with
 *     mean 0 and standard deviation sigma, the same bits on every IEEE machine.
 */
#ifndef MAVG_H_
#define MAVG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mavg_ctx *mavg_handle;

typedef enum {
  MAVG_OK = 0,
  MAVG_ERR_INVALID_ARG = 1, /* a scalar argument is out of its domain, or a required pointer is NULL */
  MAVG_ERR_BAD_BUFFER = 2,  /* a buffer is NULL, misaligned or too small */
  MAVG_ERR_STATE = 3,       /* call not valid for this handle (wrong objective, destroyed handle) */
  MAVG_ERR_UNSUPPORTED = 4, /* shape outside what the kernels cover, or no sm_100 device */
  MAVG_ERR_CUDA = 5,        /* a CUDA call or kernel failed; see mavg_last_error */
  MAVG_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up; the context stays usable */
} mavg_status;

typedef enum {
  MAVG_OBJ_NONE = 0,       /* no learner level: the caller writes the replicas (meta-update only) */
  MAVG_OBJ_PSEUDOGRAD = 1, /* grad F(w; xi) replaced by seeded N(0, sigma^2)-like variates (tag 2) */
  MAVG_OBJ_MLP = 2         /* MLP with bias, ReLU, softmax cross-entropy averaged over the batch */
} mavg_objective;

typedef enum { MAVG_X_F32 = 0, MAVG_X_BF16 = 1 } mavg_x_dtype;

#define MAVG_MAX_LAYERS 8

/* Problem statement: the five hyper-parameters the paper lists (P, B, K, step size, mu) plus the
 * objective the learners descend.  Plain data, copied by mavg_create. */
typedef struct {
  int32_t P;         /* learners, >= 1 */
  int32_t K;         /* local steps per round, >= 1 */
  int32_t B;         /* minibatch per learner and step, >= 1 (ignored unless MLP) */
  float local_lr;    /* gamma of Algorithm 1, finite */
  float block_lr;    /* zeta, finite; 1 reproduces Algorithm 1 */
  float mu;          /* block momentum, 0 <= mu < 1 (Theorem 1's domain) */
  uint64_t seed;
  int32_t objective; /* mavg_objective */
  int64_t n;         /* parameters per replica, >= 1; for MLP must equal the layout's count */
  /* MLP: layer l = 1..n_layers maps dims[l-1] -> dims[l]; flat layout per replica
   * [W_1 (dims[1] x dims[0], row-major), b_1, W_2, b_2, ...]. */
  int32_t n_layers;
  int32_t dims[MAVG_MAX_LAYERS + 1];
  int32_t gemm_bf16; /* 0: fp32 FMA arithmetic throughout.  1: every matrix-product operand
                        (weights, activations, dZ) rounded to bf16 (nearest-even), fp32
                        accumulation, fp32 master weights, bias, ReLU, softmax and SGD in fp32 */
  float pseudo_grad_sigma; /* PSEUDOGRAD: standard deviation of the variates */
  const void *x;     /* DEVICE [n_samples, dims[0]] row-major, fp32 or bf16 per x_dtype */
  int32_t x_dtype;   /* mavg_x_dtype; bf16 requires gemm_bf16 */
  const int32_t *y;  /* DEVICE [n_samples] labels in [0, dims[n_layers]) */
  int64_t n_samples; /* S >= P, < 2^31 */
  void *stream;      /* cudaStream_t (NULL = the legacy default stream) */
  int32_t defer_broadcast; /* 0: "set w^j = w~" is carried out as P copies by mavg_create,
                        mavg_meta_update, mavg_set_round and mavg_round_host (the replica array
                        then equals w~ between rounds).  1: those calls leave the replica array
                        untouched; the first local step of the next round reads w~ in place of
                        every w^j and writes each learner's own result, which is the same
                        assignment with 4P bytes per element less traffic.  Between a meta-update
                        and the next local step the replica array then holds the previous round's
                        learner models; mavg_materialize_replicas writes the copies on request. */
  /* Learner-level momentum (the variant the paper names after Eq. 2 and in its conclusion:
   * momentum SGD inside each learner, under the block momentum of the meta level).  With
   * beta = learner_momentum != 0 the local step of Algorithm 1 becomes, in the form Eq. 2 uses,
   *     u^j <- beta u^j - gamma g;   w^j <- w^j + u^j
   * with one buffer u^j per learner (mavg_buffers.learner_u).  beta = 0 is Algorithm 1 as printed.
   * The paper does not say what happens to u^j when a round ends; learner_momentum_reset picks:
   * 0: u^j is kept over the rounds (zero only before the first round); 1: u^j <- 0 whenever the
   * learners restart from w~ (the first local step after a (re-)broadcast). */
  float learner_momentum;         /* beta, 0 <= beta < 1 */
  int32_t learner_momentum_reset; /* 0 or 1 */
  int32_t l2_keep;   /* 0 (default): the library leaves the L2 cache's partitioning alone.
                        1: an MLP handle on the tensor-core path whose P master copies together
                        take at most half the L2 asks mavg_create to set aside that much of the
                        L2 for them (see mavg_create); ignored by every other handle.  This is an
                        opt-in because the set-aside belongs to the whole CUDA context: while it is
                        in force, every streaming kernel of the process -- this library's
                        meta-update of a large model included -- has only the rest of the L2 and
                        was measured 25-30 % slower (6.2 -> 4.4 TB/s), against a gain of 2-3 % on
                        a small MLP round. */
} mavg_config;

/* Caller-owned DEVICE buffers.  Every base pointer must be 16-byte aligned. */
typedef struct {
  float *replicas;        /* [P, replica_stride] fp32; row j is w^j */
  int64_t replica_stride; /* floats between rows, >= n and a multiple of 4 */
  float *global_w;        /* [n] w~; on entry to mavg_create it holds w~_1 */
  float *momentum;        /* [n] v */
  void *workspace;        /* scratch, at least mavg_workspace_bytes() bytes */
  size_t workspace_bytes;
  float *learner_u;       /* [P, replica_stride] fp32 learner momentum buffers u^j, same layout as
                             replicas; required iff learner_momentum != 0 (else ignored, may be
                             NULL).  mavg_create zeroes it. */
} mavg_buffers;

/* Bytes of scratch the configuration needs (activations, bf16 operand copies, batch indices,
 * loss accumulators, the device status word).  Checks the configuration like mavg_create. */
mavg_status mavg_workspace_bytes(const mavg_config *cfg, size_t *out_bytes);

/* Algorithm 1, the two initialisation lines and the first "set w^j = w~": v <- 0, w^j <- w~_1
 * (the copies are skipped with defer_broadcast, see there).
 * Validates everything; on failure *out is NULL.  Enqueues the initialisation on the stream.
 * With cfg->l2_keep = 1, for an MLP handle on the tensor-core path whose P master copies together
 * take at most half the L2, the call also raises the CUDA context's limit
 * cudaLimitPersistingL2CacheSize to their size (capped by the device's maximum): the
 * weight-gradient kernels then ask the L2 to keep the masters from one local step to the next
 * instead of sending them through HBM.  The limit belongs to the calling process's context: it
 * follows the largest request among the live handles on the device (never below the value
 * found), and the mavg_destroy of the last of them puts the previous value back.  Without
 * l2_keep the library never touches that limit. */
mavg_status mavg_create(const mavg_config *cfg, const mavg_buffers *buf, mavg_handle *out);

/* Learner level of Algorithm 1 (inner loop over k): K SGD steps on all P replicas for the round
 * that follows the last completed meta-update.  MAVG_ERR_STATE for MAVG_OBJ_NONE. */
mavg_status mavg_local_steps(mavg_handle h);

/* Meta level of Algorithm 1 (a, d, v, w~) fused with the re-broadcast w^j <- w~ that opens the
 * next round (folded into the next local step instead with defer_broadcast); advances the round
 * counter. */
mavg_status mavg_meta_update(mavg_handle h);

/* With defer_broadcast: writes w^j <- w~ into the replica array now if the handle is at a round
 * boundary and has not done so yet (a caller that wants to read the P copies).  Otherwise, and
 * without defer_broadcast, a no-op. */
mavg_status mavg_materialize_replicas(mavg_handle h);

/* One round = mavg_local_steps then mavg_meta_update.  If mean_loss is not NULL (HOST, one
 * float) the call waits for the stream and stores the mean of the round's P*K minibatch losses
 * (0 for objectives without a loss). */
mavg_status mavg_round(mavg_handle h, float *mean_loss);

/* The same round for a caller whose model lives in HOST memory: copies w~ and v (n floats each,
 * HOST, read and written) to the device, re-broadcasts w~ to the replicas, runs the round,
 * copies w~ and v back and waits.  The upload of v runs on a stream the handle owns, beside the
 * local steps; both host arrays must stay untouched until the call returns.  mean_loss as in
 * mavg_round. */
mavg_status mavg_round_host(mavg_handle h, float *w_host, float *v_host, float *mean_loss);

/* Per-round schedules (Algorithm 1 lets gamma_n and B_n vary with n; B stays fixed here). */
mavg_status mavg_set_hparams(mavg_handle h, int32_t K, float local_lr, float block_lr, float mu);

/* Changes the learner-level momentum between rounds (see mavg_config).  beta != 0 needs the
 * learner_u buffer given at mavg_create; the buffer's contents are left as they are. */
mavg_status mavg_set_learner_momentum(mavg_handle h, float beta, int32_t reset);

/* Runs the device index generator for (round, learner, step) and copies the B indices to
 * out (HOST, B int32); waits for the stream.  MLP objective only. */
mavg_status mavg_get_batch_indices(mavg_handle h, int64_t round, int32_t learner, int32_t step,
                                   int32_t *out);

/* The P*K minibatch losses of the last mavg_local_steps, out[j*K + k-1] (HOST); waits.
 * MAVG_ERR_STATE for objectives without a loss (everything but MAVG_OBJ_MLP). */
mavg_status mavg_get_losses(mavg_handle h, float *out);

/* Number of completed meta-updates (the next round is this + 1), and its setter for resuming
 * from saved (w~, v, round): the caller restores global_w and momentum, then calls
 * mavg_set_round, which re-broadcasts w~ to the replicas. */
mavg_status mavg_get_round(mavg_handle h, int64_t *round);
mavg_status mavg_set_round(mavg_handle h, int64_t round);

/* Kernels launched by this handle so far. */
mavg_status mavg_get_launch_count(mavg_handle h, int64_t *count);

/* How one local step of the learner level (Algorithm 1's inner loop) is laid out in launches, for
 * measurement and tests; out: HOST array of MAVG_PLAN_COUNT entries.  All entries are 0 for
 * handles without the MLP objective.  MAVG_ERR_INVALID_ARG for a NULL argument. */
typedef enum {
  MAVG_PLAN_TENSOR_PATH = 0,    /* 1: the products run on the tensor cores (bf16 operands) */
  MAVG_PLAN_WGRAD_MERGED = 1,   /* 1: all layers' weight gradients + SGD share one launch */
  MAVG_PLAN_FWD_WITH_WGRAD = 2, /* m >= 0: under the default schedule, in steps 1..K-1 the
                                   weight-gradient launches of layers 1..m also form the next
                                   step's forward product of their layer from the updated tiles
                                   (m <= L-1; layer 1's bf16 copy is not written in those steps) */
  MAVG_PLAN_FWD_RUN_TILES = 3,  /* first of MAVG_MAX_LAYERS entries: for layer l <= m, entry
                                   3 + l - 1 is the number of column tiles per partial sum */
  MAVG_PLAN_DENSE_FIRST_STEP = 3 + MAVG_MAX_LAYERS, /* bit l-1 set: under the default schedule the
                                   forward product of hidden layer l at the first step of a round
                                   (all learners hold w~) is one dense product over the batch rows
                                   of all learners, the weights read once */
  MAVG_PLAN_FWD_WHOLE_ROWS = 4 + MAVG_MAX_LAYERS, /* first of MAVG_MAX_LAYERS entries: for layer
                                   l <= m, how many of its P x ceil(out / 128) (learner, row tile)
                                   pairs are taken as one run over all column tiles (no partial
                                   sums); the others are cut into runs of FWD_RUN_TILES tiles */
  MAVG_PLAN_COUNT = 4 + 2 * MAVG_MAX_LAYERS
} mavg_plan_entry;
mavg_status mavg_get_step_plan(mavg_handle h, int32_t *out);

/* Measurement aid (the paper has no counterpart).  While profiling is on, every kernel launch of
 * this handle is bracketed by a pair of CUDA events on the stream.  mavg_get_profile waits for the
 * stream and returns, per kernel class, the summed device time in milliseconds and the number of
 * launches since the last reset (ms and launches: HOST arrays of MAVG_K_COUNT entries). */
typedef enum {
  MAVG_K_META = 0,      /* fused meta-update + re-broadcast */
  MAVG_K_BROADCAST = 1, /* initial / resume broadcast */
  MAVG_K_PSEUDOGRAD = 2,
  MAVG_K_BATCH = 3,     /* index stream and gather */
  MAVG_K_FWD = 4,       /* forward GEMMs (+bias, ReLU) */
  MAVG_K_LOSS = 5,      /* softmax cross-entropy and loss reductions; the fused last-layer kernel */
  MAVG_K_DGRAD = 6,     /* backward-data GEMMs (+ReLU mask, bias step) */
  MAVG_K_WGRAD_SGD = 7, /* backward-weight GEMMs fused with the SGD step */
  MAVG_K_AUX = 8,       /* operand copies (bf16 shadows) */
  MAVG_K_COUNT = 9
} mavg_kernel_class;
mavg_status mavg_set_profiling(mavg_handle h, int32_t on);
/* Schedule of the tensor-core MLP learner level (the paper has no counterpart).
 *   MAVG_SCHED_GRAPH (default): one launch per matrix product, the K steps of a round replayed
 *     from a CUDA graph; where the last layer's tensor-core tiles would leave most of the GPU idle
 *     (at most 32 classes, few learners) that layer -- forward, loss, dZ_L, its data gradient and
 *     the bias steps -- runs as one CUDA-core kernel, and hidden-layer forward products may split
 *     their contraction over a thread-block cluster.
 *   MAVG_SCHED_GRAPH_TC: the same graph with every product as plain one-tile-per-block
 *     tensor-core launches.  The two differ in the summation order of the products they run
 *     differently, nothing else; this one exists for comparison.
 * Profiled rounds (mavg_set_profiling) take the launch-by-launch form of the chosen schedule. */
typedef enum { MAVG_SCHED_GRAPH = 0, MAVG_SCHED_GRAPH_TC = 2 } mavg_schedule;
mavg_status mavg_set_schedule(mavg_handle h, int32_t mode);
mavg_status mavg_get_profile(mavg_handle h, float *ms, int64_t *launches, int32_t reset);

/* Waits for the stream; reports CUDA errors and a tripped device-side wait limit. */
mavg_status mavg_sync(mavg_handle h);

/* Every wait inside the kernels (on an mbarrier, on another block's counter) gives up after a time
 * limit instead of spinning forever; the kernel then records an error code, lets its own copies
 * in flight land, frees what it holds and returns, and the next mavg_sync reports
 * MAVG_ERR_TIMEOUT and clears the record (the paper has no counterpart: this is failure detection
 * of the engine itself).  The default limit is 2 s.  mavg_set_wait_limit changes it for this
 * handle's later launches (microseconds, >= 1; 0 restores the default); stream-ordered.
 * mavg_selftest_wait launches a one-warp kernel that waits on a barrier nobody will ever arrive
 * on, so that the wait runs out: after it, mavg_sync must return MAVG_ERR_TIMEOUT once and
 * MAVG_OK afterwards, and the handle must work as before.  Nothing traps or faults; the kernel
 * returns by itself after the limit. */
mavg_status mavg_set_wait_limit(mavg_handle h, int32_t microseconds);
mavg_status mavg_selftest_wait(mavg_handle h);

/* Waits for the stream, then returns every L2 line that this context asked to be kept (see
 * mavg_create) to normal eviction; a no-op for handles that keep nothing.  For measurements that
 * want a cold cache at the start of a round: lines kept this way survive an ordinary flush. */
mavg_status mavg_cache_release(mavg_handle h);

/* Message for the last failure on this handle ("" if none); with h == NULL, for the last failed
 * mavg_create / mavg_workspace_bytes of the calling thread.  Valid until the next call. */
const char *mavg_last_error(mavg_handle h);

/* The index stream of mavg_get_batch_indices for callers that cannot allocate device memory (the
 * paper has no counterpart; this is an addition for such hosts).  Think of a process whose
 * device memory has all been handed to another component's pool, a plug-in that runs under a
 * fixed memory budget, or a latency-critical loop that must not call cudaMalloc because that
 * call may stall the whole device: none of them can provide the workspace a handle needs.
 * Here no handle and no workspace exist.  The B indices that `learner` draws at local step
 * `step` of round `round` (same generator, same shard rule, same bits as the handle-based call)
 * are staged in an array that is part of the library image on the GPU -- 65536 int32 = 256 KB,
 * held by every GPU that loads the library until the process exits -- and copied to out
 * (HOST, B int32); the call waits for the stream.  B > 65536 is refused with
 * MAVG_ERR_INVALID_ARG.  The call itself allocates and frees nothing.
 * The first call on a device looks up the array's device address (the device must be current);
 * make that first call before any stream capture begins.  All calls share the one array, which
 * keeps the previous call's indices; nothing in it needs clearing because every call overwrites
 * the B entries it reads back.  Two calls in flight at once on the same GPU (different host
 * threads or streams) would race on it: issue them one after the other.
 * stream: cudaStream_t (NULL = default stream).  Errors: mavg_last_error(NULL). */
mavg_status mavg_batch_indices_noalloc(uint64_t seed, int64_t round, int32_t P, int32_t learner,
                                       int32_t step, int64_t n_samples, int32_t B, void *stream,
                                       int32_t *out);

/* Releases the handle (host memory only).  NULL is a no-op. */
mavg_status mavg_destroy(mavg_handle h);

#ifdef __cplusplus
}
#endif
#endif /* MAVG_H_ */
