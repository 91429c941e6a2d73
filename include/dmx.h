/*
 * dmx.h — C ABI of the DYNAMIX data-parallel gradient step on one GPU.
 *
 * The operation (Algorithm 1, the body of the innermost loop over the workers: each worker
 * computes a gradient g_i at its own batch size x_i and the global model is updated under
 * BSP; Section "State representation", paragraph "Training Statistical Efficiency Metrics":
 * the controller reads gradient statistics, sigma_norm and sigma^2_norm):
 *
 *   K emulated workers hand in flat gradient vectors x_k[0..P) computed at batch sizes b_k.
 *   One call forms the batch-size-weighted aggregate g = sum_k b_k x_k / sum_k b_k, the
 *   statistics the batch-size policy reads, and the SGD-momentum update
 *   m <- beta*m + g, theta <- theta - lr*m, prev_agg <- g.
 *
 * The paper states no formula for the aggregate, the statistics or the optimizer; the
 * definitions below are this library's reading and are the contract.
 *
 * Conventions
 *   - Every function returns DMX_OK (0) or a negative DMX_ERR_* code. Nothing throws,
 *     aborts or traps, on the host or on the device.
 *   - "HOST" / "DEVICE" on a pointer says which memory it addresses.
 *   - dmx_step is asynchronous: it enqueues work on the given stream and returns. It does
 *     not allocate, does not synchronise and copies nothing host-to-device (worker pointers,
 *     weights and batch sizes travel as kernel arguments).
 *   - A handle may be used from one stream at a time (its scratch is shared by its calls).
 *   - A handle belongs to the CUDA device that was current in dmx_create: its tables and scratch
 *     live there. A step issued while another device is current returns DMX_ERR_HANDLE before
 *     anything is enqueued (make the handle's device current first).
 *   - Handles are looked up in a table of live handles, never read through the pointer first:
 *     a call on a destroyed (or never created) handle returns DMX_ERR_HANDLE and touches no
 *     freed memory. An address reused by a later create names that later handle.
 *   - dmx_step, dmx_step_adam and their _partial forms enqueue two kernel launches and nothing
 *     else, so (with per-kernel timing off) they can be captured in a CUDA graph and replayed:
 *     the kernels leave the handle's scratch ready for the next run.
 */
#ifndef DMX_H_
#define DMX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dmx_handle dmx_handle;

/* gradient element types */
enum { DMX_F32 = 0, DMX_BF16 = 1 };

/* return codes */
enum {
  DMX_OK = 0,
  DMX_ERR_ARG = -1,      /* null pointer, K/P/S out of range, aliasing buffers, bad dtype  */
  DMX_ERR_SEGMENTS = -2, /* segment table not o[0]=0 <= o[1] <= ... <= o[S]=P              */
  DMX_ERR_BATCH = -3,    /* some batch size < 1                                            */
  DMX_ERR_ALIGN = -4,    /* a device pointer is not 16-byte aligned                        */
  DMX_ERR_NOMEM = -5,    /* host or device allocation failed                               */
  DMX_ERR_CUDA = -6,     /* a CUDA runtime call failed (see dmx_last_cuda_error)           */
  DMX_ERR_HANDLE = -7,   /* handle is NULL, destroyed, or belongs to another CUDA device   */
  DMX_ERR_LIMIT = -8,    /* problem too large for the fixed scratch of dmx_step_static     */
  DMX_ERR_GUARD = -9     /* dmx_check_guards: a guard word beside the scratch was overwritten */
};

/* limits */
#define DMX_MAX_WORKERS 64
#define DMX_MAX_SEGMENTS 65536
#define DMX_MAX_PARAMS (((int64_t)1) << 40)

/*
 * Layout of out_state (fp32, length dmx_state_len = 16 + K + 2*S).
 * With B = sum_k b_k, q_k = sum_j x_kj^2, A = sum_j g_j^2,
 * D = sum_j sum_k b_k (x_kj - g_j)^2, a = prev_agg as passed in:
 */
enum {
  DMX_ST_B_TOTAL = 0,      /* B                                                            */
  DMX_ST_AGG_SQNORM = 1,   /* A                                                            */
  DMX_ST_TR_SIGMA = 2,     /* tr(Sigma)^ = D/(K-1); unbiased for the per-sample covariance */
                           /* trace when x_k is a mean of b_k i.i.d. samples; 0 if K == 1  */
  DMX_ST_G2 = 3,           /* |G|^2^ = A - tr(Sigma)^/B; unbiased, may be <= 0             */
  DMX_ST_GNS = 4,          /* gradient noise scale tr(Sigma)^ / |G|^2^ if |G|^2^ > 0 else 0
                              (the quantity behind the paper's large->medium->small
                              batch schedule, Section "RL Agent Inference Evaluation",
                              paragraph "Batch Size Adaptation Dynamics")                      */
  DMX_ST_COS_PREV = 5,     /* <g,a> / sqrt(A * |a|^2) if both norms > 0 else 0             */
  DMX_ST_DOT_PREV = 6,     /* <g,a>                                                        */
  DMX_ST_PREV_SQNORM = 7,  /* |a|^2                                                        */
  DMX_ST_SIGMA2_NORM = 8,  /* sigma^2_norm = tr(Sigma)^ / (B*A) if A > 0 else 0            */
  DMX_ST_SIGMA_NORM = 9,   /* sigma_norm = sqrt(max(sigma^2_norm, 0))                      */
  DMX_ST_WMEAN_SQNORM = 10,/* sum_k b_k q_k / B                                            */
  DMX_ST_FLAGS = 11,       /* bit mask stored as a float, DMX_FLAG_*                       */
  DMX_ST_HDR = 16          /* 12..15 reserved (0); then q_k [K], V_s [S], N_s [S]          */
};
/* V_s = (sum_{j in s} sum_k b_k (x_kj-g_j)^2)/(K-1): segment s's additive share of
 * tr(Sigma)^ (0 if K == 1).  N_s = sum_{j in s} g_j^2.  Empty segments give 0. */

enum {
  DMX_FLAG_NONFINITE = 1,  /* some q_k, |a|^2 or A is not finite as fp32                   */
  DMX_FLAG_G2_NONPOS = 2,  /* |G|^2^ <= 0 (or NaN): gns reported as 0                      */
  DMX_FLAG_COS_UNDEF = 4,  /* A == 0 or |a|^2 == 0 (first step): cosine reported as 0      */
  DMX_FLAG_SINGLE = 8,     /* K == 1: no across-worker variance                            */
  DMX_FLAG_INTERNAL = 16,  /* a bounded wait inside the kernel ran out; results invalid    */
  DMX_FLAG_BOUNDS = 32     /* checked build only: an index into the tables or the scratch was
                              out of range and the access was skipped; results invalid     */
};

/*
 * dmx_create — validate (K, P, segment table), choose the launch configuration for the
 * current CUDA device, build the device-side tables and allocate the reduction scratch.
 *   K            number of workers, 1..DMX_MAX_WORKERS
 *   P            number of parameters, 1..DMX_MAX_PARAMS-1
 *   seg_offsets  HOST, S+1 entries: o[0]=0 <= o[1] <= ... <= o[S]=P; segment s is
 *                [o[s], o[s+1]); zero-length segments allowed; the table is copied
 *   S            number of segments, 1..DMX_MAX_SEGMENTS
 *   grad_dtype   DMX_F32 or DMX_BF16 (params, momentum, prev_agg, out_state are fp32)
 *   out          HOST, receives the handle
 * Errors: DMX_ERR_ARG, DMX_ERR_SEGMENTS, DMX_ERR_NOMEM, DMX_ERR_CUDA. Synchronous. On any error
 * everything allocated so far is released and *out is NULL.
 * For tests of that clean-up: with the environment variable DMX_TEST_FAIL_ALLOC=n the n-th
 * allocation of a create call (counted from 1, the handle structure first, then the device
 * buffers) is refused on the host as if memory had run out; no device call is made for it.
 * dmx_agg_create honours the same variable.
 */
int dmx_create(int K, int64_t P, const int64_t* seg_offsets, int S, int grad_dtype,
               dmx_handle** out);

/* 16 + K + 2*S, or DMX_ERR_HANDLE. */
int dmx_state_len(const dmx_handle* h);

/*
 * dmx_step — one iteration: aggregate, statistics, SGD-momentum update, state vector.
 *   grad_ptrs    HOST array of K DEVICE pointers; each addresses P elements of grad_dtype,
 *                16-byte aligned, read only
 *   batch_sizes  HOST array of K ints, each >= 1
 *   params       DEVICE, P fp32, 16-byte aligned, updated in place: theta - lr*m'
 *   momentum     DEVICE, P fp32, 16-byte aligned, updated in place: m' = beta*m + g
 *   lr, beta     learning rate and momentum coefficient (used as fp32)
 *   prev_agg     DEVICE, P fp32, 16-byte aligned; in: the previous step's aggregate
 *                (zeros before the first step); out: this step's aggregate g
 *   out_state    DEVICE, dmx_state_len(h) fp32, 4-byte aligned, fully overwritten
 *   cuda_stream  a cudaStream_t passed as void*; NULL = the legacy default stream
 * Buffers stay owned by the caller and must stay alive and untouched until the stream has
 * passed the step. params, momentum, prev_agg, out_state and the gradient buffers must be
 * pairwise disjoint (checked by address range; gradient buffers may alias one another).
 * Argument errors return before anything is enqueued: DMX_ERR_HANDLE, DMX_ERR_ARG,
 * DMX_ERR_BATCH, DMX_ERR_ALIGN; a failed launch returns DMX_ERR_CUDA.
 * Data problems (non-finite inputs, zero norms, |G|^2^ <= 0) are not errors: they set
 * bits in out_state[DMX_ST_FLAGS].
 */
int dmx_step(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes,
             float* params, float* momentum, float lr, float beta, float* prev_agg,
             float* out_state, void* cuda_stream);

/*
 * dmx_step_adam — the same pass with the Adam update in place of SGD with momentum (the paper
 * evaluates both optimizers, Section "Workloads and Datasets", and its state vector carries
 * sigma_norm and sigma^2_norm when the optimizer is adaptive, Section "State representation"). With g the
 * aggregate (Kingma & Ba 2015, Algorithm 1, bias-corrected form):
 *   m' = beta1 m + (1-beta1) g          v' = beta2 v + (1-beta2) g^2
 *   mhat = m' / (1-beta1^t)             vhat = v' / (1-beta2^t)
 *   theta' = theta - lr * mhat / (sqrt(vhat) + eps)          prev_agg' = g
 *   first_moment, second_moment   DEVICE, P fp32 each, 16-byte aligned, updated in place
 *   t                             1-based step count of this call (bias correction), >= 1
 *   0 <= beta1, beta2 < 1, eps >= 0, else DMX_ERR_ARG
 * Everything else (arguments, errors, asynchrony, statistics) is as dmx_step. out_state has the
 * same layout; three of its reserved entries carry the optimizer-normalised gradient statistics,
 * with ghat_j = g_j / (sqrt(vhat_j) + eps), the aggregate in units of Adam's running scale:
 *   out_state[12] = mean_j ghat_j     out_state[13] = var_j ghat_j (population variance over
 *   the P parameters)                 out_state[14] = sqrt(max(out_state[13], 0))
 * (dmx_step leaves 12..15 at 0.) This reading of the gradient variance and standard deviation
 * normalized for an adaptive optimizer is this library's: the paper gives no formula.
 */
int dmx_step_adam(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes,
                  float* params, float* first_moment, float* second_moment, float lr, float beta1,
                  float beta2, float eps, int64_t t, float* prev_agg, float* out_state,
                  void* cuda_stream);
enum { DMX_ST_ADAM_GHAT_MEAN = 12, DMX_ST_ADAM_GHAT_VAR = 13, DMX_ST_ADAM_GHAT_STD = 14 };

/*
 * Sharding one problem by parameter range (several GPUs, or several passes on one).
 * Every output of the step is either per parameter or a sum over parameters, so a problem splits
 * by parameter range with one small exchange: shard r owns elements [lo, hi) of all K gradient
 * buffers and of params/momentum/prev_agg, runs the same fused pass on them, and emits its raw
 * fp64 sums; the shards' sums are added (an all-reduce of K + 5 + 2 S doubles: the one exchange
 * step, e.g. NCCL over NVLink), and the state vector is derived from the total. This mirrors
 * the paper's scaling of the worker loop over 8 to 32 nodes (Section "Scalability of DYNAMIX"); the
 * paper has no formula for it. In a cluster where worker k is GPU k, the gradient shards come from
 * a reduce-scatter-like exchange that leaves every GPU with all workers' values of its range.
 *
 *   dmx_shard_range     HOST only. [lo, hi) of shard `shard` of `nshards`: boundaries on multiples
 *                       of 1024 elements (pointer alignment survives), the last shard ends at P;
 *                       a shard may be empty (lo == hi) when P is small: skip it.
 *   dmx_shard_segments  HOST only. The shard's own segment table (S+1 entries, written to
 *                       shard_offsets): the problem's table clipped to [lo, hi) and shifted by lo;
 *                       segments outside the shard become empty. Create the shard's handle with
 *                       dmx_create(K, hi - lo, shard_offsets, S, dtype): S and the state layout
 *                       stay those of the whole problem.
 *   dmx_partials_len    K + 5 + 2 S.
 *   dmx_step_partial, dmx_step_adam_partial
 *                       as dmx_step / dmx_step_adam on the shard's buffers (pointers to element lo),
 *                       but instead of out_state they write `partials` (DEVICE, dmx_partials_len
 *                       doubles, 8-byte aligned): q_k [K] in the caller's worker order, <g,a>, |a|^2,
 *                       Adam's sum and sum of squares of ghat (0 for SGD), Vraw_s [S] (before the
 *                       division by K-1), N_s [S], and an error word (1 if a bounded wait inside
 *                       the kernel ran out, plus 65536 if the checked build found an index out
 *                       of range; added over the shards like the rest).
 *   dmx_finalize_partials
 *                       batch_sizes: HOST, K ints; partials: DEVICE, the entry-wise sum over all
 *                       shards; P_total: the whole problem's parameter count (Adam's mean); writes
 *                       out_state (DEVICE, 16 + K + 2 S fp32) exactly as dmx_step defines it.
 *                       Asynchronous, one small launch.
 * Errors as dmx_step; DMX_ERR_SEGMENTS for a bad table or a range outside it.
 */
int dmx_shard_range(int64_t P, int nshards, int shard, int64_t* lo, int64_t* hi);
int dmx_shard_segments(const int64_t* seg_offsets, int S, int64_t lo, int64_t hi, int64_t* shard_offsets);
int dmx_partials_len(const dmx_handle* h);
int dmx_step_partial(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
                     float* momentum, float lr, float beta, float* prev_agg, double* partials,
                     void* cuda_stream);
int dmx_step_adam_partial(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes,
                          float* params, float* first_moment, float* second_moment, float lr, float beta1,
                          float beta2, float eps, int64_t t, float* prev_agg, double* partials,
                          void* cuda_stream);
int dmx_finalize_partials(int K, int S, const int32_t* batch_sizes, const double* partials, int adam,
                          int64_t P_total, float* out_state, void* cuda_stream);

/*
 * dmx_step_host — the same step for a caller whose gradients sit in HOST memory (the end-to-end
 * form of Algorithm 1's worker loop on one machine: gradients arrive from the workers' side of
 * the bus, the model state stays resident on the GPU).
 *   host_grad_ptrs  HOST array of K HOST pointers (pinned memory for full copy speed), each P
 *                   elements of grad_dtype
 *   staging_ptrs    HOST array of K DEVICE pointers, caller-owned staging buffers of P elements
 *                   each, 16-byte aligned; they receive the copies and feed the step
 *   out_state_dev   DEVICE, as out_state of dmx_step
 *   out_state_host  HOST, dmx_state_len(h) fp32; filled before the call returns
 * Enqueues K host-to-device copies, the step, and the device-to-host copy of the state vector
 * on the stream, then waits for the stream (so this call, unlike dmx_step, is synchronous).
 * Other arguments and errors as dmx_step; a failed copy returns DMX_ERR_CUDA.
 */
int dmx_step_host(dmx_handle* h, const void* const* host_grad_ptrs, void* const* staging_ptrs,
                  const int32_t* batch_sizes, float* params, float* momentum, float lr, float beta,
                  float* prev_agg, float* out_state_dev, float* out_state_host, void* cuda_stream);

/*
 * Per-kernel device timing of the steps of a handle (for benchmarks; off by default).
 * With profiling on, each dmx_step records CUDA events on its stream before the fused pass,
 * between the two kernels and after finalize. dmx_get_profile waits for the last step's
 * events and returns the two durations in milliseconds. Errors: DMX_ERR_HANDLE,
 * DMX_ERR_ARG (no step recorded, or profiling off), DMX_ERR_CUDA.
 * For timeline tools every step is also bracketed by NVTX ranges on the host ("dmx_step" or
 * "dmx_step_adam", with "dmx fused pass" and "dmx finalize" inside); they cost a pointer test
 * when no tool is attached.
 */
int dmx_set_profiling(dmx_handle* h, int on);
int dmx_get_profile(dmx_handle* h, float* fused_ms, float* finalize_ms);

/* Number of kernels one dmx_step launches (2: fused pass, finalize). */
int dmx_launches_per_step(const dmx_handle* h);

/* Sizes of a handle's launch plan, for inspection and tests: CTAs of the fused pass, chunks of
 * its work list, (V, N) partial-sum slots. Any pointer may be NULL. DMX_ERR_HANDLE or DMX_OK. */
int dmx_scratch_info(const dmx_handle* h, int* grid, int* nchunks, int* nslots);

/*
 * Checks of the library's own machinery (the paper has no counterpart; robustness is one of its
 * stated requirements, and these are how this library shows it without ever faulting a GPU).
 *
 * dmx_check_guards — every scratch array a handle's kernels write lies between two guard regions
 *   filled with a fixed word by dmx_create. This reads them back (synchronous copies; call it when
 *   no step of the handle is running) and returns DMX_OK, or DMX_ERR_GUARD if a word has changed,
 *   i.e. some kernel wrote just outside its array.
 *
 * dmx_selftest_wait — every wait inside the fused pass is bounded: after a fixed number of polls
 *   it gives up, raises the handle's error word and the CTA drains; the step's state vector then
 *   carries DMX_FLAG_INTERNAL and the word is cleared for the next step. This launches one warp
 *   that waits, with a budget of `polls` (1..2^24; the fused pass itself uses 2^18, about one
 *   second on B200 at 4 us per unsuccessful poll) polls, on a barrier that nothing will ever
 *   complete (no copy in flight, nobody to arrive): the wait must run out. *timed_out (HOST)
 *   receives 1 if it did; *waited_ms (HOST) the time the warp spent waiting, by the GPU's timer.
 *   The handle's error word is raised exactly as by a failed wait in a step: the next step of the
 *   handle reports DMX_FLAG_INTERNAL (its other outputs are valid) and clears it. Synchronous.
 *   Errors: DMX_ERR_HANDLE, DMX_ERR_ARG, DMX_ERR_NOMEM, DMX_ERR_CUDA.
 */
int dmx_check_guards(dmx_handle* h);
int dmx_selftest_wait(dmx_handle* h, uint32_t polls, int* timed_out, double* waited_ms, void* cuda_stream);

/*
 * dmx_plan_chunks — the work list dmx_create builds for the fused pass (host only: no CUDA call,
 * no device needed). For inspection and for tests of the planning logic.
 * The P parameters are cut into tiles of tile_elems elements (the last may be ragged); tiles are
 * taken in groups of *group_tiles consecutive tiles; chunk c consists of num_tiles[c] tiles:
 * tile i of the chunk is first_tile[c] + (i / G) * group_stride[c] + i % G with G = *group_tiles.
 * Every tile belongs to exactly one chunk. The fused kernel's CTAs draw chunks in list order
 * (CTA b starts with chunk b), so the list's order is the schedule: full waves first, shrinking
 * waves towards the end, and the chunk holding a ragged last tile moved to the front.
 *   resident_ctas   CTAs the device runs at once (SM count x CTAs per SM); *grid receives the
 *                   number of CTAs the kernel is launched with
 *   first_tile, num_tiles, group_stride   HOST, capacity entries each (may be NULL with capacity 0)
 * Returns the number of chunks (the arrays are filled only if capacity is at least that), or
 * DMX_ERR_ARG. The tuning variables dmx_create reads (DMX_TILE_GROUP, DMX_CHUNK_TILES,
 * DMX_MIN_CHUNK_KB) apply here too.
 */
int dmx_plan_chunks(int64_t P, int K, int grad_dtype, int tile_elems, int resident_ctas,
                    int32_t* first_tile, int32_t* num_tiles, int32_t* group_stride, int capacity,
                    int* group_tiles, int* grid);

/*
 * Window statistics of the state vector over k consecutive steps, kept on the device.
 * The controller acts on metrics aggregated over k iterations (Section "System architecture";
 * Section "State representation": state vectors are built from metrics collected every k
 * iterations, as means and standard deviations); with this the host reads one vector per
 * window instead of one per step.
 *   dmx_agg_create   state_len = dmx_state_len(h) (> DMX_ST_FLAGS), k >= 1; allocates two fp64
 *                    vectors on the current device
 *   dmx_agg_push     out_state: DEVICE, state_len fp32, as written by a step (enqueue the push on
 *                    the step's stream, after it); window_out: DEVICE, 2*state_len fp32. On every
 *                    k-th push window_out receives, per entry i over the window's k vectors,
 *                    mean (at i) and population standard deviation sqrt(sum (x-mean)^2 / k) (at
 *                    state_len + i), and the window restarts; entry DMX_ST_FLAGS gets the OR of
 *                    the k flag words and spread 0. Other pushes leave window_out untouched.
 *                    *emitted (HOST, may be NULL) is set to 1 on the pushes that write, else 0.
 *                    Asynchronous, no allocation. The position inside the window is counted on the
 *                    host, by call (which is why *emitted is known when the call returns, without
 *                    waiting for the device): a handle's pushes must be issued one after the other
 *                    (not concurrently from several threads), in the order of the steps, and on
 *                    one stream, so that the device executes them in that same order.
 * Errors: DMX_ERR_ARG, DMX_ERR_NOMEM, DMX_ERR_HANDLE, DMX_ERR_CUDA.
 */
typedef struct dmx_agg dmx_agg;
int dmx_agg_create(int state_len, int k, dmx_agg** out);
int dmx_agg_push(dmx_agg* a, const float* out_state, float* window_out, int* emitted, void* cuda_stream);
int dmx_agg_destroy(dmx_agg* a);

/*
 * dmx_ctl_decide — the controller's decision at the end of an adjustment cycle, on the device
 * (Algorithm 1, the loops after the k training iterations: build each worker's state vector,
 * evaluate the policy, apply the action within the batch-size limits, compute the reward).
 * What the paper fixes: the action set {-100, -25, 0, +25, +100} and the update
 * x_i <- max(min(x_i + a_i, x_max), x_min) (Section "Action space and batch size adjustment"),
 * and the reward (Section "Reward function design")
 *   r_i = Abar_i + alpha*max(0, dA_i) - beta_t*T_iter,i - delta*(log2 x_i - 5) - eta*(sigma2_norm + sigma_norm)
 * with x_i the batch size used during the cycle; eta = 0 gives the SGD form. What it leaves open,
 * and this library defines: the layout of the state vector and the policy network.
 *
 *   K, M, H        workers (1..DMX_MAX_WORKERS); caller-supplied metrics per worker
 *                  (0..DMX_CTL_MAX_AUX: accuracy, accuracy gain, iteration time, network and system
 *                  figures); hidden width of the policy network (1..DMX_CTL_MAX_HIDDEN)
 *   state_len      length of the step's state vector (>= DMX_ST_HDR + K)
 *   window         DEVICE, 2*state_len fp32: window means then deviations, as dmx_agg_push emits
 *   aux            DEVICE, K x M fp32 row-major (may be NULL when M == 0)
 *   batch          DEVICE, K int32: batch sizes used during the cycle (each >= 1)
 *   weights        DEVICE, dmx_ctl_num_weights(M, H) fp32, row-major, in this order:
 *                  W1 (H x F), c1 (H), W2 (H x H), c2 (H), W3 (5 x H), c3 (5), F = dmx_ctl_num_features(M)
 *   col_acc, col_gain, col_titer   columns of aux holding Abar, dA, T_iter; -1 leaves the term out
 *   alpha, beta_t, delta, eta      reward coefficients
 *   b_min, b_max   batch-size limits (the paper uses 32 and 1024), 1 <= b_min <= b_max
 *   uniforms       DEVICE, K fp32 in [0,1), or NULL. NULL: the action with the largest logit (lowest
 *                  index on ties). Otherwise the action is drawn from softmax(logits): the smallest a
 *                  whose cumulative probability exceeds uniforms[i] (the caller owns the generator)
 *   next_batch     DEVICE out, K int32     action   DEVICE out, K int32 (index 0..4 into the action set)
 *   reward         DEVICE out, K fp32      logits   DEVICE out, K x 5 fp32
 *   features       DEVICE out, K x F fp32, or NULL
 *
 * State vector of worker i (F = M + 9 entries), with mean/dev the two halves of `window`:
 *   aux[i][0..M), log2 x_i - 5, x_i*K / mean[B_TOTAL], mean[worker_sqnorm i] / mean[WMEAN_SQNORM],
 *   mean[SIGMA_NORM], mean[SIGMA2_NORM], dev[SIGMA_NORM], mean[COS_PREV], dev[COS_PREV],
 *   log2(1 + max(mean[GNS], 0) / mean[B_TOTAL])          (ratios with a zero denominator give 0)
 * Policy: logits = W3 tanh(W2 tanh(W1 s + c1) + c2) + c3. Arithmetic is fp64, stored as fp32; the
 * action is chosen from the fp32 logits as emitted.
 * Asynchronous, one launch, no allocation, no host-device copy. Errors: DMX_ERR_ARG, DMX_ERR_CUDA.
 */
#define DMX_CTL_ACTIONS 5
#define DMX_CTL_MAX_AUX 32
#define DMX_CTL_MAX_HIDDEN 256
#define DMX_CTL_LOCAL_EXTRA 3
#define DMX_CTL_GLOBAL_FEATURES 6
int dmx_ctl_num_features(int M);          /* M + 9, or DMX_ERR_ARG */
int64_t dmx_ctl_num_weights(int M, int H);  /* H*F + H + H*H + H + 5*H + 5, or DMX_ERR_ARG */
int dmx_ctl_decide(int K, int M, int H, int state_len, const float* window, const float* aux,
                   const int32_t* batch, const float* weights, int col_acc, int col_gain, int col_titer,
                   float alpha, float beta_t, float delta, float eta, int b_min, int b_max,
                   const float* uniforms, int32_t* next_batch, int32_t* action, float* reward,
                   float* logits, float* features, void* cuda_stream);

/*
 * dmx_step_static — the same step without a handle and without any allocation.
 * (The paper has no counterpart: this entry point exists for the library's callers only.)
 *
 * For callers that cannot allocate device memory at the point where they need the step:
 * code running under an allocator or memory pool that must account for every byte, a
 * latency-critical loop that cannot afford the device-wide synchronisation a cudaMalloc may
 * bring, or a process whose memory budget is spoken for. dmx_create allocates tables and
 * reduction scratch; this call uses neither. Its reduction scratch is a fixed array of
 * DMX_STATIC_SCRATCH_BYTES inside the library's device image: every GPU on which the library
 * is loaded holds that array until the process exits.
 *
 *   K, P, seg_offsets, S, grad_dtype   as dmx_create, but S <= DMX_STATIC_MAX_SEGMENTS.
 *                                      seg_offsets is HOST memory. It is validated during the call
 *                                      and copied to the device by an asynchronous copy on the
 *                                      stream: from pageable memory the runtime has taken its copy
 *                                      when the call returns; from pinned memory the table must
 *                                      stay unchanged until the stream has passed the call (and
 *                                      for as long as a captured copy of the call may be replayed)
 *   grad_ptrs ... cuda_stream          as dmx_step
 *
 * It calls no cudaMalloc, cudaFree or other allocating routine; the caller still provides
 * every input and output buffer. It runs the plain-load kernel with one contiguous range of
 * tiles per CTA, so it is slower than dmx_step, and its sums are taken in a different order:
 * results agree with dmx_step to rounding, not bit for bit.
 *
 * The first call on each device looks up the array's device address (with that device
 * current). Make that first call outside any stream capture.
 * All calls on a GPU share the one array, and it keeps what the previous call left: the
 * kernels clear what they need at the start of each call, and two calls that overlap on
 * the same GPU (different streams, different threads) race on it. Keep calls on one GPU in
 * stream order.
 * Errors: as dmx_create and dmx_step, and DMX_ERR_LIMIT when S exceeds
 * DMX_STATIC_MAX_SEGMENTS or the partial sums of this device's grid would not fit in the array.
 */
#define DMX_STATIC_MAX_SEGMENTS 512
#define DMX_STATIC_SCRATCH_BYTES (1 << 20)
int dmx_step_static(int K, int64_t P, const int64_t* seg_offsets, int S, int grad_dtype,
                    const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
                    float* momentum, float lr, float beta, float* prev_agg, float* out_state,
                    void* cuda_stream);

/* Frees the tables and the scratch. NULL is accepted; a handle that is not live (destroyed
 * already) gives DMX_ERR_HANDLE. The caller makes sure no step of this handle is still running. */
int dmx_destroy(dmx_handle* h);

/* Static, NUL-terminated description of a return code. */
const char* dmx_strerror(int code);

/* The cudaError_t (as int) of the last failed CUDA call made by this library on the
 * calling thread, 0 if none. */
int dmx_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DMX_H_ */
