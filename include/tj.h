/*
 * tj.h -- C ABI of the B200 (sm_100a) sample production/consumption library.
 *
 * The library runs, on ONE GPU and one CUDA stream (or two: tj_set_learner_stream), the data-parallel hot path of
 * a TianJi-style actor/buffer/learner pipeline (arXiv 2502.20190):
 *
 *   actor   (Sec. 3.1, actor loop; Algorithm 1 tasks 1-2):
 *           observation -> policy MLP -> epsilon-greedy / categorical action ->
 *           vectorised environment step -> version-tagged trajectory record
 *   buffer  (Sec. 3.1, buffer loop; dependency III relaxed into an asynchronous
 *           hand-over): a replay ring of (s, a, r, s', done, version) records, or
 *           rollout segments for the on-policy case
 *   learner (Sec. 3.1, learner loop; Sec. 3.3 and Eq. 2-3 for staleness control):
 *           staleness-bounded minibatch sampling, gather, online/target forward,
 *           TD target and Huber error (Algorithm 1, TD-error line); GAE for the
 *           on-policy case (Table 2: gae 0.95, gamma 0.99); the parameter update
 *           (Algorithm 1, update line) as an FP32 SGD / Adam step on that loss, and
 *           PPO's clipped surrogate for the on-policy case (Sec. 4.1)
 *   weights (dependency I relaxed): the learner publishes a new parameter version,
 *           the actor picks up the newest one at its next call.
 *
 * Conventions
 *   - Every function returns a tj_status (0 = OK, negative = error).  Nothing
 *     throws, aborts or prints.  tj_last_error() gives a readable message.
 *   - All device work is enqueued on the stream given to tj_create (the learner-side
 *     calls on the stream given to tj_set_learner_stream, if any, ordered against the
 *     actor's by events); calls are asynchronous with respect to the host unless
 *     stated otherwise, and take effect in host call order.
 *   - OWNERSHIP: the caller owns every byte of device memory.  tj_query_workspace
 *     reports how much the context needs, tj_create carves the caller's buffer.
 *     The library never calls cudaMalloc/cudaFree.  tj_ctx is a small host object.
 *   - Pointers are DEVICE pointers unless the parameter name starts with host_ or
 *     the comment says "host".  Arrays are dense and row-major.
 *   - A context is not thread-safe; distinct contexts are independent.
 *   - Host-detectable errors are returned before anything is enqueued.
 */
#ifndef TJ_H
#define TJ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tj_ctx tj_ctx;

typedef enum {
  TJ_OK = 0,
  TJ_ERR_INVALID_ARG = -1,   /* null pointer, negative size, wrong blob length ... */
  TJ_ERR_CONFIG = -2,        /* inconsistent tj_config */
  TJ_ERR_WORKSPACE = -3,     /* workspace too small or misaligned */
  TJ_ERR_CUDA = -4,          /* a CUDA runtime call failed; see tj_last_error */
  TJ_ERR_NO_WEIGHTS = -5,    /* actor or learner called before the first publish */
  TJ_ERR_WARMUP = -6,        /* fewer resident records than cfg.warmup (Table 2: buffer warmup size) */
  TJ_ERR_STARVED = -7,       /* nothing eligible: the consumer is ahead of the producer (Eq. 3: TR_L ~ TR_A) */
  TJ_ERR_STALE_SEGMENT = -8, /* tj_segment_check: the producer has begun to overwrite the segment's slot */
  TJ_ERR_TIMEOUT = -9,       /* tj_stats: a kernel's bounded wait ran out (device_error holds the code); tj_wait: time limit */
  TJ_ERR_UNSUPPORTED = -10   /* valid request this build does not implement */
} tj_status;

enum { TJ_ENV_CARTPOLE = 0, TJ_ENV_ACROBOT = 1, TJ_ENV_LINGAUSS = 2 };
enum { TJ_POLICY_EPS_GREEDY = 0, TJ_POLICY_CATEGORICAL = 1 };
enum { TJ_W_FP32 = 0,      /* FP32 FMA in one fixed rounding order: outputs (and actions) reproducible bit for bit */
       TJ_W_BF16 = 1,      /* weight matrices rounded to bfloat16, tensor cores, FP32 accumulation: 2e-2 */
       TJ_W_FP32_TC = 2 }; /* FP32 weights; the actor's hidden x hidden layer on the tensor cores as three products of split
                              operands (the role a 3 x TF32 product plays, here with FP16 parts at twice that rate; about
                              2^-22 per term): outputs within 1e-5 of TJ_W_FP32's, actions equal wherever the top-2 gap
                              exceeds that.  CartPole / Acrobot, hidden 64 / 128 / 192 / 256.  First-layer activations must
                              stay below 4,094 (16 x that is FP16's range); a pass that sees a larger one latches
                              device_error 5 and its outputs are meaningless.  tj_td_error runs its two
                              forwards the same way (same tolerance); tj_td_error_static and the parameter updates
                              use the FP32 kernels. */
/* kernel classes reported by tj_stats (Sec. 3.3: performance analysis measures the production and the
 * consumption side separately) */
enum { TJ_K_ACTOR_FUSED = 0,  /* MLP + selection + env step + insert in one kernel (FP32 path, or the fused tensor-core actor) */
       TJ_K_MLP_TENSOR = 1,   /* tensor-core MLP forward alone (the learner's two forwards; the actor's where it is not fused) */
       TJ_K_ENV = 2,          /* selection + env step + insert fed by the tensor-core MLP */
       TJ_K_SAMPLE = 3,       /* eligible list + sample + gather */
       TJ_K_TD = 4,           /* TD error (FP32 forward, or the elementwise pass after tensor-core forwards) */
       TJ_K_PUBLISH = 5, TJ_K_GAE = 6,
       TJ_K_SGD = 7,          /* learner update: forward with kept activations, backward, parameter update */
       TJ_KERNEL_CLASSES = 8 };

/* Configuration (App. B: one configuration with distribution / training / model / environment groups). */
typedef struct {
  uint32_t struct_size;          /* = sizeof(tj_config); lets the struct grow */
  int32_t device;                /* CUDA device ordinal the workspace lives on */
  /* environment group */
  int32_t env_kind;              /* TJ_ENV_* */
  int32_t n_envs;                /* N, environments stepped together */
  int32_t obs_dim;               /* D: 4 CartPole, 6 Acrobot, multiple of 4 (<= 128) LinGauss */
  int32_t n_actions;             /* A: 2 CartPole, 3 Acrobot, <= 64 LinGauss */
  int32_t max_episode_steps;     /* 0 = env default (500 / 500 / 200) */
  float lg_done_norm;            /* LinGauss: terminate when ||s'|| exceeds this (4) */
  float lg_noise_std;            /* LinGauss: noise scale (0.01) */
  const float *host_lg_A;        /* LinGauss: A [D][D], HOST pointer, copied at create */
  const float *host_lg_B;        /* LinGauss: B [A][D], HOST pointer, copied at create */
  /* model group */
  int32_t hidden;                /* H, width of both hidden ReLU layers (1..768) */
  int32_t policy_kind;           /* TJ_POLICY_*: Q head, or softmax head + value head */
  int32_t weight_dtype;          /* TJ_W_* */
  float epsilon;                 /* exploration rate (eps-greedy) */
  uint64_t seed;                 /* Philox key */
  /* training / distribution group */
  int64_t replay_capacity;       /* C, multiple of n_envs; 0 => on-policy segment mode */
  int32_t minibatch;             /* B */
  int32_t staleness_bound;       /* S: a record is eligible iff learner_version - record_version <= S */
  int32_t warmup;                /* minimum resident records before sampling */
  int32_t rollout_len;           /* T (segment mode) */
  int32_t n_segments;            /* segment slots (segment mode) */
  int32_t target_sync_interval;  /* learner steps between target-network refreshes (Table 2) */
  float gamma, huber_delta, gae_lambda;
} tj_config;

/* A gathered minibatch: caller-owned device arrays, n rows each. */
typedef struct {
  int32_t n;
  float *obs;        /* [n][D] */
  int32_t *act;      /* [n] */
  float *rew;        /* [n] */
  float *next_obs;   /* [n][D] */
  int32_t *done;     /* [n] */
  int32_t *ver;      /* [n] policy version that produced the record */
} tj_batch;

/* A rollout segment: a view into the context's workspace, valid until the producer reuses the slot. */
typedef struct {
  int32_t T, N;
  int64_t version;   /* policy version in force when the segment's first step ran */
  const float *obs;      /* [T][N][D] */
  const int32_t *act;    /* [T][N] */
  const float *rew;      /* [T][N] */
  const uint8_t *done;   /* [T][N] */
  const float *logp;     /* [T][N] */
  const float *val;      /* [T+1][N]; row T is the bootstrap value of the state after the last step */
} tj_segment;

/* Environment state and counters (views into the workspace / values to restore). */
typedef struct {
  float *state;          /* [N][S_d], S_d = 4 (CartPole, Acrobot) or D (LinGauss) */
  int32_t *ep_step;      /* [N] steps taken in the running episode */
  uint64_t cursor;       /* transitions ever written to the ring */
  int64_t t;             /* actor steps taken so far (per env) */
  int64_t k;             /* learner steps taken so far */
  int64_t actor_version, learner_version;
} tj_state_view;

/* Production/consumption and staleness statistics (Eq. 2-3; Table 1 columns). */
typedef struct {
  int64_t produced;             /* transitions written */
  int64_t consumed;             /* transitions handed to the learner */
  int64_t dropped_stale;        /* summed over sample calls: resident records outside the bound at that call (a record
                                   that stays resident and stale is counted by every call that passes it over);
                                   segment mode: transitions of segments dropped for staleness, each once */
  int64_t dropped_overwritten;  /* segment transitions overwritten before they were consumed */
  int64_t starved_calls;
  int64_t actor_version, learner_version, actor_steps, learner_steps;
  int64_t max_sampled_staleness;
  int64_t episodes_finished;
  double return_sum;            /* sum of the returns of finished episodes */
  int64_t staleness_hist[33];   /* sampled staleness 0..31, last bin = 32 and more */
  int64_t device_error;         /* 0, or a code latched by a kernel's own bounded wait or bounds check */
  int64_t kernel_launches;      /* kernels this context has launched since tj_create */
  /* Per kernel class, filled while profiling is on (tj_set_profiling): launches timed and their summed
   * duration in ms, from CUDA events recorded around each launch on the context's stream. */
  int64_t kernel_count[TJ_KERNEL_CLASSES];
  double kernel_ms[TJ_KERNEL_CLASSES];
} tj_stats_t;

/* Bytes (and alignment) of device memory a context with this configuration needs. */
int tj_query_workspace(const tj_config *cfg, size_t *bytes, size_t *align);

/* Build a context inside `workspace` (device memory, >= bytes, aligned as reported) on `cuda_stream`
 * (a cudaStream_t; NULL = the legacy default stream).  Seeds every environment from the reset stream.
 * Errors: INVALID_ARG, CONFIG, WORKSPACE, CUDA. */
int tj_create(const tj_config *cfg, void *workspace, size_t bytes, void *cuda_stream, tj_ctx **out);

/* Concurrent actor and learner (Sec. 3.1, Fig. 2: the actor, buffer and learner loops run side by side; dependencies I and
 * III become asynchronous hand-overs).  After this call the learner-side entry points -- tj_replay_sample, tj_td_error(_static),
 * tj_sgd_step, tj_adam_step, tj_ppo_step, tj_gae, tj_normalize, tj_segment_minibatch and tj_publish_weights -- enqueue on
 * `cuda_stream`, tj_actor_step stays on the stream given to tj_create, and the library orders the two with CUDA events at
 * the hand-overs only:
 *   - a sample (or a segment acquisition) waits for the actor launches enqueued before it (it reads their records);
 *   - an actor call waits for the sampler launched before it (ring blocks it may overwrite), for the last publish (it reads
 *     the newest parameters) and, in segment mode, for the learner calls enqueued before it;
 *   - a publish waits for the actor launches enqueued before it (they may still read the buffer it rewrites).
 * TD error and parameter updates therefore overlap with the actor steps the host enqueues after the sample.  Results depend
 * only on the host's call order, exactly as on one stream.  The caller's arrays passed to learner-side calls must be safe to
 * use on that stream.  NULL or the create stream switches back.  Synchronises both streams. */
int tj_set_learner_stream(tj_ctx *ctx, void *cuda_stream);

/* Host-side bounded wait: returns TJ_OK once everything enqueued on the actor stream (which = 0) or the learner stream
 * (which = 1) has finished, TJ_ERR_TIMEOUT if that takes longer than timeout_ms (nothing is cancelled; call again). */
int tj_wait(tj_ctx *ctx, int32_t which, int32_t timeout_ms);

/* Free the host object.  Does not touch the workspace.  Synchronises the stream. */
int tj_destroy(tj_ctx *ctx);

/* Learner -> actor hand-over of parameters (Sec. 3.1: the learner stores the model and a trigger decides
 * when to send it; dependency I as an asynchronous exchange).  `blob` holds FP32
 *   [W1 HxD, b1 H, W2 HxH, b2 H, W3 AxH, b3 A (, Wv 1xH, bv 1 when policy_kind = categorical)]
 * row-major (out x in); nbytes must match exactly.  on_device = 0: host pointer, copied with an asynchronous
 * host-to-device copy on the stream (pageable memory is staged before the call returns; pinned memory must stay
 * unchanged until the stream has passed the copy); 1: device pointer (read on the stream).  The new parameters become version+1 (returned in version_out)
 * and are what the actor uses from its next call and what the learner's online forward uses.  The target
 * network takes the same parameters on the first publish and then on the first publish after
 * target_sync_interval further learner steps.  With TJ_W_BF16 the weight matrices are rounded to bfloat16
 * (nearest even); biases stay FP32. */
int tj_publish_weights(tj_ctx *ctx, const void *blob, size_t nbytes, int32_t on_device, int64_t *version_out);

/* Actor: n_steps environment steps for all N environments (Algorithm 1: policy inference, then
 * simulation, then the trajectory tuple; Sec. 3.1 actor loop).  Per env e and global step t:
 *   logits = MLP(obs);  action from the ACTION Philox words of (e, t);  env step;  done = terminated or
 *   step limit;  record (obs, a, r, next_obs before reset, done, version) at ring slot (cursor + e) mod C
 *   (or into the running segment);  done envs are re-seeded from the RESET words of (e, t).
 * After each step cursor += N.  dbg_logits (nullable) receives [n_steps][N][A] network outputs.
 * Errors: INVALID_ARG, NO_WEIGHTS, CUDA. */
int tj_actor_step(tj_ctx *ctx, int32_t n_steps, float *dbg_logits);

/* Learner, step 1 (Sec. 3.1: loading trajectories; Sec. 3.3 / Eq. 2-3 / App. D.1: controlling sample
 * staleness).  E = valid slots with learner_version - version <= S in ascending slot order; draw j of
 * learner step k takes E[mulhi(x0, |E|)], x0 from the SAMPLE Philox words of (j, k); with replacement.
 * staleness_bound = -1 uses the configured S.  idx_out (nullable) receives the B slots; `out` arrays
 * receive the gathered rows bit for bit.  Errors: NO_WEIGHTS, WARMUP, STARVED (nothing enqueued, k unchanged). */
int tj_replay_sample(tj_ctx *ctx, int32_t staleness_bound, int32_t *idx_out, const tj_batch *out);

/* Learner, step 2, forward half (Algorithm 1: delta = r + gamma V(s') - V(s), here with a target network
 * and a done mask): q = Q_online(obs)[act]; q' = max_a Q_target(next_obs); y = r + gamma (1-done) q';
 * delta = y - q; Huber(delta; huber_delta).  td_out, huber_out: [n] (nullable); loss_mean_out: 1 float
 * (nullable), the mean Huber loss summed in a fixed order.  1 <= batch.n <= 1,048,576.  In a TJ_W_BF16 context both
 * forwards run on the tensor cores for every batch size (batches above 65,536 rows in chunks of that many rows).
 * Should a kernel's bounded wait for its staged parameters run out, the rows of that thread block and the loss are
 * NaN and device_error is latched (tj_stats). */
int tj_td_error(tj_ctx *ctx, const tj_batch *batch, float *td_out, float *huber_out, float *loss_mean_out);

/* The same computation as tj_td_error for callers that must not allocate and have no scratch to lend.
 * (The paper has no counterpart: this is a deployment convenience of this library.)
 *
 * Who this is for: code that runs where device allocation is off limits -- a latency-critical actor or
 * evaluation loop in which a cudaMalloc would synchronise the whole device and stall every stream, a process
 * that runs under a memory plan fixed at start-up, or a plug-in living inside another framework whose
 * allocator it may not call.  tj_td_error sums the per-block losses through scratch carved from the caller's
 * workspace; this variant keeps that scratch in a fixed 32 KB array inside the library image, so every GPU
 * that loads the library holds those 32 KB until the process exits.  It calls no cudaMalloc, no cudaFree and
 * no allocating library routine; inputs and outputs are still the caller's.
 *
 * Limits and rules:
 *   - at most 65,536 rows per call; a larger batch.n is refused with TJ_ERR_INVALID_ARG and a message naming
 *     the limit (split the batch or use tj_td_error);
 *   - the first call on each device looks up the array's device address (once per device; the context's device must
 *     be the current device, else TJ_ERR_INVALID_ARG).  Make that first call at set-up, before any stream capture
 *     is under way.  The look-up is guarded by a lock, so first calls from several threads (one context each) are safe;
 *   - while per-kernel timing is on (tj_set_profiling) the call is timed only if two of the context's CUDA events are
 *     free for reuse: it never creates one;
 *   - every call, from every context on the device, shares the one array.  Each call rewrites the part it
 *     reads, so nothing needs clearing between calls, but two calls that overlap on the GPU (different
 *     streams) race on it: keep them on one stream or order them with events;
 *   - in an FP32 context the results equal tj_td_error's (same kernels, same summation order); in a BF16 context this
 *     call still runs the FP32 kernels on the BF16-rounded weights, so it agrees with tj_td_error's tensor-core
 *     result within the BF16 tolerance only. */
int tj_td_error_static(tj_ctx *ctx, const tj_batch *batch, float *td_out, float *huber_out, float *loss_mean_out);

/* Learner, step 2, update half (Algorithm 1: theta <- theta + alpha * delta * grad V(s; theta)) as one minibatch
 * semi-gradient step on the mean Huber loss of tj_td_error:
 *   L = mean_j Huber(delta_j; huber_delta),  delta_j = r_j + gamma (1 - done_j) max_a Q(s'_j, a; theta_target) - Q(s_j, a_j; theta)
 *   theta <- theta - lr * dL/dtheta   (the target term is a constant; dHuber/ddelta = clip(delta, -huber_delta, huber_delta))
 * With huber_delta = inf, one row and theta_target = theta this is Algorithm 1's update line.
 * theta (in/out) and theta_target: device FP32 blobs in the tj_publish_weights layout, distinct buffers, owned by the
 * caller; nothing in the context changes -- publish theta afterwards to hand it to the actor.  batch.n <= the configured
 * minibatch.  loss_mean_out (nullable, device): the loss before the update.  FP32 arithmetic, every sum in a fixed order;
 * hidden-layer products with at least 96 tiles of 128 x 128 outputs (e.g. 8,192 rows x 512 units) run on the tensor cores
 * as three TF32 products of high / low operand parts with FP32 accumulation: up to 3 * 2^-22 per product instead of 2^-24.
 * In a BF16 context theta is the FP32 master copy: the update and its loss are FP32 all the same, the rounding to BF16
 * happens at tj_publish_weights (so this loss differs from tj_td_error's, which uses the published BF16 copy, by that
 * rounding).  TJ_ERR_UNSUPPORTED for segment mode and the categorical policy. */
int tj_sgd_step(tj_ctx *ctx, const tj_batch *batch, float lr, float *theta, const float *theta_target, float *loss_mean_out);

/* The same gradient through Adam (the optimiser of Table 2; Kingma & Ba 2015), step counter t >= 1:
 *   m <- beta1 m + (1 - beta1) g;  v <- beta2 v + (1 - beta2) g^2;
 *   theta <- theta - lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
 * m, v: device FP32 moment blobs in the layout of theta, owned and zero-initialised by the caller, updated in place.
 * Other arguments, limits and statuses as tj_sgd_step. */
int tj_adam_step(tj_ctx *ctx, const tj_batch *batch, float lr, float beta1, float beta2, float eps, int64_t t, float *theta,
                 const float *theta_target, float *m, float *v, float *loss_mean_out);

/* On-policy learner update: PPO's clipped surrogate (Schulman et al. 2017; the paper's on-policy algorithm, Sec. 4.1, with
 * Table 2's "gae" advantages) on the shared-trunk network with the categorical policy head and the value head:
 *   ratio_j = exp(log pi(a_j | s_j; theta) - logp_old_j)
 *   L = mean_j [ -min(ratio_j A_j, clip(ratio_j, 1 - clip_eps, 1 + clip_eps) A_j) + c_v / 2 (V(s_j) - R_j)^2 - c_e H(pi(. | s_j)) ]
 * followed by one Adam step on L (arguments as tj_adam_step).  theta, m, v: device FP32 blobs in the publish layout with the
 * value head ([W1, b1, W2, b2, W3, b3, Wv, bv]).  The batch arrays are device pointers owned by the caller; rows of a
 * segment (tj_segment_acquire) and of tj_gae's outputs can be passed as they lie: obs [n][obs_dim], the others [n].
 * stats_out (nullable, device, 5 floats): L, mean policy term, mean 0.5 (V - R)^2, mean entropy, fraction of rows where
 * the clipped term is the minimum -- all before the update.  batch.n <= the configured minibatch (4096 if none).
 * BF16 contexts: theta is the FP32 master copy, as for tj_sgd_step.
 * TJ_ERR_UNSUPPORTED unless the context is in segment mode with the categorical policy. */
typedef struct {
  int32_t n;
  const float *obs;
  const int32_t *act;
  const float *logp_old;
  const float *adv;
  const float *ret;
} tj_ppo_batch;
int tj_ppo_step(tj_ctx *ctx, const tj_ppo_batch *batch, float lr, float beta1, float beta2, float eps, int64_t t, float clip_eps,
                float c_v, float c_e, float *theta, float *m, float *v, float *stats_out);

/* Generalised advantage estimation over time-major arrays (Table 2: gae lambda, discount gamma):
 *   delta_t = r_t + gamma (1-d_t) V_{t+1} - V_t;  A_t = delta_t + gamma lambda (1-d_t) A_{t+1}, A_T = 0;
 *   R_t = A_t + V_t.   rew [T][N], val [T+1][N], done [T][N] -> adv [T][N], ret [T][N].
 * ctx supplies only the stream. */
int tj_gae(tj_ctx *ctx, const float *rew, const float *val, const uint8_t *done, int32_t T, int32_t N, float gamma,
           float lambda, float *adv_out, float *ret_out);

/* On-policy consumption (App. D.1: buffer = batch, staleness controlled by how far the learner has moved
 * on): the oldest complete, unconsumed segment whose version is at most S behind the learner; staler ones
 * are dropped and counted.  Errors: STARVED. */
int tj_segment_acquire(tj_ctx *ctx, tj_segment *out);

/* On-policy consumer (App. C, synchronous mode; Table 2: PPO's batch settings), the two steps between tj_gae and tj_ppo_step.
 *
 * tj_normalize: out_i = (x_i - mean) / (sqrt(var) + eps) with the mean and the population variance of all n entries
 * (advantages of one segment: mean 0, variance 1).  Both sums are taken in double in a fixed order, so the result is
 * reproducible.  x and out: device, n floats, may be the same array.  eps >= 0. */
int tj_normalize(tj_ctx *ctx, const float *x, int64_t n, float eps, float *out);

/* tj_segment_minibatch: rows of a segment in shuffled order.  Shuffle `shuffle_id` (one per epoch, say) is a keyed
 * bijection of the segment's R = T * N rows: position i takes row perm(i) = walk(F(i)), where F is a four-round balanced
 * Feistel network on 2 * hb bits (hb = half the bits of R - 1, rounded up, at least 1) whose round function is the first
 * Philox word of the SHUFFLE stream at (index = right half, step = shuffle_id, block = round), and walk applies F again
 * until the value is below R.  The call copies the rows at positions first .. first + out->n - 1 into dense arrays:
 * obs [n][obs_dim], act, logp_old (the segment's logp), adv, ret (from the caller's [T][N] arrays, e.g. tj_gae's outputs,
 * normalised or not) and, if row is not null, the source row indices.  Every position of 0 .. R - 1 occurs exactly once
 * over the minibatches of one shuffle.  Errors: INVALID_ARG (null arrays, positions outside the segment). */
typedef struct {
  int32_t n;
  float *obs;
  int32_t *act;
  float *logp_old;
  float *adv;
  float *ret;
  int32_t *row;      /* nullable */
} tj_ppo_minibatch;
int tj_segment_minibatch(tj_ctx *ctx, const tj_segment *seg, const float *adv, const float *ret, uint64_t shuffle_id, int64_t first,
                         const tj_ppo_minibatch *out);

/* Does a segment view handed out by tj_segment_acquire still show the segment it was acquired as?  TJ_OK while the
 * producer has not come round to its slot again; TJ_ERR_STALE_SEGMENT once a later segment has begun to fill the slot
 * (the consumer was lapped: what it reads from the view may be a mixture).  Host bookkeeping only, nothing is enqueued. */
int tj_segment_check(tj_ctx *ctx, const tj_segment *seg);

/* Views of the env state and the counters; no copy, no synchronisation. */
int tj_get_state(tj_ctx *ctx, tj_state_view *out);
/* Restore env state (device pointers, nullable = keep) and the t / k counters; versions are ignored.  The ring, its
 * per-block versions and the segment slots are not part of the view, so the counters that index them cannot move:
 * in ring mode `cursor` must equal the current cursor, in segment mode `t` must equal the current t; anything else
 * is refused with TJ_ERR_UNSUPPORTED and changes nothing. */
int tj_set_state(tj_ctx *ctx, const tj_state_view *in);

/* Counters (Eq. 2-3: produced vs consumed, sampled staleness).  Synchronises the stream.  Returns TJ_ERR_TIMEOUT,
 * with host_out filled all the same, when a kernel has latched device_error. */
int tj_stats(tj_ctx *ctx, tj_stats_t *host_out);

/* Turn per-kernel timing on or off.  While on, every launch is bracketed by two CUDA events on the context's
 * stream (a few microseconds of overhead per launch); tj_stats turns them into kernel_count / kernel_ms.
 * Turning it on resets the per-class figures. */
int tj_set_profiling(tj_ctx *ctx, int32_t on);

/* Views into the ring for inspection: records [C][2D+4] (obs, next_obs, act, rew, done, ver as 32-bit words)
 * and the per-block version summary [C/N]. */
int tj_ring_view(tj_ctx *ctx, const float **records, const int32_t **block_version, int32_t *record_words);

/* Measured FP32 fused-multiply-add rate of the context's device, in TFLOP/s (Sec. 3.3: resources are sized from measured
 * rates; this is the rate the FP32 policy kernels are held against).  Runs a register-only FMA loop on every SM five times
 * on the context's stream and reports the best; synchronises.  scratch: device memory of at least sm_count * 8 KiB (each
 * thread stores one word so that the loop cannot be optimised away); tflops_out: host.  About 10 ms of GPU time. */
int tj_calibrate_fp32(tj_ctx *ctx, float *scratch, size_t scratch_bytes, double *tflops_out);

const char *tj_last_error(const tj_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* TJ_H */
