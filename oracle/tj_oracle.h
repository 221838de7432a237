/*
 * tj_oracle.h -- plain CPU oracle for the sample production/consumption path
 * (actor rollout -> version-tagged replay ring -> staleness-bounded sampling ->
 * TD/Huber, and GAE for the on-policy case).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is slow on purpose: one environment, one
 * sample, one neuron at a time, in the order the definitions are stated, with no
 * blocking, fusion or reordering.  It shares no source, header, table or helper
 * with the CUDA library and must never be linked or called from the product
 * path; only the tests, the smoke check and the CPU-baseline timing use it.
 *
 * Precision.  Integer work (Philox, indices, versions, ring arithmetic) is exact.
 * Environment physics, TD/Huber and GAE are evaluated in double from the FP32
 * inputs and rounded to FP32 where the method stores FP32.  The FP32 policy MLP
 * is evaluated in one stated rounding order (bias first, then one fused
 * multiply-add per input in index order), so its outputs -- and the argmax taken
 * from them -- are reproducible bit for bit; a double-precision MLP sits beside
 * it to size tolerances.
 *
 * What each function follows (paper = arXiv 2502.20190):
 *   actor loop (inference -> action -> simulation -> trajectory): Algorithm 1, tasks 1-2; Sec. 3.1 actor loop
 *   replay ring + version tags (dependency III as an asynchronous hand-over): Sec. 3.1 buffer loop
 *   weight publish / versions (dependency I as an asynchronous hand-over):    Sec. 3.1 learner loop
 *   staleness-bounded sampling:                                               Sec. 3.3, Eq. 2-3, App. D.1
 *   TD error:                                                                 Algorithm 1, TD-error line
 *   GAE:                                                                      Table 2 (gae 0.95, gamma 0.99)
 * Environment dynamics, Philox4x32-10, Huber and GAE themselves are textbook
 * definitions the paper only names; they are restated in tj_oracle.c.
 *
 * Pinned by tests (CPU only): hand-worked CartPole step, Acrobot energy
 * conservation and RK4 order, Philox against an independent big-integer
 * restatement, MLP against a float64 library matmul, ring/sampler against brute
 * force, TD hand values, GAE closed forms, the shuffle as a bijection with uniform positions, the
 * normalisation's moments and hand values.  Unpinned: nothing.
 */
#ifndef TJ_ORACLE_H
#define TJ_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_ENV_CARTPOLE = 0, ORC_ENV_ACROBOT = 1, ORC_ENV_LINGAUSS = 2 };
enum { ORC_POLICY_EPS_GREEDY = 0, ORC_POLICY_CATEGORICAL = 1 };
enum { ORC_W_FP32 = 0, ORC_W_BF16 = 1 };
enum { ORC_STREAM_ACTION = 0, ORC_STREAM_RESET = 1, ORC_STREAM_NOISE = 2, ORC_STREAM_SAMPLE = 3, ORC_STREAM_SHUFFLE = 4 };
enum { ORC_OK = 0, ORC_ERR_ARG = -1, ORC_ERR_CONFIG = -2, ORC_ERR_NO_WEIGHTS = -5, ORC_ERR_WARMUP = -6,
       ORC_ERR_STARVED = -7 };

typedef struct {
  int32_t env_kind, n_envs, obs_dim, n_actions, hidden, policy_kind, weight_dtype;
  float epsilon;
  uint64_t seed;
  int64_t replay_capacity;        /* 0 => on-policy segment mode */
  int32_t minibatch, staleness_bound, warmup, rollout_len, target_sync_interval, n_segments;
  float gamma, huber_delta, gae_lambda;
  int32_t max_episode_steps;      /* 0 => env default (500 / 500 / 200) */
  float lg_done_norm;             /* LinGauss: terminate when ||s'|| exceeds this (4) */
  float lg_noise_std;             /* LinGauss: noise scale (0.01) */
  const float *lg_A, *lg_B;       /* LinGauss: A [D][D], B [n_actions][D], row-major */
} orc_config;

typedef struct {
  int64_t produced, consumed, dropped_stale, dropped_overwritten, starved_calls;
  int64_t actor_version, learner_version, actor_steps, learner_steps;
  int64_t max_sampled_staleness, episodes_finished;
  double return_sum;
  int64_t staleness_hist[33];
} orc_stats;

typedef struct {
  int32_t T, N;
  int64_t version;
  const float *obs;       /* [T][N][D] */
  const int32_t *act;     /* [T][N] */
  const float *rew;       /* [T][N] */
  const uint8_t *done;    /* [T][N] */
  const float *logp;      /* [T][N] */
  const float *val;       /* [T+1][N] */
} orc_segment;

/* ---- on-policy consumer: shuffled row order of a segment and advantage normalisation (App. C; Table 2) ---- */
int64_t orc_shuffle_index(uint64_t seed, uint64_t shuffle_id, int64_t R, int64_t i);
void    orc_normalize(const float *x, int64_t n, double eps, double *out);

/* ---- building blocks (each callable on its own so that it can be pinned) ---- */
void     orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
void     orc_stream_words(uint64_t seed, uint32_t stream, uint32_t block, uint32_t c0, uint64_t step, uint32_t out[4]);
float    orc_u01(uint32_t x);
uint32_t orc_mulhi(uint32_t x, uint32_t n);
void     orc_normal4(const uint32_t w[4], double z[4]);
uint64_t orc_explore_threshold(float epsilon);

void orc_cartpole_step(const float s[4], int a, float s_next[4], float *reward, int *terminated, double *margin);
void orc_acrobot_deriv(const double y[4], double torque, double dy[4]);
double orc_acrobot_energy(const double y[4]);
void orc_acrobot_rk4(const double y[4], double torque, double dt, double y_next[4]);
void orc_acrobot_step(const float s[4], int a, float s_next[4], float *reward, int *terminated, double *margin);
void orc_acrobot_obs(const float s[4], float obs[6]);
void orc_lingauss_step(const float *s, int a, const float *A, const float *Bm, const double *noise, int D,
                       double noise_std, double done_norm, float *s_next, float *reward, int *terminated,
                       double *margin);

/* blob = [W1 H*D, b1 H, W2 H*H, b2 H, W3 A*H, b3 A (, Wv H, bv 1)], row-major out x in */
int64_t orc_blob_floats(int D, int H, int A, int value_head);
void orc_mlp_forward_f32(const float *blob, int D, int H, int A, int value_head, const float *x, float *out,
                         float *value);
void orc_mlp_forward_f64(const float *blob, int D, int H, int A, int value_head, const float *x, double *out,
                         double *value);
float orc_bf16_round(float x);

int orc_select_eps_greedy(const float *q, int A, uint32_t x0, uint32_t x1, uint64_t threshold);
int orc_argmax_lowest(const float *q, int A);
int orc_select_categorical(const float *logits, int A, float u, double *logp, double *margin);

void orc_td_one(double q_sel, double q_next_max, double r, int done, double gamma, double kappa, double *td,
                double *huber);
/* Algorithm 1's update line as one minibatch semi-gradient step on the mean Huber loss; theta blobs in the layout above
 * (no value head); theta_out may not alias theta */
void orc_sgd_step(const float *theta, const float *theta_target, int D, int H, int A, const float *obs,
                  const int32_t *act, const float *rew, const float *next_obs, const int32_t *done, int n, double gamma,
                  double kappa, double lr, float *theta_out, double *loss_mean);
/* the same gradient through Adam (Table 2's optimiser); t >= 1 counts the steps; m, v: FP32 moment blobs */
void orc_adam_step(const float *theta, const float *theta_target, int D, int H, int A, const float *obs,
                   const int32_t *act, const float *rew, const float *next_obs, const int32_t *done, int n, double gamma,
                   double kappa, double lr, double beta1, double beta2, double eps, int64_t t, const float *m, const float *v,
                   float *theta_out, float *m_out, float *v_out, double *loss_mean);
/* PPO's clipped surrogate + value loss - entropy bonus on the shared-trunk network (blob with the value head), one Adam
 * step; stats[4] = mean policy loss, mean value loss (0.5 (V-R)^2), mean entropy, clip fraction */
void orc_ppo_step(const float *theta, int D, int H, int A, const float *obs, const int32_t *act, const float *logp_old,
                  const float *adv, const float *ret, int n, double clip_eps, double c_v, double c_e, double lr, double beta1,
                  double beta2, double eps, int64_t t, const float *m, const float *v, float *theta_out, float *m_out,
                  float *v_out, double *loss, double *stats);
void orc_gae(const float *rew, const float *val, const uint8_t *done, int T, int N, double gamma, double lambda,
             double *adv, double *ret);

/* ---- the whole path as a state machine with the library's call semantics ---- */
typedef struct orc_ctx orc_ctx;
orc_ctx *orc_create(const orc_config *cfg, int *status);
void orc_destroy(orc_ctx *);
int  orc_publish(orc_ctx *, const float *blob, int64_t n_floats);
int  orc_actor_step(orc_ctx *, int n_steps);
int  orc_sample(orc_ctx *, int staleness_bound /* -1 = config */, int32_t *idx_out, float *records_out);
int  orc_td(orc_ctx *, const float *records, int n, double *td, double *huber, double *loss_mean,
            double *q_sel, double *q_next_max);
int  orc_segment_acquire(orc_ctx *, orc_segment *out);
void orc_get_stats(const orc_ctx *, orc_stats *out);

/* state access (for stepping the oracle from a state taken elsewhere) */
int      orc_state_dim(const orc_ctx *);
int      orc_record_words(const orc_ctx *);
float   *orc_state(orc_ctx *);            /* [N][S_d] */
int32_t *orc_ep_step(orc_ctx *);          /* [N] */
void     orc_set_counters(orc_ctx *, uint64_t cursor, int64_t t, int64_t k);
uint64_t orc_cursor(const orc_ctx *);
float   *orc_ring(orc_ctx *);             /* [C][record_words] */
int32_t *orc_block_version(orc_ctx *);    /* [C / N] */
/* per-env results of the most recent actor step */
const float   *orc_last_obs(const orc_ctx *);     /* [N][D] */
const float   *orc_last_logits(const orc_ctx *);  /* [N][A] */
const int32_t *orc_last_act(const orc_ctx *);
const float   *orc_last_rew(const orc_ctx *);
const int32_t *orc_last_done(const orc_ctx *);
const float   *orc_last_next_obs(const orc_ctx *);/* [N][D] */
const double  *orc_last_done_margin(const orc_ctx *);
const double  *orc_last_act_margin(const orc_ctx *);
const float   *orc_last_logp(const orc_ctx *);
const float   *orc_last_value(const orc_ctx *);
const float   *orc_online_blob(const orc_ctx *);
const float   *orc_target_blob(const orc_ctx *);

#ifdef __cplusplus
}
#endif
#endif
