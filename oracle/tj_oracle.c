/*
 * tj_oracle.c -- plain CPU oracle (test infrastructure; see tj_oracle.h).
 *
 * Compile with -ffp-contract=off so that no multiply-add is fused unless the
 * code asks for it with fma()/fmaf().
 */
#include "tj_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define ORC_PI 3.14159265358979323846

/* ===================================================================== */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:   */
/* as easy as 1, 2, 3", SC'11).  Ten rounds; each round multiplies two of */
/* the four counter words by fixed odd constants, mixes the high halves   */
/* with the other two words and the key, and the key advances by Weyl     */
/* constants between rounds.                                              */
/* ===================================================================== */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)M0 * c0;
    uint64_t p1 = (uint64_t)M1 * c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Keying used by the whole path: key = the 64-bit seed; counter =
 * (c0 = env index or minibatch slot, c1 = low half of the step index,
 *  c2 = stream id | block << 8, c3 = high half of the step index). */
void orc_stream_words(uint64_t seed, uint32_t stream, uint32_t block, uint32_t c0, uint64_t step,
                      uint32_t out[4]) {
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t ctr[4] = {c0, (uint32_t)step, stream | (block << 8), (uint32_t)(step >> 32)};
  orc_philox4x32_10(ctr, key, out);
}

/* uint32 -> uniform in (0,1): the top 23 bits plus one half, scaled by 2^-23.
 * 2n+1 < 2^24, so the value is exactly representable in FP32. */
float orc_u01(uint32_t x) { return (float)(((double)(x >> 9) + 0.5) * (1.0 / 8388608.0)); }

/* integer in [0,n): high word of the 64-bit product */
uint32_t orc_mulhi(uint32_t x, uint32_t n) { return (uint32_t)(((uint64_t)x * (uint64_t)n) >> 32); }

/* four standard normals from four words: two Box-Muller pairs */
void orc_normal4(const uint32_t w[4], double z[4]) {
  for (int p = 0; p < 2; ++p) {
    double u1 = (double)orc_u01(w[2 * p]);
    double u2 = (double)orc_u01(w[2 * p + 1]);
    double r = sqrt(-2.0 * log(u1));
    z[2 * p] = r * cos(2.0 * ORC_PI * u2);
    z[2 * p + 1] = r * sin(2.0 * ORC_PI * u2);
  }
}

/* explore iff x0 < floor(epsilon * 2^32) */
uint64_t orc_explore_threshold(float epsilon) {
  double e = (double)epsilon;
  if (!(e > 0.0)) return 0;
  if (e >= 1.0) return 4294967296ull;
  return (uint64_t)floor(e * 4294967296.0);
}

/* U(lo, lo+width) from one word, as one FP32 fused multiply-add */
static float uniform_range(uint32_t x, float lo, float width) { return fmaf(orc_u01(x), width, lo); }

/* ===================================================================== */
/* CartPole: frictionless cart-pole of Barto, Sutton & Anderson (1983),   */
/* explicit Euler, positions advanced with the old velocities.            */
/* ===================================================================== */
void orc_cartpole_step(const float s[4], int a, float s_next[4], float *reward, int *terminated, double *margin) {
  const double g = 9.8, masscart = 1.0, masspole = 0.1, length = 0.5, force_mag = 10.0, tau = 0.02;
  const double total_mass = masscart + masspole, polemass_length = masspole * length;
  double x = s[0], x_dot = s[1], theta = s[2], theta_dot = s[3];
  double force = (a == 1) ? force_mag : -force_mag;
  double costheta = cos(theta), sintheta = sin(theta);
  double temp = (force + polemass_length * theta_dot * theta_dot * sintheta) / total_mass;
  double thetaacc =
      (g * sintheta - costheta * temp) / (length * (4.0 / 3.0 - masspole * costheta * costheta / total_mass));
  double xacc = temp - polemass_length * thetaacc * costheta / total_mass;
  s_next[0] = (float)(x + tau * x_dot);
  s_next[1] = (float)(x_dot + tau * xacc);
  s_next[2] = (float)(theta + tau * theta_dot);
  s_next[3] = (float)(theta_dot + tau * thetaacc);
  /* termination is decided on the stored (FP32) state against FP32 thresholds */
  const float x_thr = 2.4f, th_thr = (float)(12.0 * 2.0 * ORC_PI / 360.0);
  *terminated = (fabsf(s_next[0]) > x_thr) || (fabsf(s_next[2]) > th_thr);
  *reward = 1.0f;
  if (margin) {
    double mx = fabs(fabs((double)s_next[0]) - (double)x_thr) / (double)x_thr;
    double mt = fabs(fabs((double)s_next[2]) - (double)th_thr) / (double)th_thr;
    *margin = mx < mt ? mx : mt;
  }
}

/* ===================================================================== */
/* Acrobot (Sutton & Barto's two-link pendulum, torque on the second      */
/* joint), general-constant form; angles are measured from the downward   */
/* vertical, so the gravity terms are g sin(theta).                       */
/* ===================================================================== */
static const double ACR_M1 = 1.0, ACR_M2 = 1.0, ACR_L1 = 1.0, ACR_LC1 = 0.5, ACR_LC2 = 0.5, ACR_I1 = 1.0,
                    ACR_I2 = 1.0, ACR_G = 9.8;

void orc_acrobot_deriv(const double y[4], double torque, double dy[4]) {
  double th1 = y[0], th2 = y[1], w1 = y[2], w2 = y[3];
  double d1 = ACR_M1 * ACR_LC1 * ACR_LC1 +
              ACR_M2 * (ACR_L1 * ACR_L1 + ACR_LC2 * ACR_LC2 + 2.0 * ACR_L1 * ACR_LC2 * cos(th2)) + ACR_I1 + ACR_I2;
  double d2 = ACR_M2 * (ACR_LC2 * ACR_LC2 + ACR_L1 * ACR_LC2 * cos(th2)) + ACR_I2;
  double phi2 = ACR_M2 * ACR_LC2 * ACR_G * sin(th1 + th2);
  double phi1 = -ACR_M2 * ACR_L1 * ACR_LC2 * w2 * w2 * sin(th2) -
                2.0 * ACR_M2 * ACR_L1 * ACR_LC2 * w2 * w1 * sin(th2) +
                (ACR_M1 * ACR_LC1 + ACR_M2 * ACR_L1) * ACR_G * sin(th1) + phi2;
  double ddth2 = (torque + d2 / d1 * phi1 - ACR_M2 * ACR_L1 * ACR_LC2 * w1 * w1 * sin(th2) - phi2) /
                 (ACR_M2 * ACR_LC2 * ACR_LC2 + ACR_I2 - d2 * d2 / d1);
  double ddth1 = -(d2 * ddth2 + phi1) / d1;
  dy[0] = w1; dy[1] = w2; dy[2] = ddth1; dy[3] = ddth2;
}

/* total mechanical energy of the same system (used only to pin the equations) */
double orc_acrobot_energy(const double y[4]) {
  double th1 = y[0], th2 = y[1], w1 = y[2], w2 = y[3];
  double d1 = ACR_M1 * ACR_LC1 * ACR_LC1 +
              ACR_M2 * (ACR_L1 * ACR_L1 + ACR_LC2 * ACR_LC2 + 2.0 * ACR_L1 * ACR_LC2 * cos(th2)) + ACR_I1 + ACR_I2;
  double d2 = ACR_M2 * (ACR_LC2 * ACR_LC2 + ACR_L1 * ACR_LC2 * cos(th2)) + ACR_I2;
  double m22 = ACR_M2 * ACR_LC2 * ACR_LC2 + ACR_I2;
  double kinetic = 0.5 * d1 * w1 * w1 + d2 * w1 * w2 + 0.5 * m22 * w2 * w2;
  double potential = -(ACR_M1 * ACR_LC1 + ACR_M2 * ACR_L1) * ACR_G * cos(th1) - ACR_M2 * ACR_LC2 * ACR_G * cos(th1 + th2);
  return kinetic + potential;
}

/* one classical fourth-order Runge-Kutta step with the torque held */
void orc_acrobot_rk4(const double y[4], double torque, double dt, double y_next[4]) {
  double k1[4], k2[4], k3[4], k4[4], tmp[4];
  orc_acrobot_deriv(y, torque, k1);
  for (int i = 0; i < 4; ++i) tmp[i] = y[i] + 0.5 * dt * k1[i];
  orc_acrobot_deriv(tmp, torque, k2);
  for (int i = 0; i < 4; ++i) tmp[i] = y[i] + 0.5 * dt * k2[i];
  orc_acrobot_deriv(tmp, torque, k3);
  for (int i = 0; i < 4; ++i) tmp[i] = y[i] + dt * k3[i];
  orc_acrobot_deriv(tmp, torque, k4);
  for (int i = 0; i < 4; ++i) y_next[i] = y[i] + dt / 6.0 * (k1[i] + 2.0 * k2[i] + 2.0 * k3[i] + k4[i]);
}

static double wrap_pi(double x) { return x - 2.0 * ORC_PI * floor((x + ORC_PI) / (2.0 * ORC_PI)); }
static double clampd(double x, double lo, double hi) { return x < lo ? lo : (x > hi ? hi : x); }

void orc_acrobot_step(const float s[4], int a, float s_next[4], float *reward, int *terminated, double *margin) {
  double y[4] = {s[0], s[1], s[2], s[3]}, yn[4];
  double torque = (double)(a - 1);
  orc_acrobot_rk4(y, torque, 0.2, yn);
  yn[0] = wrap_pi(yn[0]);
  yn[1] = wrap_pi(yn[1]);
  yn[2] = clampd(yn[2], -4.0 * ORC_PI, 4.0 * ORC_PI);
  yn[3] = clampd(yn[3], -9.0 * ORC_PI, 9.0 * ORC_PI);
  for (int i = 0; i < 4; ++i) s_next[i] = (float)yn[i];
  double tip = -cos((double)s_next[0]) - cos((double)s_next[0] + (double)s_next[1]);
  *terminated = tip > 1.0;
  *reward = *terminated ? 0.0f : -1.0f;
  if (margin) *margin = fabs(tip - 1.0);
}

void orc_acrobot_obs(const float s[4], float obs[6]) {
  obs[0] = (float)cos((double)s[0]);
  obs[1] = (float)sin((double)s[0]);
  obs[2] = (float)cos((double)s[1]);
  obs[3] = (float)sin((double)s[1]);
  obs[4] = s[2];
  obs[5] = s[3];
}

/* ===================================================================== */
/* Linear-Gaussian env: s' = tanh(A s + B[a]) + noise_std * n;            */
/* reward = -||s'||^2 / D; terminated when ||s'|| > done_norm.            */
/* ===================================================================== */
void orc_lingauss_step(const float *s, int a, const float *A, const float *Bm, const double *noise, int D,
                       double noise_std, double done_norm, float *s_next, float *reward, int *terminated,
                       double *margin) {
  double sq = 0.0;
  for (int i = 0; i < D; ++i) {
    double z = (double)Bm[(size_t)a * D + i];
    for (int k = 0; k < D; ++k) z += (double)A[(size_t)i * D + k] * (double)s[k];
    s_next[i] = (float)(tanh(z) + noise_std * noise[i]);
    sq += (double)s_next[i] * (double)s_next[i];
  }
  double norm = sqrt(sq);
  *reward = (float)(-sq / (double)D);
  *terminated = norm > done_norm;
  if (margin) *margin = fabs(norm - done_norm) / done_norm;
}

/* ===================================================================== */
/* Policy MLP: two hidden ReLU layers and a linear head (plus a value     */
/* head that shares the trunk).                                           */
/* ===================================================================== */
int64_t orc_blob_floats(int D, int H, int A, int value_head) {
  return (int64_t)H * D + H + (int64_t)H * H + H + (int64_t)A * H + A + (value_head ? (H + 1) : 0);
}

/* FP32 with a stated rounding order: acc = bias; acc = fmaf(w[k], x[k], acc) for k = 0, 1, ... */
static void dense_f32(const float *W, const float *b, int n_out, int n_in, const float *x, float *y, int relu) {
  for (int i = 0; i < n_out; ++i) {
    float acc = b[i];
    for (int k = 0; k < n_in; ++k) acc = fmaf(W[(size_t)i * n_in + k], x[k], acc);
    y[i] = (relu && !(acc > 0.0f)) ? 0.0f : acc;
  }
}
static void dense_f64(const float *W, const float *b, int n_out, int n_in, const double *x, double *y, int relu) {
  for (int i = 0; i < n_out; ++i) {
    double acc = (double)b[i];
    for (int k = 0; k < n_in; ++k) acc += (double)W[(size_t)i * n_in + k] * x[k];
    y[i] = (relu && !(acc > 0.0)) ? 0.0 : acc;
  }
}

void orc_mlp_forward_f32(const float *blob, int D, int H, int A, int value_head, const float *x, float *out,
                         float *value) {
  const float *W1 = blob, *b1 = W1 + (size_t)H * D, *W2 = b1 + H, *b2 = W2 + (size_t)H * H, *W3 = b2 + H,
              *b3 = W3 + (size_t)A * H, *Wv = b3 + A, *bv = Wv + H;
  float *h1 = (float *)malloc(sizeof(float) * H), *h2 = (float *)malloc(sizeof(float) * H);
  dense_f32(W1, b1, H, D, x, h1, 1);
  dense_f32(W2, b2, H, H, h1, h2, 1);
  dense_f32(W3, b3, A, H, h2, out, 0);
  if (value_head && value) dense_f32(Wv, bv, 1, H, h2, value, 0);
  free(h1); free(h2);
}

void orc_mlp_forward_f64(const float *blob, int D, int H, int A, int value_head, const float *x, double *out,
                         double *value) {
  const float *W1 = blob, *b1 = W1 + (size_t)H * D, *W2 = b1 + H, *b2 = W2 + (size_t)H * H, *W3 = b2 + H,
              *b3 = W3 + (size_t)A * H, *Wv = b3 + A, *bv = Wv + H;
  double *xd = (double *)malloc(sizeof(double) * D), *h1 = (double *)malloc(sizeof(double) * H),
         *h2 = (double *)malloc(sizeof(double) * H);
  for (int k = 0; k < D; ++k) xd[k] = (double)x[k];
  dense_f64(W1, b1, H, D, xd, h1, 1);
  dense_f64(W2, b2, H, H, h1, h2, 1);
  dense_f64(W3, b3, A, H, h2, out, 0);
  if (value_head && value) dense_f64(Wv, bv, 1, H, h2, value, 0);
  free(xd); free(h1); free(h2);
}

/* bfloat16 = the top 16 bits of an FP32 value; round to nearest, ties to even */
float orc_bf16_round(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return x; /* inf / nan unchanged */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  float y;
  memcpy(&y, &u, 4);
  return y;
}

/* ===================================================================== */
/* Action selection                                                       */
/* ===================================================================== */
int orc_argmax_lowest(const float *q, int A) {
  int best = 0;
  for (int i = 1; i < A; ++i)
    if (q[i] > q[best]) best = i; /* strict: the lowest index wins ties, NaN never wins */
  return best;
}

int orc_select_eps_greedy(const float *q, int A, uint32_t x0, uint32_t x1, uint64_t threshold) {
  if ((uint64_t)x0 < threshold) return (int)orc_mulhi(x1, (uint32_t)A);
  return orc_argmax_lowest(q, A);
}

/* inverse-CDF draw over softmax(logits): the smallest i whose cumulative mass exceeds u * Z */
int orc_select_categorical(const float *logits, int A, float u, double *logp, double *margin) {
  double m = (double)logits[0];
  for (int i = 1; i < A; ++i)
    if ((double)logits[i] > m) m = (double)logits[i];
  double Z = 0.0;
  for (int i = 0; i < A; ++i) Z += exp((double)logits[i] - m);
  double target = (double)u * Z, cum = 0.0, mg = 1e300;
  int a = A - 1, found = 0;
  for (int i = 0; i < A; ++i) {
    cum += exp((double)logits[i] - m);
    if (i < A - 1) {
      double d = fabs(cum - target) / Z;
      if (d < mg) mg = d;
    }
    if (!found && cum > target) { a = i; found = 1; }
  }
  if (logp) *logp = (double)logits[a] - m - log(Z);
  if (margin) *margin = mg;
  return a;
}

/* ===================================================================== */
/* TD target, TD error, Huber loss (one sample)                           */
/* ===================================================================== */
void orc_td_one(double q_sel, double q_next_max, double r, int done, double gamma, double kappa, double *td,
                double *huber) {
  double y = r + gamma * (done ? 0.0 : 1.0) * q_next_max;
  double delta = y - q_sel;
  double ad = fabs(delta);
  *td = delta;
  *huber = (ad <= kappa) ? 0.5 * delta * delta : kappa * (ad - 0.5 * kappa);
}

/* ===================================================================== */
/* Learner update (Algorithm 1: theta <- theta + alpha * delta * grad V(s; theta)), as one minibatch step:   */
/*   L(theta) = mean_j Huber(delta_j),  delta_j = r_j + gamma (1 - done_j) max_a Q(s'_j, a; theta_target)     */
/*                                               - Q(s_j, a_j; theta)                                         */
/*   theta <- theta - lr * dL/dtheta, the target term held constant (semi-gradient).                          */
/* dHuber/ddelta = clip(delta, -kappa, kappa), so dL/dQ(s_j, a_j) = -clip(delta_j) / n: with kappa = inf,     */
/* n = 1 and theta_target = theta this is Algorithm 1's update line.  Everything in double from the FP32      */
/* inputs; the new parameters are rounded to FP32 once, at the end.                                           */
/* ===================================================================== */
/* grad[i] = dL/dtheta_i (double, caller-allocated, orc_blob_floats entries); returns the mean Huber loss */
static double td_loss_gradient(const float *theta, const float *theta_target, int D, int H, int A, const float *obs,
                               const int32_t *act, const float *rew, const float *next_obs, const int32_t *done, int n,
                               double gamma, double kappa, double *grad) {
  const size_t nW1 = (size_t)H * D, nW2 = (size_t)H * H, nW3 = (size_t)A * H;
  const size_t o_b1 = nW1, o_W2 = o_b1 + H, o_b2 = o_W2 + nW2, o_W3 = o_b2 + H, o_b3 = o_W3 + nW3, total = o_b3 + A;
  for (size_t i = 0; i < total; ++i) grad[i] = 0.0;
  double *h1 = (double *)malloc(sizeof(double) * H), *h2 = (double *)malloc(sizeof(double) * H);
  double *dh1 = (double *)malloc(sizeof(double) * H), *dh2 = (double *)malloc(sizeof(double) * H);
  double *qn = (double *)malloc(sizeof(double) * A);
  const float *W1 = theta, *b1 = theta + o_b1, *W2 = theta + o_W2, *b2 = theta + o_b2, *W3 = theta + o_W3, *b3 = theta + o_b3;
  double loss = 0.0;
  for (int j = 0; j < n; ++j) {
    const float *x = obs + (size_t)j * D;
    int a = act[j];
    if (a < 0) a = 0;
    if (a >= A) a = A - 1;
    /* online forward, activations kept */
    for (int i = 0; i < H; ++i) {
      double s = (double)b1[i];
      for (int k = 0; k < D; ++k) s += (double)W1[(size_t)i * D + k] * (double)x[k];
      h1[i] = s > 0.0 ? s : 0.0;
    }
    for (int i = 0; i < H; ++i) {
      double s = (double)b2[i];
      for (int k = 0; k < H; ++k) s += (double)W2[(size_t)i * H + k] * h1[k];
      h2[i] = s > 0.0 ? s : 0.0;
    }
    double q = (double)b3[a];
    for (int k = 0; k < H; ++k) q += (double)W3[(size_t)a * H + k] * h2[k];
    /* target: max over the target network's outputs at the next observation */
    orc_mlp_forward_f64(theta_target, D, H, A, 0, next_obs + (size_t)j * D, qn, NULL);
    double qmax = qn[0];
    for (int i = 1; i < A; ++i)
      if (qn[i] > qmax) qmax = qn[i];
    double delta, hub;
    orc_td_one(q, qmax, (double)rew[j], done[j], gamma, kappa, &delta, &hub);
    loss += hub;
    /* dL/dq = -clip(delta, -kappa, kappa) / n */
    double c = delta > kappa ? kappa : (delta < -kappa ? -kappa : delta);
    const double g = -c / (double)n;
    /* head row a */
    grad[o_b3 + a] += g;
    for (int k = 0; k < H; ++k) {
      grad[o_W3 + (size_t)a * H + k] += g * h2[k];
      dh2[k] = h2[k] > 0.0 ? g * (double)W3[(size_t)a * H + k] : 0.0;
    }
    /* layer 2 */
    for (int k = 0; k < H; ++k) dh1[k] = 0.0;
    for (int i = 0; i < H; ++i) {
      if (dh2[i] == 0.0) continue;
      grad[o_b2 + i] += dh2[i];
      for (int k = 0; k < H; ++k) {
        grad[o_W2 + (size_t)i * H + k] += dh2[i] * h1[k];
        dh1[k] += dh2[i] * (double)W2[(size_t)i * H + k];
      }
    }
    /* layer 1 */
    for (int i = 0; i < H; ++i) {
      const double d = h1[i] > 0.0 ? dh1[i] : 0.0;
      if (d == 0.0) continue;
      grad[o_b1 + i] += d;
      for (int k = 0; k < D; ++k) grad[(size_t)i * D + k] += d * (double)x[k];
    }
  }
  free(h1); free(h2); free(dh1); free(dh2); free(qn);
  return loss / (double)n;
}


void orc_sgd_step(const float *theta, const float *theta_target, int D, int H, int A, const float *obs,
                  const int32_t *act, const float *rew, const float *next_obs, const int32_t *done, int n, double gamma,
                  double kappa, double lr, float *theta_out, double *loss_mean) {
  const size_t total = (size_t)orc_blob_floats(D, H, A, 0);
  double *grad = (double *)malloc(total * sizeof(double));
  const double loss = td_loss_gradient(theta, theta_target, D, H, A, obs, act, rew, next_obs, done, n, gamma, kappa, grad);
  for (size_t i = 0; i < total; ++i) theta_out[i] = (float)((double)theta[i] - lr * grad[i]);
  if (loss_mean) *loss_mean = loss;
  free(grad);
}

/* The same gradient fed to Adam (Kingma & Ba 2015; the optimiser of Table 2), step counter t >= 1:                   */
/*   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;  theta <- theta - lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps) */
/* m and v are FP32 state blobs like theta (read from m, v; written to m_out, v_out), arithmetic in double.            */
void orc_adam_step(const float *theta, const float *theta_target, int D, int H, int A, const float *obs,
                   const int32_t *act, const float *rew, const float *next_obs, const int32_t *done, int n, double gamma,
                   double kappa, double lr, double beta1, double beta2, double eps, int64_t t, const float *m, const float *v,
                   float *theta_out, float *m_out, float *v_out, double *loss_mean) {
  const size_t total = (size_t)orc_blob_floats(D, H, A, 0);
  double *grad = (double *)malloc(total * sizeof(double));
  const double loss = td_loss_gradient(theta, theta_target, D, H, A, obs, act, rew, next_obs, done, n, gamma, kappa, grad);
  const double c1 = 1.0 - pow(beta1, (double)t), c2 = 1.0 - pow(beta2, (double)t);
  for (size_t i = 0; i < total; ++i) {
    /* the moments are stored in FP32: the update uses the values as stored */
    const float mf = (float)(beta1 * (double)m[i] + (1.0 - beta1) * grad[i]);
    const float vf = (float)(beta2 * (double)v[i] + (1.0 - beta2) * grad[i] * grad[i]);
    m_out[i] = mf;
    v_out[i] = vf;
    theta_out[i] = (float)((double)theta[i] - lr * ((double)mf / c1) / (sqrt((double)vf / c2) + eps));
  }
  if (loss_mean) *loss_mean = loss;
  free(grad);
}

/* ===================================================================== */
/* On-policy learner update: PPO's clipped surrogate (Schulman et al. 2017; the paper's on-policy algorithm,       */
/* Sec. 4.1) on the shared-trunk network with a categorical policy head and a value head:                          */
/*   p = softmax(logits), ratio = exp(log p[a] - logp_old),                                                         */
/*   L = mean_j [ -min(ratio A, clip(ratio, 1-eps, 1+eps) A) + c_v/2 (V - R)^2 - c_e H(p) ]                          */
/* then one Adam step on L.  Blob layout with the value head: [W1, b1, W2, b2, W3, b3, Wv, bv].                      */
/* stats[0..3] = mean policy loss, mean value loss (without c_v), mean entropy, fraction of rows with the clip active */
/* ===================================================================== */
static double ppo_loss_gradient(const float *theta, int D, int H, int A, const float *obs, const int32_t *act,
                                const float *logp_old, const float *adv, const float *ret, int n, double clip_eps, double c_v,
                                double c_e, double *grad, double *stats) {
  const size_t nW1 = (size_t)H * D, nW2 = (size_t)H * H, nW3 = (size_t)A * H;
  const size_t o_b1 = nW1, o_W2 = o_b1 + H, o_b2 = o_W2 + nW2, o_W3 = o_b2 + H, o_b3 = o_W3 + nW3, o_Wv = o_b3 + A,
               o_bv = o_Wv + H, total = o_bv + 1;
  for (size_t i = 0; i < total; ++i) grad[i] = 0.0;
  double *h1 = (double *)malloc(sizeof(double) * H), *h2 = (double *)malloc(sizeof(double) * H);
  double *dh1 = (double *)malloc(sizeof(double) * H), *dh2 = (double *)malloc(sizeof(double) * H);
  double *l = (double *)malloc(sizeof(double) * A), *pr = (double *)malloc(sizeof(double) * A),
         *gl = (double *)malloc(sizeof(double) * A);
  const float *W1 = theta, *b1 = theta + o_b1, *W2 = theta + o_W2, *b2 = theta + o_b2, *W3 = theta + o_W3, *b3 = theta + o_b3,
              *Wv = theta + o_Wv, *bv = theta + o_bv;
  double s_pi = 0.0, s_v = 0.0, s_h = 0.0, s_clip = 0.0;
  for (int j = 0; j < n; ++j) {
    const float *x = obs + (size_t)j * D;
    int a = act[j];
    if (a < 0) a = 0;
    if (a >= A) a = A - 1;
    for (int i = 0; i < H; ++i) {
      double s = (double)b1[i];
      for (int k = 0; k < D; ++k) s += (double)W1[(size_t)i * D + k] * (double)x[k];
      h1[i] = s > 0.0 ? s : 0.0;
    }
    for (int i = 0; i < H; ++i) {
      double s = (double)b2[i];
      for (int k = 0; k < H; ++k) s += (double)W2[(size_t)i * H + k] * h1[k];
      h2[i] = s > 0.0 ? s : 0.0;
    }
    double lmax = -1e300;
    for (int i = 0; i < A; ++i) {
      double s = (double)b3[i];
      for (int k = 0; k < H; ++k) s += (double)W3[(size_t)i * H + k] * h2[k];
      l[i] = s;
      if (s > lmax) lmax = s;
    }
    double val = (double)bv[0];
    for (int k = 0; k < H; ++k) val += (double)Wv[k] * h2[k];
    double Z = 0.0;
    for (int i = 0; i < A; ++i) Z += exp(l[i] - lmax);
    const double logZ = lmax + log(Z);
    double ent = 0.0;
    for (int i = 0; i < A; ++i) {
      pr[i] = exp(l[i] - logZ);
      ent -= pr[i] * (l[i] - logZ);
    }
    const double logp = l[a] - logZ, ratio = exp(logp - (double)logp_old[j]), Aj = (double)adv[j];
    const double rc = ratio < 1.0 - clip_eps ? 1.0 - clip_eps : (ratio > 1.0 + clip_eps ? 1.0 + clip_eps : ratio);
    const double t1 = ratio * Aj, t2 = rc * Aj;
    const int unclipped = t1 <= t2; /* the minimum is the unclipped term (also when both are equal) */
    s_pi += -(unclipped ? t1 : t2);
    s_clip += unclipped ? 0.0 : 1.0;
    const double dv = val - (double)ret[j];
    s_v += 0.5 * dv * dv;
    s_h += ent;
    /* gradients at the outputs, already divided by n */
    const double g_logp = unclipped ? -Aj * ratio : 0.0;
    for (int i = 0; i < A; ++i) {
      const double dlogp = (i == a ? 1.0 : 0.0) - pr[i];
      const double dent = -pr[i] * ((l[i] - logZ) + ent); /* dH/dl_i */
      gl[i] = (g_logp * dlogp - c_e * dent) / (double)n;
    }
    const double gv = c_v * dv / (double)n;
    /* heads */
    for (int k = 0; k < H; ++k) dh2[k] = 0.0;
    for (int i = 0; i < A; ++i) {
      grad[o_b3 + i] += gl[i];
      for (int k = 0; k < H; ++k) {
        grad[o_W3 + (size_t)i * H + k] += gl[i] * h2[k];
        dh2[k] += gl[i] * (double)W3[(size_t)i * H + k];
      }
    }
    grad[o_bv] += gv;
    for (int k = 0; k < H; ++k) {
      grad[o_Wv + k] += gv * h2[k];
      dh2[k] += gv * (double)Wv[k];
      if (!(h2[k] > 0.0)) dh2[k] = 0.0;
    }
    /* layer 2 */
    for (int k = 0; k < H; ++k) dh1[k] = 0.0;
    for (int i = 0; i < H; ++i) {
      if (dh2[i] == 0.0) continue;
      grad[o_b2 + i] += dh2[i];
      for (int k = 0; k < H; ++k) {
        grad[o_W2 + (size_t)i * H + k] += dh2[i] * h1[k];
        dh1[k] += dh2[i] * (double)W2[(size_t)i * H + k];
      }
    }
    /* layer 1 */
    for (int i = 0; i < H; ++i) {
      const double d = h1[i] > 0.0 ? dh1[i] : 0.0;
      if (d == 0.0) continue;
      grad[o_b1 + i] += d;
      for (int k = 0; k < D; ++k) grad[(size_t)i * D + k] += d * (double)x[k];
    }
  }
  free(h1); free(h2); free(dh1); free(dh2); free(l); free(pr); free(gl);
  if (stats) {
    stats[0] = s_pi / n; stats[1] = s_v / n; stats[2] = s_h / n; stats[3] = s_clip / n;
  }
  return (s_pi + c_v * s_v - c_e * s_h) / (double)n;
}

void orc_ppo_step(const float *theta, int D, int H, int A, const float *obs, const int32_t *act, const float *logp_old,
                  const float *adv, const float *ret, int n, double clip_eps, double c_v, double c_e, double lr, double beta1,
                  double beta2, double eps, int64_t t, const float *m, const float *v, float *theta_out, float *m_out,
                  float *v_out, double *loss, double *stats) {
  const size_t total = (size_t)orc_blob_floats(D, H, A, 1);
  double *grad = (double *)malloc(total * sizeof(double));
  const double L = ppo_loss_gradient(theta, D, H, A, obs, act, logp_old, adv, ret, n, clip_eps, c_v, c_e, grad, stats);
  const double c1 = 1.0 - pow(beta1, (double)t), c2 = 1.0 - pow(beta2, (double)t);
  for (size_t i = 0; i < total; ++i) {
    const float mf = (float)(beta1 * (double)m[i] + (1.0 - beta1) * grad[i]);
    const float vf = (float)(beta2 * (double)v[i] + (1.0 - beta2) * grad[i] * grad[i]);
    m_out[i] = mf;
    v_out[i] = vf;
    theta_out[i] = (float)((double)theta[i] - lr * ((double)mf / c1) / (sqrt((double)vf / c2) + eps));
  }
  if (loss) *loss = L;
  free(grad);
}

/* ===================================================================== */
/* GAE: delta_t = r_t + gamma (1-d_t) V_{t+1} - V_t;                      */
/*      A_t = delta_t + gamma lambda (1-d_t) A_{t+1}, A_T = 0; R_t = A_t + V_t */
/* arrays are time-major: rew[T][N], val[T+1][N], done[T][N]              */
/* ===================================================================== */
void orc_gae(const float *rew, const float *val, const uint8_t *done, int T, int N, double gamma, double lambda,
             double *adv, double *ret) {
  for (int e = 0; e < N; ++e) {
    double next_adv = 0.0;
    for (int t = T - 1; t >= 0; --t) {
      size_t i = (size_t)t * N + e;
      double nd = done[i] ? 0.0 : 1.0;
      double delta = (double)rew[i] + gamma * nd * (double)val[(size_t)(t + 1) * N + e] - (double)val[i];
      double a = delta + gamma * lambda * nd * next_adv;
      adv[i] = a;
      ret[i] = a + (double)val[i];
      next_adv = a;
    }
  }
}

/* ===================================================================== */
/* On-policy consumer (App. C synchronous mode; Table 2's PPO batch settings): per-segment advantage            */
/* normalisation and shuffled minibatches.                                                                      */
/*                                                                                                              */
/* The row order of a shuffle is a keyed bijection of [0, R): a four-round balanced Feistel network on          */
/* 2*hb bits (hb = half the bits of R - 1, rounded up, at least 1) whose round function is the first            */
/* Philox word of the SHUFFLE stream at (index = right half, step = shuffle id, block = round), followed        */
/* by cycle walking (apply again until the value falls below R).  A Feistel network is a bijection of its       */
/* power-of-two domain and cycle walking restricts it to [0, R) (Black & Rogaway, "Ciphers with arbitrary       */
/* finite domains", 2002).                                                                                      */
/* ===================================================================== */
static int shuffle_half_bits(uint64_t R) {
  int bits = 0;
  while (bits < 62 && ((uint64_t)1 << bits) < R) ++bits; /* 2^bits >= R */
  int hb = (bits + 1) / 2;
  return hb < 1 ? 1 : hb;
}

static uint64_t shuffle_feistel(uint64_t seed, uint64_t shuffle_id, int hb, uint64_t x) {
  const uint64_t mask = ((uint64_t)1 << hb) - 1;
  uint64_t left = x >> hb, right = x & mask;
  for (uint32_t round = 0; round < 4; ++round) {
    uint32_t w[4];
    orc_stream_words(seed, ORC_STREAM_SHUFFLE, round, (uint32_t)right, shuffle_id, w);
    uint64_t f = (uint64_t)w[0] & mask;
    uint64_t new_right = left ^ f;
    left = right;
    right = new_right;
  }
  return (left << hb) | right;
}

/* row that position i of the shuffled order takes, out of R rows */
int64_t orc_shuffle_index(uint64_t seed, uint64_t shuffle_id, int64_t R, int64_t i) {
  if (R <= 0 || i < 0 || i >= R) return -1;
  const int hb = shuffle_half_bits((uint64_t)R);
  uint64_t y = shuffle_feistel(seed, shuffle_id, hb, (uint64_t)i);
  while (y >= (uint64_t)R) y = shuffle_feistel(seed, shuffle_id, hb, y);
  return (int64_t)y;
}

/* out_i = (x_i - mean) / (sqrt(var) + eps): mean and population variance over all n entries, in double */
void orc_normalize(const float *x, int64_t n, double eps, double *out) {
  if (n <= 0) return;
  double sum = 0.0;
  for (int64_t i = 0; i < n; ++i) sum += (double)x[i];
  const double mean = sum / (double)n;
  double sq = 0.0;
  for (int64_t i = 0; i < n; ++i) sq += ((double)x[i] - mean) * ((double)x[i] - mean);
  const double sd = sqrt(sq / (double)n);
  for (int64_t i = 0; i < n; ++i) out[i] = ((double)x[i] - mean) / (sd + eps);
}

/* ===================================================================== */
/* The whole path as a state machine                                      */
/* ===================================================================== */
struct orc_ctx {
  orc_config cfg;
  int S_d, D, A, H, N, value_head, rec_words, max_ep;
  int64_t n_blob;
  float *lgA, *lgB;
  float *state;      /* [N][S_d] */
  int32_t *ep_step;  /* [N] */
  double *ep_return; /* [N] */
  /* weights: online = newest published (actor and learner read it), target = snapshot */
  float *online, *target;
  int64_t version;          /* number of publishes so far */
  int64_t k_last_sync;
  int has_target;
  /* replay ring */
  int64_t C;
  uint64_t cursor;
  float *ring;              /* [C][rec_words] */
  int32_t *block_ver;       /* [C/N] */
  int64_t t, k;
  /* segments */
  int T, n_seg;
  float *seg_obs, *seg_rew, *seg_logp, *seg_val;
  int32_t *seg_act;
  uint8_t *seg_done;
  int64_t *seg_version;
  int64_t *seg_index;       /* which segment number sits in the slot (-1 = none) */
  int *seg_state;           /* 0 empty, 1 filling, 2 complete, 3 consumed */
  int64_t next_consume;     /* segment number the consumer looks at next */
  /* last-step outputs */
  float *l_obs, *l_logits, *l_rew, *l_next_obs, *l_logp, *l_value;
  int32_t *l_act, *l_done;
  double *l_done_margin, *l_act_margin;
  orc_stats st;
};

static int env_state_dim(int kind, int D) { return kind == ORC_ENV_LINGAUSS ? D : 4; }

static void observe(const orc_ctx *c, const float *s, float *obs) {
  if (c->cfg.env_kind == ORC_ENV_ACROBOT) orc_acrobot_obs(s, obs);
  else memcpy(obs, s, sizeof(float) * c->D);
}

static void reset_env(const orc_ctx *c, int e, uint64_t step, float *s) {
  float lo, width;
  if (c->cfg.env_kind == ORC_ENV_CARTPOLE) { lo = -0.05f; width = 0.1f; }
  else { lo = -0.1f; width = 0.2f; }
  for (int b = 0; b < c->S_d / 4; ++b) {
    uint32_t w[4];
    orc_stream_words(c->cfg.seed, ORC_STREAM_RESET, (uint32_t)b, (uint32_t)e, step, w);
    for (int j = 0; j < 4; ++j) s[4 * b + j] = uniform_range(w[j], lo, width);
  }
}

/* weights as the MLP uses them: FP32 as given, or every weight matrix rounded to bfloat16 (biases stay FP32) */
static void store_weights(const orc_ctx *c, const float *blob, float *dst) {
  memcpy(dst, blob, sizeof(float) * c->n_blob);
  if (c->cfg.weight_dtype == ORC_W_BF16) {
    int D = c->D, H = c->H, A = c->A;
    float *W1 = dst, *W2 = W1 + (size_t)H * D + H, *W3 = W2 + (size_t)H * H + H, *Wv = W3 + (size_t)A * H + A;
    for (size_t i = 0; i < (size_t)H * D; ++i) W1[i] = orc_bf16_round(W1[i]);
    for (size_t i = 0; i < (size_t)H * H; ++i) W2[i] = orc_bf16_round(W2[i]);
    for (size_t i = 0; i < (size_t)A * H; ++i) W3[i] = orc_bf16_round(W3[i]);
    if (c->value_head)
      for (int i = 0; i < H; ++i) Wv[i] = orc_bf16_round(Wv[i]);
  }
}

/* forward pass in the arithmetic the configuration names */
static void policy_forward(const orc_ctx *c, const float *blob, const float *x, float *out, float *value) {
  if (c->cfg.weight_dtype == ORC_W_FP32) {
    orc_mlp_forward_f32(blob, c->D, c->H, c->A, c->value_head, x, out, value);
  } else {
    double o[64], v = 0.0;
    orc_mlp_forward_f64(blob, c->D, c->H, c->A, c->value_head, x, o, &v);
    for (int i = 0; i < c->A; ++i) out[i] = (float)o[i];
    if (value) *value = (float)v;
  }
}

orc_ctx *orc_create(const orc_config *cfg, int *status) {
  int st = ORC_OK;
  orc_ctx *c = NULL;
  if (!cfg) { st = ORC_ERR_ARG; goto out; }
  if (cfg->n_envs < 1 || cfg->hidden < 1 || cfg->n_actions < 1 || cfg->n_actions > 64 || cfg->obs_dim < 1) {
    st = ORC_ERR_CONFIG; goto out;
  }
  if (cfg->env_kind == ORC_ENV_CARTPOLE && (cfg->obs_dim != 4 || cfg->n_actions != 2)) { st = ORC_ERR_CONFIG; goto out; }
  if (cfg->env_kind == ORC_ENV_ACROBOT && (cfg->obs_dim != 6 || cfg->n_actions != 3)) { st = ORC_ERR_CONFIG; goto out; }
  if (cfg->env_kind == ORC_ENV_LINGAUSS && (cfg->obs_dim % 4 != 0 || !cfg->lg_A || !cfg->lg_B)) { st = ORC_ERR_CONFIG; goto out; }
  if (cfg->replay_capacity > 0 && (cfg->replay_capacity % cfg->n_envs != 0 || cfg->minibatch < 1)) { st = ORC_ERR_CONFIG; goto out; }
  if (cfg->replay_capacity == 0 && (cfg->rollout_len < 1 || cfg->n_segments < 1)) { st = ORC_ERR_CONFIG; goto out; }
  c = (orc_ctx *)calloc(1, sizeof(orc_ctx));
  c->cfg = *cfg;
  c->N = cfg->n_envs; c->D = cfg->obs_dim; c->A = cfg->n_actions; c->H = cfg->hidden;
  c->S_d = env_state_dim(cfg->env_kind, cfg->obs_dim);
  c->value_head = cfg->policy_kind == ORC_POLICY_CATEGORICAL;
  c->rec_words = 2 * c->D + 4;
  c->n_blob = orc_blob_floats(c->D, c->H, c->A, c->value_head);
  c->max_ep = cfg->max_episode_steps > 0 ? cfg->max_episode_steps : (cfg->env_kind == ORC_ENV_LINGAUSS ? 200 : 500);
  if (cfg->env_kind == ORC_ENV_LINGAUSS) {
    size_t nA = (size_t)c->D * c->D, nB = (size_t)c->A * c->D;
    c->lgA = (float *)malloc(sizeof(float) * nA); memcpy(c->lgA, cfg->lg_A, sizeof(float) * nA);
    c->lgB = (float *)malloc(sizeof(float) * nB); memcpy(c->lgB, cfg->lg_B, sizeof(float) * nB);
  }
  int N = c->N;
  c->state = (float *)calloc((size_t)N * c->S_d, sizeof(float));
  c->ep_step = (int32_t *)calloc(N, sizeof(int32_t));
  c->ep_return = (double *)calloc(N, sizeof(double));
  c->online = (float *)calloc(c->n_blob, sizeof(float));
  c->target = (float *)calloc(c->n_blob, sizeof(float));
  c->C = cfg->replay_capacity;
  if (c->C > 0) {
    c->ring = (float *)calloc((size_t)c->C * c->rec_words, sizeof(float));
    c->block_ver = (int32_t *)calloc((size_t)(c->C / N), sizeof(int32_t));
  } else {
    int T = cfg->rollout_len, G = cfg->n_segments;
    c->T = T; c->n_seg = G;
    size_t TN = (size_t)T * N;
    c->seg_obs = (float *)calloc(G * TN * c->D, sizeof(float));
    c->seg_act = (int32_t *)calloc(G * TN, sizeof(int32_t));
    c->seg_rew = (float *)calloc(G * TN, sizeof(float));
    c->seg_done = (uint8_t *)calloc(G * TN, 1);
    c->seg_logp = (float *)calloc(G * TN, sizeof(float));
    c->seg_val = (float *)calloc((size_t)G * (T + 1) * N, sizeof(float));
    c->seg_version = (int64_t *)calloc(G, sizeof(int64_t));
    c->seg_index = (int64_t *)calloc(G, sizeof(int64_t));
    c->seg_state = (int *)calloc(G, sizeof(int));
    for (int g = 0; g < G; ++g) c->seg_index[g] = -1;
  }
  c->l_obs = (float *)calloc((size_t)N * c->D, sizeof(float));
  c->l_next_obs = (float *)calloc((size_t)N * c->D, sizeof(float));
  c->l_logits = (float *)calloc((size_t)N * c->A, sizeof(float));
  c->l_rew = (float *)calloc(N, sizeof(float));
  c->l_logp = (float *)calloc(N, sizeof(float));
  c->l_value = (float *)calloc(N, sizeof(float));
  c->l_act = (int32_t *)calloc(N, sizeof(int32_t));
  c->l_done = (int32_t *)calloc(N, sizeof(int32_t));
  c->l_done_margin = (double *)calloc(N, sizeof(double));
  c->l_act_margin = (double *)calloc(N, sizeof(double));
  /* initial states: the reset stream at the all-ones step index, which no real step reaches */
  for (int e = 0; e < N; ++e) reset_env(c, e, ~(uint64_t)0, c->state + (size_t)e * c->S_d);
out:
  if (status) *status = st;
  return c;
}

void orc_destroy(orc_ctx *c) {
  if (!c) return;
  free(c->lgA); free(c->lgB); free(c->state); free(c->ep_step); free(c->ep_return); free(c->online);
  free(c->target); free(c->ring); free(c->block_ver); free(c->seg_obs); free(c->seg_act); free(c->seg_rew);
  free(c->seg_done); free(c->seg_logp); free(c->seg_val); free(c->seg_version); free(c->seg_index);
  free(c->seg_state); free(c->l_obs); free(c->l_next_obs); free(c->l_logits); free(c->l_rew); free(c->l_logp);
  free(c->l_value); free(c->l_act); free(c->l_done); free(c->l_done_margin); free(c->l_act_margin);
  free(c);
}

/* Learner hands a new parameter set over: it becomes version+1; the target network takes the same
 * parameters on the first publish and then whenever target_sync_interval learner steps have passed
 * since it last did. */
int orc_publish(orc_ctx *c, const float *blob, int64_t n_floats) {
  if (!c || !blob || n_floats != c->n_blob) return ORC_ERR_ARG;
  store_weights(c, blob, c->online);
  c->version += 1;
  if (!c->has_target || (c->cfg.target_sync_interval > 0 && c->k - c->k_last_sync >= c->cfg.target_sync_interval)) {
    memcpy(c->target, c->online, sizeof(float) * c->n_blob);
    c->has_target = 1;
    c->k_last_sync = c->k;
  }
  c->st.actor_version = c->st.learner_version = c->version;
  return (int)c->version;
}

static void one_actor_step(orc_ctx *c) {
  const int N = c->N, D = c->D, A = c->A, S_d = c->S_d;
  const uint64_t t = (uint64_t)c->t;
  const int32_t v_actor = (int32_t)c->version;
  const uint64_t thr = orc_explore_threshold(c->cfg.epsilon);
  const int on_policy = c->C == 0;
  int slot_seg = 0, p = 0;
  if (on_policy) {
    int64_t g = c->t / c->T;
    p = (int)(c->t % c->T);
    slot_seg = (int)(g % c->n_seg);
    if (p == 0) {
      if (c->seg_state[slot_seg] == 2) c->st.dropped_overwritten += (int64_t)c->T * N; /* never consumed */
      c->seg_state[slot_seg] = 1;
      c->seg_index[slot_seg] = g;
      c->seg_version[slot_seg] = c->version;
    }
  } else {
    c->block_ver[(c->cursor % (uint64_t)c->C) / (uint64_t)N] = v_actor;
  }
  float *s_next = (float *)malloc(sizeof(float) * S_d);
  double *noise = (double *)malloc(sizeof(double) * (S_d > 4 ? S_d : 4));
  for (int e = 0; e < N; ++e) {
    float *s = c->state + (size_t)e * S_d;
    float *obs = c->l_obs + (size_t)e * D, *logits = c->l_logits + (size_t)e * A;
    float value = 0.0f;
    /* task 1: policy inference */
    observe(c, s, obs);
    policy_forward(c, c->online, obs, logits, c->value_head ? &value : NULL);
    uint32_t w[4];
    orc_stream_words(c->cfg.seed, ORC_STREAM_ACTION, 0, (uint32_t)e, t, w);
    int a;
    double logp = 0.0, amargin = 0.0;
    if (c->cfg.policy_kind == ORC_POLICY_EPS_GREEDY) {
      a = orc_select_eps_greedy(logits, A, w[0], w[1], thr);
      /* greedy decision margin: gap between the two largest outputs (0 when exploring is irrelevant) */
      int best = orc_argmax_lowest(logits, A);
      double gap = 1e300;
      for (int i = 0; i < A; ++i)
        if (i != best && (double)logits[best] - (double)logits[i] < gap) gap = (double)logits[best] - (double)logits[i];
      amargin = ((uint64_t)w[0] < thr) ? 1e300 : gap;
    } else {
      a = orc_select_categorical(logits, A, orc_u01(w[0]), &logp, &amargin);
    }
    /* task 2: simulation */
    float r;
    int terminated;
    double dmargin;
    if (c->cfg.env_kind == ORC_ENV_CARTPOLE) orc_cartpole_step(s, a, s_next, &r, &terminated, &dmargin);
    else if (c->cfg.env_kind == ORC_ENV_ACROBOT) orc_acrobot_step(s, a, s_next, &r, &terminated, &dmargin);
    else {
      for (int b = 0; b < S_d / 4; ++b) {
        uint32_t nw[4];
        orc_stream_words(c->cfg.seed, ORC_STREAM_NOISE, (uint32_t)b, (uint32_t)e, t, nw);
        orc_normal4(nw, noise + 4 * b);
      }
      orc_lingauss_step(s, a, c->lgA, c->lgB, noise, D, (double)c->cfg.lg_noise_std, (double)c->cfg.lg_done_norm,
                        s_next, &r, &terminated, &dmargin);
    }
    c->ep_step[e] += 1;
    int truncated = c->ep_step[e] >= c->max_ep;
    int done = terminated || truncated;
    if (truncated) dmargin = 1e300; /* the step limit is an integer decision */
    float *next_obs = c->l_next_obs + (size_t)e * D;
    observe(c, s_next, next_obs);
    c->l_act[e] = a; c->l_rew[e] = r; c->l_done[e] = done;
    c->l_done_margin[e] = dmargin; c->l_act_margin[e] = amargin;
    c->l_logp[e] = (float)logp; c->l_value[e] = value;
    /* trajectory (s, a, r, s') with the version of the policy that produced it */
    if (on_policy) {
      size_t i = ((size_t)slot_seg * c->T + p) * N + e;
      memcpy(c->seg_obs + i * D, obs, sizeof(float) * D);
      c->seg_act[i] = a; c->seg_rew[i] = r; c->seg_done[i] = (uint8_t)done; c->seg_logp[i] = (float)logp;
      c->seg_val[((size_t)slot_seg * (c->T + 1) + p) * N + e] = value;
    } else {
      uint64_t slot = (c->cursor + (uint64_t)e) % (uint64_t)c->C;
      float *rec = c->ring + slot * c->rec_words;
      memcpy(rec, obs, sizeof(float) * D);
      memcpy(rec + D, next_obs, sizeof(float) * D);
      int32_t ai = a, di = done, vi = v_actor;
      memcpy(rec + 2 * D, &ai, 4);
      rec[2 * D + 1] = r;
      memcpy(rec + 2 * D + 2, &di, 4);
      memcpy(rec + 2 * D + 3, &vi, 4);
    }
    c->ep_return[e] += (double)r;
    if (done) {
      c->st.episodes_finished += 1;
      c->st.return_sum += c->ep_return[e];
      c->ep_return[e] = 0.0;
      reset_env(c, e, t, s);
      c->ep_step[e] = 0;
    } else {
      memcpy(s, s_next, sizeof(float) * S_d);
    }
  }
  if (on_policy && p == c->T - 1) {
    /* bootstrap value of the state each env is in after the last step of the segment */
    float *obs = (float *)malloc(sizeof(float) * D), *lg = (float *)malloc(sizeof(float) * A);
    for (int e = 0; e < N; ++e) {
      float value = 0.0f;
      observe(c, c->state + (size_t)e * S_d, obs);
      policy_forward(c, c->online, obs, lg, &value);
      c->seg_val[((size_t)slot_seg * (c->T + 1) + c->T) * N + e] = value;
    }
    free(obs); free(lg);
    c->seg_state[slot_seg] = 2;
  }
  free(s_next); free(noise);
  if (!on_policy) c->cursor += (uint64_t)N;
  c->t += 1;
  c->st.produced += N;
  c->st.actor_steps += 1;
}

int orc_actor_step(orc_ctx *c, int n_steps) {
  if (!c || n_steps < 0) return ORC_ERR_ARG;
  if (c->version == 0) return ORC_ERR_NO_WEIGHTS;
  for (int i = 0; i < n_steps; ++i) one_actor_step(c);
  return ORC_OK;
}

/* Staleness-bounded uniform sampling with replacement.  The eligible set E holds every valid slot whose
 * version tag is at most `bound` versions behind the learner, in ascending slot order; draw j of learner
 * step k takes E[mulhi(x0, |E|)] with x0 from the SAMPLE stream at (j, k). */
int orc_sample(orc_ctx *c, int staleness_bound, int32_t *idx_out, float *records_out) {
  if (!c || c->C == 0 || !idx_out) return ORC_ERR_ARG;
  if (c->version == 0) return ORC_ERR_NO_WEIGHTS;
  const int64_t S = staleness_bound >= 0 ? staleness_bound : c->cfg.staleness_bound;
  const int64_t valid = c->cursor < (uint64_t)c->C ? (int64_t)c->cursor : c->C;
  if (valid < c->cfg.warmup) return ORC_ERR_WARMUP;
  const int64_t v_learner = c->version;
  int32_t *E = (int32_t *)malloc(sizeof(int32_t) * (size_t)(valid > 0 ? valid : 1));
  int64_t nE = 0;
  for (int64_t i = 0; i < valid; ++i) {
    int32_t ver;
    memcpy(&ver, c->ring + (size_t)i * c->rec_words + 2 * c->D + 3, 4);
    if (v_learner - (int64_t)ver <= S) E[nE++] = (int32_t)i;
  }
  if (nE == 0) { free(E); c->st.starved_calls += 1; return ORC_ERR_STARVED; }
  const int B = c->cfg.minibatch;
  for (int j = 0; j < B; ++j) {
    uint32_t w[4];
    orc_stream_words(c->cfg.seed, ORC_STREAM_SAMPLE, 0, (uint32_t)j, (uint64_t)c->k, w);
    int32_t slot = E[orc_mulhi(w[0], (uint32_t)nE)];
    idx_out[j] = slot;
    const float *rec = c->ring + (size_t)slot * c->rec_words;
    if (records_out) memcpy(records_out + (size_t)j * c->rec_words, rec, sizeof(float) * c->rec_words);
    int32_t ver;
    memcpy(&ver, rec + 2 * c->D + 3, 4);
    int64_t stale = v_learner - (int64_t)ver;
    if (stale > c->st.max_sampled_staleness) c->st.max_sampled_staleness = stale;
    c->st.staleness_hist[stale > 32 ? 32 : stale] += 1;
  }
  c->st.dropped_stale += valid - nE; /* resident records this call could not use */
  free(E);
  c->k += 1;
  c->st.learner_steps += 1;
  c->st.consumed += B;
  return ORC_OK;
}

/* Forward half of the policy update on a gathered minibatch: q = Q_online(s)[a], q' = max_a Q_target(s'),
 * TD error and Huber loss per sample, mean loss. */
int orc_td(orc_ctx *c, const float *records, int n, double *td, double *huber, double *loss_mean, double *q_sel,
           double *q_next_max) {
  if (!c || !records || n < 1) return ORC_ERR_ARG;
  if (c->version == 0) return ORC_ERR_NO_WEIGHTS;
  const int D = c->D, A = c->A;
  float *q = (float *)malloc(sizeof(float) * A), *qn = (float *)malloc(sizeof(float) * A);
  double sum = 0.0;
  for (int j = 0; j < n; ++j) {
    const float *rec = records + (size_t)j * c->rec_words;
    int32_t a, d;
    memcpy(&a, rec + 2 * D, 4);
    memcpy(&d, rec + 2 * D + 2, 4);
    policy_forward(c, c->online, rec, q, NULL);
    policy_forward(c, c->target, rec + D, qn, NULL);
    double qmax = (double)qn[orc_argmax_lowest(qn, A)];
    double t_, h_;
    orc_td_one((double)q[a], qmax, (double)rec[2 * D + 1], d, (double)c->cfg.gamma, (double)c->cfg.huber_delta, &t_, &h_);
    if (td) td[j] = t_;
    if (huber) huber[j] = h_;
    if (q_sel) q_sel[j] = (double)q[a];
    if (q_next_max) q_next_max[j] = qmax;
    sum += h_;
  }
  if (loss_mean) *loss_mean = sum / (double)n;
  free(q); free(qn);
  return ORC_OK;
}

/* On-policy consumption: the oldest complete, unconsumed segment whose policy version is at most
 * staleness_bound versions behind; staler ones are dropped and counted. */
int orc_segment_acquire(orc_ctx *c, orc_segment *out) {
  if (!c || c->C != 0 || !out) return ORC_ERR_ARG;
  const int N = c->N, T = c->T;
  int64_t n_started = (c->t + T - 1) / T; /* segments begun so far */
  if (c->next_consume < n_started - c->n_seg) c->next_consume = n_started - c->n_seg; /* overwritten ones */
  while (c->next_consume < n_started) {
    int slot = (int)(c->next_consume % c->n_seg);
    if (c->seg_index[slot] != c->next_consume || c->seg_state[slot] != 2) {
      if (c->seg_index[slot] == c->next_consume && c->seg_state[slot] == 1) break; /* still filling */
      c->next_consume += 1;
      continue;
    }
    if (c->version - c->seg_version[slot] > c->cfg.staleness_bound) {
      c->seg_state[slot] = 3;
      c->st.dropped_stale += (int64_t)T * N;
      c->next_consume += 1;
      continue;
    }
    size_t TN = (size_t)T * N;
    out->T = T; out->N = N; out->version = c->seg_version[slot];
    out->obs = c->seg_obs + slot * TN * c->D;
    out->act = c->seg_act + slot * TN;
    out->rew = c->seg_rew + slot * TN;
    out->done = c->seg_done + slot * TN;
    out->logp = c->seg_logp + slot * TN;
    out->val = c->seg_val + (size_t)slot * (T + 1) * N;
    c->seg_state[slot] = 3;
    c->next_consume += 1;
    c->k += 1;
    c->st.learner_steps += 1;
    c->st.consumed += (int64_t)T * N;
    int64_t stale = c->version - out->version;
    if (stale > c->st.max_sampled_staleness) c->st.max_sampled_staleness = stale;
    c->st.staleness_hist[stale > 32 ? 32 : stale] += (int64_t)T * N;
    return ORC_OK;
  }
  c->st.starved_calls += 1;
  return ORC_ERR_STARVED;
}

void orc_get_stats(const orc_ctx *c, orc_stats *out) {
  *out = c->st;
  out->actor_version = out->learner_version = c->version;
}

int orc_state_dim(const orc_ctx *c) { return c->S_d; }
int orc_record_words(const orc_ctx *c) { return c->rec_words; }
float *orc_state(orc_ctx *c) { return c->state; }
int32_t *orc_ep_step(orc_ctx *c) { return c->ep_step; }
void orc_set_counters(orc_ctx *c, uint64_t cursor, int64_t t, int64_t k) { c->cursor = cursor; c->t = t; c->k = k; }
uint64_t orc_cursor(const orc_ctx *c) { return c->cursor; }
float *orc_ring(orc_ctx *c) { return c->ring; }
int32_t *orc_block_version(orc_ctx *c) { return c->block_ver; }
const float *orc_last_obs(const orc_ctx *c) { return c->l_obs; }
const float *orc_last_logits(const orc_ctx *c) { return c->l_logits; }
const int32_t *orc_last_act(const orc_ctx *c) { return c->l_act; }
const float *orc_last_rew(const orc_ctx *c) { return c->l_rew; }
const int32_t *orc_last_done(const orc_ctx *c) { return c->l_done; }
const float *orc_last_next_obs(const orc_ctx *c) { return c->l_next_obs; }
const double *orc_last_done_margin(const orc_ctx *c) { return c->l_done_margin; }
const double *orc_last_act_margin(const orc_ctx *c) { return c->l_act_margin; }
const float *orc_last_logp(const orc_ctx *c) { return c->l_logp; }
const float *orc_last_value(const orc_ctx *c) { return c->l_value; }
const float *orc_online_blob(const orc_ctx *c) { return c->online; }
const float *orc_target_blob(const orc_ctx *c) { return c->target; }
