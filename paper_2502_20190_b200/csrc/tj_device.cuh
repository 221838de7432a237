// Device-side building blocks: Philox4x32-10, uniform / normal transforms, the three
// environment steps and the two action-selection rules.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tj {

enum : uint32_t { STREAM_ACTION = 0, STREAM_RESET = 1, STREAM_NOISE = 2, STREAM_SAMPLE = 3, STREAM_SHUFFLE = 4 };

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and xors, the key
// advancing by the two Weyl constants each round.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // one widening multiply per product (both halves at once), one three-input xor per output word
    const unsigned long long p0 = (unsigned long long)M0 * c.x, p1 = (unsigned long long)M1 * c.z;
    c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ k.x, (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ k.y, (uint32_t)p0);
    k.x += W0;
    k.y += W1;
  }
  return c;
}

// counter = (index, step low, stream | block << 8, step high), key = seed
__device__ __forceinline__ uint4 stream_words(uint2 seed, uint32_t stream, uint32_t block, uint32_t index,
                                              unsigned long long step) {
  return philox4x32_10(make_uint4(index, (uint32_t)step, stream | (block << 8), (uint32_t)(step >> 32)), seed);
}

// top 23 bits plus one half, times 2^-23: exact in FP32, strictly inside (0,1)
__device__ __forceinline__ float u01(uint32_t x) { return ((float)(x >> 9) + 0.5f) * (1.0f / 8388608.0f); }

// U(lo, lo+width) as a single fused multiply-add (one rounding)
__device__ __forceinline__ float uniform_range(uint32_t x, float lo, float width) { return fmaf(u01(x), width, lo); }

// two standard normals from two words (Box-Muller); 2*u2 is exact, so the *pi functions see the exact angle
__device__ __forceinline__ float2 box_muller(uint32_t a, uint32_t b) {
  const float r = sqrtf(-2.0f * logf(u01(a)));
  float s, c;
  sincospif(2.0f * u01(b), &s, &c);
  return make_float2(r * c, r * s);
}

// ------------------------------------------------------------------ CartPole
// Frictionless cart-pole, explicit Euler with the positions advanced by the old velocities.
struct StepResult {
  float reward;
  bool terminated;
};

__device__ __forceinline__ StepResult cartpole_step(float4 s, int a, float4& sn) {
  constexpr float g = 9.8f, masspole = 0.1f, total_mass = 1.1f, length = 0.5f, polemass_length = 0.05f,
                  force_mag = 10.0f, tau = 0.02f;
  const float force = (a == 1) ? force_mag : -force_mag;
  float sinth, costh;
  sincosf(s.z, &sinth, &costh);
  const float temp = (force + polemass_length * s.w * s.w * sinth) / total_mass;
  const float thetaacc = (g * sinth - costh * temp) / (length * (4.0f / 3.0f - masspole * costh * costh / total_mass));
  const float xacc = temp - polemass_length * thetaacc * costh / total_mass;
  sn.x = s.x + tau * s.y;
  sn.y = s.y + tau * xacc;
  sn.z = s.z + tau * s.w;
  sn.w = s.w + tau * thetaacc;
  constexpr float x_thr = 2.4f;
  constexpr float th_thr = (float)(12.0 * 2.0 * 3.14159265358979323846 / 360.0);
  StepResult r;
  r.reward = 1.0f;
  r.terminated = (fabsf(sn.x) > x_thr) || (fabsf(sn.z) > th_thr);
  return r;
}

// ------------------------------------------------------------------ Acrobot
// Two-link pendulum (Sutton & Barto), torque on the second joint, angles from the downward vertical.
__device__ __forceinline__ float4 acrobot_deriv(float4 y, float torque) {
  constexpr float m1 = 1.0f, m2 = 1.0f, l1 = 1.0f, lc1 = 0.5f, lc2 = 0.5f, I1 = 1.0f, I2 = 1.0f, g = 9.8f;
  const float th1 = y.x, th2 = y.y, w1 = y.z, w2 = y.w;
  float s2, c2;
  sincosf(th2, &s2, &c2);
  const float d1 = m1 * lc1 * lc1 + m2 * (l1 * l1 + lc2 * lc2 + 2.0f * l1 * lc2 * c2) + I1 + I2;
  const float d2 = m2 * (lc2 * lc2 + l1 * lc2 * c2) + I2;
  const float phi2 = m2 * lc2 * g * sinf(th1 + th2);
  const float phi1 = -m2 * l1 * lc2 * w2 * w2 * s2 - 2.0f * m2 * l1 * lc2 * w2 * w1 * s2 +
                     (m1 * lc1 + m2 * l1) * g * sinf(th1) + phi2;
  const float ddth2 = (torque + d2 / d1 * phi1 - m2 * l1 * lc2 * w1 * w1 * s2 - phi2) / (m2 * lc2 * lc2 + I2 - d2 * d2 / d1);
  const float ddth1 = -(d2 * ddth2 + phi1) / d1;
  return make_float4(w1, w2, ddth1, ddth2);
}

__device__ __forceinline__ float4 axpy4(float4 y, float h, float4 k) {
  return make_float4(y.x + h * k.x, y.y + h * k.y, y.z + h * k.z, y.w + h * k.w);
}

__device__ __forceinline__ float wrap_pi(float x) {
  constexpr float PI = 3.14159265358979323846f, TWO_PI = 6.28318530717958647692f;
  return x - TWO_PI * floorf((x + PI) / TWO_PI);
}

__device__ __forceinline__ StepResult acrobot_step(float4 s, int a, float4& sn) {
  constexpr float dt = 0.2f, PI = 3.14159265358979323846f;
  const float torque = (float)(a - 1);
  const float4 k1 = acrobot_deriv(s, torque);
  const float4 k2 = acrobot_deriv(axpy4(s, 0.5f * dt, k1), torque);
  const float4 k3 = acrobot_deriv(axpy4(s, 0.5f * dt, k2), torque);
  const float4 k4 = acrobot_deriv(axpy4(s, dt, k3), torque);
  float4 y;
  y.x = s.x + dt / 6.0f * (k1.x + 2.0f * k2.x + 2.0f * k3.x + k4.x);
  y.y = s.y + dt / 6.0f * (k1.y + 2.0f * k2.y + 2.0f * k3.y + k4.y);
  y.z = s.z + dt / 6.0f * (k1.z + 2.0f * k2.z + 2.0f * k3.z + k4.z);
  y.w = s.w + dt / 6.0f * (k1.w + 2.0f * k2.w + 2.0f * k3.w + k4.w);
  sn.x = wrap_pi(y.x);
  sn.y = wrap_pi(y.y);
  sn.z = fminf(fmaxf(y.z, -4.0f * PI), 4.0f * PI);
  sn.w = fminf(fmaxf(y.w, -9.0f * PI), 9.0f * PI);
  const float tip = -cosf(sn.x) - cosf(sn.x + sn.y);
  StepResult r;
  r.terminated = tip > 1.0f;
  r.reward = r.terminated ? 0.0f : -1.0f;
  return r;
}

// ------------------------------------------------------------------ action selection
// greedy: strict '>' scan, so the lowest index wins ties and NaN never wins
template <typename GetLogit>
__device__ __forceinline__ int argmax_lowest(int A, GetLogit q) {
  int best = 0;
  float qb = q(0);
  for (int i = 1; i < A; ++i) {
    const float qi = q(i);
    if (qi > qb) { qb = qi; best = i; }
  }
  return best;
}

// explore iff x0 < floor(eps * 2^32); the random action is the high word of x1 * A
template <typename GetLogit>
__device__ __forceinline__ int select_eps_greedy(int A, GetLogit q, uint4 w, unsigned long long threshold) {
  if ((unsigned long long)w.x < threshold) return (int)__umulhi(w.y, (uint32_t)A);
  return argmax_lowest(A, q);
}

// inverse-CDF draw over softmax(logits): smallest i whose cumulative mass exceeds u * Z
template <typename GetLogit>
__device__ __forceinline__ int select_categorical(int A, GetLogit q, float u, float& logp) {
  float m = q(0);
  for (int i = 1; i < A; ++i) m = fmaxf(m, q(i));
  float Z = 0.0f;
  for (int i = 0; i < A; ++i) Z += expf(q(i) - m);
  const float target = u * Z;
  float cum = 0.0f;
  int a = A - 1;
  bool found = false;
  for (int i = 0; i < A; ++i) {
    cum += expf(q(i) - m);
    if (!found && cum > target) { a = i; found = true; }
  }
  logp = q(a) - m - logf(Z);
  return a;
}

}  // namespace tj
