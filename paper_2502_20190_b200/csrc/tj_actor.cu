// Actor kernel: policy inference, action selection, environment step and the version-tagged trajectory
// write for a tile of environments, looped over n_steps inside one launch.
//
// Environments are independent, so a thread block keeps its TE environments for the whole call: state lives
// in registers (CartPole, Acrobot) or shared memory (linear-Gaussian) between steps, and no block ever waits
// on another.  The ring cursor advances by N per step, which every block can compute on its own.
#include "tj_async.cuh"
#include "tj_device.cuh"
#include "tj_internal.h"
#include "tj_mlp.cuh"

namespace tj {

namespace {

struct ActorSmem {
  float *w, *xs, *h1, *h2, *out, *nxt, *rew;
  int *act, *done;
};

// STAGE: 0 = parameters read from global memory, 1 = everything but the HxH matrix staged in shared memory,
//        2 = all parameters staged.
__host__ __device__ inline size_t staged_floats(int stage, size_t w_total, size_t off_W2t, size_t off_b2) {
  if (stage == 2) return w_total;
  if (stage == 1) return w_total - (off_b2 - off_W2t);
  return 0;
}

__host__ __device__ inline size_t actor_smem_floats(int TE, int D, int Hp, int Ap, bool lingauss, size_t staged) {
  const int Dx = (D + 3) & ~3;
  size_t n = staged + (size_t)Dx * TE + 2 * (size_t)Hp * TE + (size_t)Ap * TE;
  if (lingauss) n += (size_t)Dx * TE;
  n += 3 * TE;  // rew, act, done
  return n;
}

__device__ inline ActorSmem carve(float* base, int TE, int D, int Hp, int Ap, bool lingauss, size_t staged) {
  const int Dx = (D + 3) & ~3;
  ActorSmem s;
  s.w = base; base += staged;
  s.xs = base; base += (size_t)Dx * TE;
  s.h1 = base; base += (size_t)Hp * TE;
  s.h2 = base; base += (size_t)Hp * TE;
  s.out = base; base += (size_t)Ap * TE;
  s.nxt = base;
  if (lingauss) base += (size_t)Dx * TE;
  s.rew = base; base += TE;
  s.act = reinterpret_cast<int*>(base); base += TE;
  s.done = reinterpret_cast<int*>(base);
  return s;
}

__device__ __forceinline__ float4 reset4(uint2 seed, uint32_t block, uint32_t e, unsigned long long step, float lo,
                                         float width) {
  const uint4 w = stream_words(seed, STREAM_RESET, block, e, step);
  return make_float4(uniform_range(w.x, lo, width), uniform_range(w.y, lo, width), uniform_range(w.z, lo, width),
                     uniform_range(w.w, lo, width));
}

// ------------------------------------------------------------------------------------------------
// CartPole / Acrobot: one thread owns one environment (state in registers).
// ------------------------------------------------------------------------------------------------
template <int TE, int NT, int EPT, int NPT, int ENV, int STAGE>
__global__ void __launch_bounds__(NT) actor_small_env_kernel(const ActorParams p) {
  extern __shared__ __align__(128) float smem[];
  __shared__ __align__(8) uint64_t wbar;
  const ActorSmem sm = carve(smem, TE, p.D, p.Hp, p.Ap, false, staged_floats(STAGE, p.w_total, p.off_W2t, p.off_b2));
  const int tid = threadIdx.x;
  const int e = blockIdx.x * TE + tid;
  const bool owner = tid < TE && e < p.N;
  const bool on_policy = p.C == 0;
  if (STAGE > 0) {
    if (tid == 0) mbar_init(&wbar, 1);
    __syncthreads();
  }
  const MlpWeights mw = stage_mlp_weights<STAGE>(p, p.W, sm.w, &wbar, tid == 0);

  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  int ep = 0;
  float ep_ret = 0.f;
  if (owner) {
    s = reinterpret_cast<const float4*>(p.state)[e];
    ep = p.ep_step[e];
    ep_ret = p.ep_return[e];
  }
  unsigned long long n_episodes = 0;
  double ret_sum = 0.0;
  if (STAGE > 0 && !mbar_wait_bounded(&wbar, 0)) {  // parameters never arrived: flag it and leave
    if (tid == 0) atomicExch(&p.stats->error, 1ull);
    return;
  }

  for (int step = 0; step < p.n_steps; ++step) {
    const unsigned long long t = (unsigned long long)p.t0 + step;
    // observation -> xs[k][e]
    float obs[6];
    if (ENV == TJ_ENV_CARTPOLE) {
      obs[0] = s.x; obs[1] = s.y; obs[2] = s.z; obs[3] = s.w; obs[4] = obs[5] = 0.f;
    } else {
      float s1, c1, s2, c2;
      sincosf(s.x, &s1, &c1);
      sincosf(s.y, &s2, &c2);
      obs[0] = c1; obs[1] = s1; obs[2] = c2; obs[3] = s2; obs[4] = s.z; obs[5] = s.w;
    }
    if (tid < TE) {
#pragma unroll
      for (int k = 0; k < 6; ++k)
        if (k < p.D) sm.xs[k * TE + tid] = owner ? obs[k] : 0.f;
    }
    __syncthreads();
    mlp_forward_tile<TE, NT, EPT, (STAGE > 0), (STAGE == 2), NPT>(mw, p.D, p.H, p.Hp, p.Aout, p.Ap, sm.xs, sm.h1, sm.h2, sm.out);
    if (owner) {
      auto logit = [&](int i) { return sm.out[i * TE + tid]; };
      if (p.dbg_logits) {
        float* dl = p.dbg_logits + ((size_t)step * p.N + e) * p.A;
        for (int i = 0; i < p.A; ++i) dl[i] = logit(i);
      }
      const uint4 w = stream_words(p.seed, STREAM_ACTION, 0, (uint32_t)e, t);
      int a;
      float logp = 0.f;
      if (p.policy_kind == TJ_POLICY_EPS_GREEDY) a = select_eps_greedy(p.A, logit, w, p.explore_thr);
      else a = select_categorical(p.A, logit, u01(w.x), logp);
      float4 sn;
      const StepResult r = (ENV == TJ_ENV_CARTPOLE) ? cartpole_step(s, a, sn) : acrobot_step(s, a, sn);
      ep += 1;
      const int done = (r.terminated || ep >= p.max_ep) ? 1 : 0;
      if (on_policy) {
        const long long g = (long long)(t / (unsigned long long)p.T);
        const int pos = (int)(t % (unsigned long long)p.T);
        const int slot = (int)(g % p.G);
        const size_t i = ((size_t)slot * p.T + pos) * p.N + e;
        float* so = p.seg_obs + i * p.D;
        if (ENV == TJ_ENV_CARTPOLE) *reinterpret_cast<float4*>(so) = s;
        else
          for (int k = 0; k < 6; ++k) so[k] = obs[k];
        p.seg_act[i] = a;
        p.seg_rew[i] = r.reward;
        p.seg_done[i] = (uint8_t)done;
        p.seg_logp[i] = logp;
        p.seg_val[((size_t)slot * (p.T + 1) + pos) * p.N + e] = logit(p.A);  // value head = column A
      } else {
        const unsigned long long slot = (p.cursor0 + (unsigned long long)step * p.N + e) % (unsigned long long)p.C;
        float4* rec = reinterpret_cast<float4*>(p.ring + slot * p.rec_words);
        const float4 tail = make_float4(__int_as_float(a), r.reward, __int_as_float(done), __int_as_float(p.version));
        if (ENV == TJ_ENV_CARTPOLE) {
          rec[0] = s;
          rec[1] = sn;
          rec[2] = tail;
        } else {
          float s1, c1, s2, c2;
          sincosf(sn.x, &s1, &c1);
          sincosf(sn.y, &s2, &c2);
          rec[0] = make_float4(obs[0], obs[1], obs[2], obs[3]);
          rec[1] = make_float4(obs[4], obs[5], c1, s1);
          rec[2] = make_float4(c2, s2, sn.z, sn.w);
          rec[3] = tail;
        }
      }
      ep_ret += r.reward;
      if (done) {
        n_episodes += 1;
        ret_sum += (double)ep_ret;
        ep_ret = 0.f;
        ep = 0;
        s = (ENV == TJ_ENV_CARTPOLE) ? reset4(p.seed, 0, (uint32_t)e, t, -0.05f, 0.1f)
                                     : reset4(p.seed, 0, (uint32_t)e, t, -0.1f, 0.2f);
      } else {
        s = sn;
      }
    }
    if (!on_policy && blockIdx.x == 0 && tid == 0)
      p.block_ver[((p.cursor0 + (unsigned long long)step * p.N) % (unsigned long long)p.C) / p.N] = p.version;
    __syncthreads();
    // last step of a segment: bootstrap value of the state each env is now in
    if (on_policy && (int)(t % (unsigned long long)p.T) == p.T - 1) {
      if (tid < TE) {
        float o2[6];
        if (ENV == TJ_ENV_CARTPOLE) {
          o2[0] = s.x; o2[1] = s.y; o2[2] = s.z; o2[3] = s.w; o2[4] = o2[5] = 0.f;
        } else {
          float s1, c1, s2, c2;
          sincosf(s.x, &s1, &c1);
          sincosf(s.y, &s2, &c2);
          o2[0] = c1; o2[1] = s1; o2[2] = c2; o2[3] = s2; o2[4] = s.z; o2[5] = s.w;
        }
#pragma unroll
        for (int k = 0; k < 6; ++k)
          if (k < p.D) sm.xs[k * TE + tid] = owner ? o2[k] : 0.f;
      }
      __syncthreads();
      mlp_forward_tile<TE, NT, EPT, (STAGE > 0), (STAGE == 2), NPT>(mw, p.D, p.H, p.Hp, p.Aout, p.Ap, sm.xs, sm.h1, sm.h2, sm.out);
      if (owner) {
        const int slot = (int)((long long)(t / (unsigned long long)p.T) % p.G);
        p.seg_val[((size_t)slot * (p.T + 1) + p.T) * p.N + e] = sm.out[p.A * TE + tid];
      }
      __syncthreads();
    }
  }
  if (owner) {
    reinterpret_cast<float4*>(p.state)[e] = s;
    p.ep_step[e] = ep;
    p.ep_return[e] = ep_ret;
    if (n_episodes) {
      atomicAdd(&p.stats->episodes, n_episodes);
      atomicAdd(&p.stats->return_sum, ret_sum);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Linear-Gaussian env: the state (= observation) of the tile lives in shared memory, k-major.
// ------------------------------------------------------------------------------------------------
template <int TE, int NT>
__global__ void __launch_bounds__(NT) actor_lingauss_kernel(const ActorParams p) {
  extern __shared__ __align__(128) float smem[];
  const bool ext = p.logits_in != nullptr;   // network outputs come from the tensor-core kernel
  const ActorSmem sm = carve(smem, TE, p.D, ext ? 0 : p.Hp, ext ? 0 : p.Ap, true, 0);
  __shared__ uint64_t unused_bar;
  const MlpWeights mw = stage_mlp_weights<0>(p, p.W, nullptr, &unused_bar, false);
  const int tid = threadIdx.x;
  const int e0 = blockIdx.x * TE;
  const int D = p.D, Dp = (p.D + 3) & ~3;
  const int n_here = min(TE, p.N - e0);

  // state -> xs[k][e]
  for (int i = tid; i < TE * D; i += NT) {
    const int el = i / D, k = i % D;
    sm.xs[k * TE + el] = el < n_here ? p.state[(size_t)(e0 + el) * D + k] : 0.f;
  }
  int ep = 0;
  float ep_ret = 0.f;
  if (tid < n_here) {
    ep = p.ep_step[e0 + tid];
    ep_ret = p.ep_return[e0 + tid];
  }
  unsigned long long n_episodes = 0;
  double ret_sum = 0.0;
  __syncthreads();

  for (int step = 0; step < p.n_steps; ++step) {
    const unsigned long long t = (unsigned long long)p.t0 + step;
    if (!ext) mlp_forward_tile<TE, NT, 4, false, false>(mw, D, p.H, p.Hp, p.Aout, p.Ap, sm.xs, sm.h1, sm.h2, sm.out);
    if (tid < TE) {
      int a = 0;
      if (tid < n_here) {
        const int e = e0 + tid;
        auto logit = [&](int i) { return ext ? p.logits_in[(size_t)e * p.A + i] : sm.out[i * TE + tid]; };
        if (p.dbg_logits) {
          float* dl = p.dbg_logits + ((size_t)step * p.N + e) * p.A;
          for (int i = 0; i < p.A; ++i) dl[i] = logit(i);
        }
        const uint4 w = stream_words(p.seed, STREAM_ACTION, 0, (uint32_t)e, t);
        a = select_eps_greedy(p.A, logit, w, p.explore_thr);
      }
      sm.act[tid] = a;
    }
    __syncthreads();
    // s' = tanh(A s + B[a]) ...
    dense_layer<TE, NT, 4, ACT_TANH, true, false>(p.lgAt, p.lgB, Dp, D, D, sm.xs, sm.nxt, sm.act);
    __syncthreads();
    // ... + noise_std * n, four normals per Philox call
    for (int i = tid; i < TE * (D / 4); i += NT) {
      const int el = i % TE, b = i / TE;
      if (el < n_here) {
        const uint4 w = stream_words(p.seed, STREAM_NOISE, (uint32_t)b, (uint32_t)(e0 + el), t);
        const float2 z01 = box_muller(w.x, w.y), z23 = box_muller(w.z, w.w);
        sm.nxt[(4 * b + 0) * TE + el] += p.lg_noise_std * z01.x;
        sm.nxt[(4 * b + 1) * TE + el] += p.lg_noise_std * z01.y;
        sm.nxt[(4 * b + 2) * TE + el] += p.lg_noise_std * z23.x;
        sm.nxt[(4 * b + 3) * TE + el] += p.lg_noise_std * z23.y;
      }
    }
    __syncthreads();
    if (tid < TE) {
      int done = 0;
      float rew = 0.f;
      if (tid < n_here) {
        float sq = 0.f;
        for (int k = 0; k < D; ++k) {
          const float v = sm.nxt[k * TE + tid];
          sq = fmaf(v, v, sq);
        }
        rew = -sq / (float)D;
        ep += 1;
        done = (sqrtf(sq) > p.lg_done_norm || ep >= p.max_ep) ? 1 : 0;
        ep_ret += rew;
        if (done) {
          n_episodes += 1;
          ret_sum += (double)ep_ret;
          ep_ret = 0.f;
          ep = 0;
        }
      }
      sm.done[tid] = done;
      sm.rew[tid] = rew;
    }
    __syncthreads();
    // record rows: [obs D][next_obs D][act, rew, done, ver]
    {
      const int rw = p.rec_words;
      for (int i = tid; i < n_here * rw; i += NT) {
        const int el = i / rw, w = i % rw;
        const unsigned long long slot = (p.cursor0 + (unsigned long long)step * p.N + (e0 + el)) % (unsigned long long)p.C;
        float v;
        if (w < D) v = sm.xs[w * TE + el];
        else if (w < 2 * D) v = sm.nxt[(w - D) * TE + el];
        else if (w == 2 * D) v = __int_as_float(sm.act[el]);
        else if (w == 2 * D + 1) v = sm.rew[el];
        else if (w == 2 * D + 2) v = __int_as_float(sm.done[el]);
        else v = __int_as_float(p.version);
        p.ring[slot * rw + w] = v;
      }
    }
    if (blockIdx.x == 0 && tid == 0)
      p.block_ver[((p.cursor0 + (unsigned long long)step * p.N) % (unsigned long long)p.C) / p.N] = p.version;
    __syncthreads();
    // next state: the stepped state, or a fresh draw for finished episodes
    for (int i = tid; i < TE * (D / 4); i += NT) {
      const int el = i % TE, b = i / TE;
      float4 v;
      if (el < n_here && sm.done[el]) {
        v = reset4(p.seed, (uint32_t)b, (uint32_t)(e0 + el), t, -0.1f, 0.2f);
      } else {
        v = make_float4(sm.nxt[(4 * b + 0) * TE + el], sm.nxt[(4 * b + 1) * TE + el], sm.nxt[(4 * b + 2) * TE + el],
                        sm.nxt[(4 * b + 3) * TE + el]);
      }
      sm.xs[(4 * b + 0) * TE + el] = v.x;
      sm.xs[(4 * b + 1) * TE + el] = v.y;
      sm.xs[(4 * b + 2) * TE + el] = v.z;
      sm.xs[(4 * b + 3) * TE + el] = v.w;
    }
    __syncthreads();
  }
  for (int i = tid; i < n_here * D; i += NT) {
    const int el = i / D, k = i % D;
    p.state[(size_t)(e0 + el) * D + k] = sm.xs[k * TE + el];
  }
  if (tid < n_here) {
    p.ep_step[e0 + tid] = ep;
    p.ep_return[e0 + tid] = ep_ret;
    if (n_episodes) {
      atomicAdd(&p.stats->episodes, n_episodes);
      atomicAdd(&p.stats->return_sum, ret_sum);
    }
  }
}

__global__ void init_env_kernel(int env_kind, int N, int S_d, uint2 seed, float* state, int* ep_step, float* ep_return) {
  const int nb = S_d / 4;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)N * nb) return;
  const int e = (int)(i / nb), b = (int)(i % nb);
  const float lo = env_kind == TJ_ENV_CARTPOLE ? -0.05f : -0.1f, width = env_kind == TJ_ENV_CARTPOLE ? 0.1f : 0.2f;
  reinterpret_cast<float4*>(state + (size_t)e * S_d)[b] = reset4(seed, (uint32_t)b, (uint32_t)e, ~0ull, lo, width);
  if (b == 0) {
    ep_step[e] = 0;
    ep_return[e] = 0.f;
  }
}

template <typename K>
cudaError_t launch_with_smem(K kernel, int grid, int threads, size_t smem_bytes, const ActorParams& p, cudaStream_t s) {
  if (smem_bytes > 48 * 1024) {
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (err != cudaSuccess) return err;
  }
  kernel<<<grid, threads, smem_bytes, s>>>(p);
  return cudaGetLastError();
}

constexpr size_t kSmemMax = 227 * 1024 - 1024;   // per block, leaving room for static shared memory
constexpr size_t kSmemTwoPerSm = 112 * 1024;     // two resident blocks per SM

template <int TE, int NT, int EPT, int NPT, int ENV>
cudaError_t launch_small(int stage, size_t smem, const ActorParams& p, cudaStream_t s) {
  const int grid = (p.N + TE - 1) / TE;
  if (stage == 2) return launch_with_smem(actor_small_env_kernel<TE, NT, EPT, NPT, ENV, 2>, grid, NT, smem, p, s);
  if (stage == 1) return launch_with_smem(actor_small_env_kernel<TE, NT, EPT, NPT, ENV, 1>, grid, NT, smem, p, s);
  return launch_with_smem(actor_small_env_kernel<TE, NT, EPT, NPT, ENV, 0>, grid, NT, smem, p, s);
}

}  // namespace

cudaError_t launch_init_env(int env_kind, int N, int S_d, uint2 seed, float* state, int* ep_step, float* ep_return,
                            cudaStream_t s) {
  const long long n = (long long)N * (S_d / 4);
  init_env_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(env_kind, N, S_d, seed, state, ep_step, ep_return);
  return cudaGetLastError();
}

cudaError_t launch_actor(int env_kind, const ActorParams& p, cudaStream_t s) {
  if (env_kind == TJ_ENV_LINGAUSS) {
    constexpr int TE = 32, NT = 256;
    const bool ext = p.logits_in != nullptr;
    const size_t smem = actor_smem_floats(TE, p.D, ext ? 0 : p.Hp, ext ? 0 : p.Ap, true, 0) * sizeof(float);
    if (smem > kSmemMax) return cudaErrorInvalidConfiguration;
    return launch_with_smem(actor_lingauss_kernel<TE, NT>, (p.N + TE - 1) / TE, NT, smem, p, s);
  }
  // Tile: 16 envs x 128 threads while that still leaves SMs short of two blocks each, else 32 x 256.
  const bool small_tile = p.N < 148 * 2 * 32;
  const int TE = small_tile ? 16 : 32;
  // Staging: everything if it fits (preferring a size that lets two blocks share an SM), else all but W2.
  int stage = 0;
  size_t smem = 0;
  for (int st = 2; st >= 0; --st) {
    smem = actor_smem_floats(TE, p.D, p.Hp, p.Ap, false, staged_floats(st, p.w_total, p.off_W2t, p.off_b2)) * sizeof(float);
    if (smem <= (st == 0 ? kSmemMax : kSmemTwoPerSm) || (st == 2 && smem <= kSmemMax && p.H <= 160)) { stage = st; break; }
    if (st == 0) return cudaErrorInvalidConfiguration;
  }
  // Small N: 16 envs x 128 threads, 4 envs x 4 neurons per thread (more warps; the problem is latency-bound).
  // Large N: 32 envs per block, 8 envs per thread; wide layers (hidden >= 192) use 8 x 8 register tiles on 128
  // threads (64 FMAs per four operand loads), narrower ones 4 neurons per thread on 256 threads.
  const bool wide = p.H >= 192;
  if (env_kind == TJ_ENV_CARTPOLE) {
    if (small_tile) return launch_small<16, 128, 4, 4, TJ_ENV_CARTPOLE>(stage, smem, p, s);
    if (wide) return launch_small<32, 128, 8, 8, TJ_ENV_CARTPOLE>(stage, smem, p, s);
    return launch_small<32, 256, 8, 4, TJ_ENV_CARTPOLE>(stage, smem, p, s);
  }
  if (small_tile) return launch_small<16, 128, 4, 4, TJ_ENV_ACROBOT>(stage, smem, p, s);
  if (wide) return launch_small<32, 128, 8, 8, TJ_ENV_ACROBOT>(stage, smem, p, s);
  return launch_small<32, 256, 8, 4, TJ_ENV_ACROBOT>(stage, smem, p, s);
}

}  // namespace tj
