// FP32-accuracy tensor-core actor for the small environments (CartPole, Acrobot) with hidden widths of 64 .. 256: the
// hidden x hidden layer -- the one dense contraction of these networks (Algorithm 1, task 1: 65,536 of a 6-256-256-3
// network's 67,840 multiply-adds per env step) -- runs on the tensor cores as three FP16 products of split operands,
//   W2 h1 = W_hi h_hi + W_hi h_lo + W_lo h_hi,   x = x_hi + x_lo with x_hi the 11 leading bits of the (power-of-two scaled) value,
// with FP32 accumulation in tensor memory (error about 2^-22 per term, the dropped lo x lo term; FP16 runs at twice the rate
// of the 3 x TF32 form of the same idea).  Layer 1 (4 or 6 inputs) and the head (2-4 outputs) stay on the FP32 pipes.
//
// One thread block keeps a tile of 128 environments for all n_steps of the call (environments are independent): thread e
// owns env e's state in registers.  Eight worker warps, one MMA-issuing warp, one copy warp; per step:
//   observation -> shared memory;
//   workers: layer 1 in the fixed FMA order of the FP32 path, ReLU, split -> FP16 A operand, 32 hidden units (one K chunk of
//     the next layer) at a time, each chunk handed to the issuing lane through its own mbarrier;
//   copy lane: streams W2's parts in 32-column chunks (bulk copies, four ring slots, the stream running on across steps);
//   issuing lane: per K chunk, issues W_hi x (h_hi, h_lo) and W_lo x h_hi (M = 128, N = H) as soon as that chunk of h1 exists, so
//     the tensor pipe works underneath layer 1;
//   workers: accumulator -> + b2, ReLU, head partial sums by two threads per row -> outputs;
//   then exactly the FP32 kernel's selection, env step, record / segment write and reset.
// Every wait is bounded; a timeout latches the context's error word and the block leaves after freeing its tensor memory.
#include <cuda_fp16.h>

#include "tj_internal.h"
#include "tj_mlp.cuh"
#include "tj_tc.cuh"

namespace tj {

namespace {

constexpr int SA_TE = 128;            // envs per tile = rows of the MMA
constexpr int SA_WORKERS = 256;       // threads of the worker warps; one more warp issues
constexpr int SA_NT = SA_WORKERS + 64;   // + the MMA-issuing warp and the copy warp
constexpr int SA_KC = 32;             // K columns per streamed chunk of W2
constexpr int SA_SLOTS = 4;
constexpr int SA_MAX_KC = 256 / SA_KC;
constexpr float SA_H_SCALE = 16.0f;   // hidden activations are split after this scaling (|h1| < 4,094 stays inside FP16)

struct SaCtl {
  uint64_t full[SA_SLOTS], empty[SA_SLOTS];
  uint64_t a_ready[SA_MAX_KC];   // K chunk of the A operand written (one arrival per worker warp)
  uint64_t wbar;                 // small parameters staged
  uint64_t acc_full;             // all MMAs of a forward pass complete
  uint32_t tmem_base;
  int abort_flag;
  int range_flag;               // a scaled hidden activation left FP16's range: the outputs of that pass are meaningless
};

__device__ __forceinline__ float4 sa_reset4(uint2 seed, uint32_t e, unsigned long long step, float lo, float width) {
  const uint4 w = stream_words(seed, STREAM_RESET, 0, e, step);
  return make_float4(uniform_range(w.x, lo, width), uniform_range(w.y, lo, width), uniform_range(w.z, lo, width),
                     uniform_range(w.w, lo, width));
}

template <int ENV>
__device__ __forceinline__ void sa_observe(float4 s, float* obs) {
  if (ENV == TJ_ENV_CARTPOLE) {
    obs[0] = s.x; obs[1] = s.y; obs[2] = s.z; obs[3] = s.w; obs[4] = obs[5] = 0.f;
  } else {
    float s1, c1, s2, c2;
    sincosf(s.x, &s1, &c1);
    sincosf(s.y, &s2, &c2);
    obs[0] = c1; obs[1] = s1; obs[2] = c2; obs[3] = s2; obs[4] = s.z; obs[5] = s.w;
  }
}

struct SaShared {
  uint8_t *a_hi, *a_lo, *ring;
  float *xs, *out, *part;
  SaCtl* ctl;
};

// eight hidden units n0 .. n0+7 of layer 1 for one env, in the canonical order (bias, then inputs in index order), ReLU,
// scaling, split; one 16-byte row segment of each part of the A operand
template <int D>
__device__ __forceinline__ float sa_layer1_block(const MlpWeights& mw, int Hp, const float* x, int n0, uint8_t* a_hi, uint8_t* a_lo, size_t off) {
  float acc[8];
  const float4 b0 = *reinterpret_cast<const float4*>(mw.b1 + n0), b1 = *reinterpret_cast<const float4*>(mw.b1 + n0 + 4);
  acc[0] = b0.x; acc[1] = b0.y; acc[2] = b0.z; acc[3] = b0.w; acc[4] = b1.x; acc[5] = b1.y; acc[6] = b1.z; acc[7] = b1.w;
#pragma unroll
  for (int k = 0; k < D; ++k) {
    const float4 w0 = *reinterpret_cast<const float4*>(mw.W1t + (size_t)k * Hp + n0);
    const float4 w1 = *reinterpret_cast<const float4*>(mw.W1t + (size_t)k * Hp + n0 + 4);
    acc[0] = fmaf(w0.x, x[k], acc[0]); acc[1] = fmaf(w0.y, x[k], acc[1]); acc[2] = fmaf(w0.z, x[k], acc[2]); acc[3] = fmaf(w0.w, x[k], acc[3]);
    acc[4] = fmaf(w1.x, x[k], acc[4]); acc[5] = fmaf(w1.y, x[k], acc[5]); acc[6] = fmaf(w1.z, x[k], acc[6]); acc[7] = fmaf(w1.w, x[k], acc[7]);
  }
  uint32_t hi2[4], lo2[4];
  float vmax = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float v0 = fmaxf(acc[2 * i], 0.f) * SA_H_SCALE, v1 = fmaxf(acc[2 * i + 1], 0.f) * SA_H_SCALE;
    vmax = fmaxf(vmax, fmaxf(v0, v1));
    const float h0 = __uint_as_float(__float_as_uint(v0) & 0xFFFFE000u), h1 = __uint_as_float(__float_as_uint(v1) & 0xFFFFE000u);
    hi2[i] = pack_f16x2(h0, h1);
    lo2[i] = pack_f16x2(v0 - h0, v1 - h1);
  }
  *reinterpret_cast<uint4*>(a_hi + off) = make_uint4(hi2[0], hi2[1], hi2[2], hi2[3]);
  *reinterpret_cast<uint4*>(a_lo + off) = make_uint4(lo2[0], lo2[1], lo2[2], lo2[3]);
  return vmax;
}

// Network outputs of the observations in xs -> out[i][e], i < Aout.  Called by every thread of the block; `pass` counts the
// calls, `copied` is the copy lane's position in the chunk stream: pass q reads the split matrix parts[q & 1] (the actor
// passes the same matrix twice, the TD kernel the online and the target network's).  Returns false after a timeout.
template <int D, int H>
__device__ __forceinline__ bool sa_forward(int Hp, int Aout, const MlpWeights& mw, const SaShared& sh, const uint16_t* parts0,
                                           const uint16_t* parts1, float inv_scale, uint32_t tmem, uint32_t pass, uint32_t& copied,
                                           volatile int* abort_flag) {
  constexpr int NKC = H / SA_KC;                 // K chunks of the hidden x hidden layer
  constexpr uint32_t NSTREAM = 2 * NKC;          // chunks of W2 per pass: (high, low) per K chunk
  constexpr uint32_t CHUNK_BYTES = H * SA_KC * 2;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  SaCtl* ctl = sh.ctl;
  if (tid < SA_WORKERS) {
    const int e = tid & (SA_TE - 1), half = tid >> 7;
    float x[D];
#pragma unroll
    for (int k = 0; k < D; ++k) x[k] = sh.xs[k * SA_TE + e];
    tc_fence_before();                            // this thread's accumulator reads of the previous pass are complete
    float vmax = 0.f;
#pragma unroll 1
    for (int kc = 0; kc < NKC; ++kc) {
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        const int n0 = kc * SA_KC + half * 16 + b * 8;
        const size_t off = ((size_t)(e >> 3) * (H / 8) + (n0 >> 3)) * 128 + (e & 7) * 16;
        vmax = fmaxf(vmax, sa_layer1_block<D>(mw, Hp, x, n0, sh.a_hi, sh.a_lo, off));
      }
      fence_async_smem();
      mbar_arrive_warp(&ctl->a_ready[kc]);
    }
    // 65,504 is FP16's largest finite value (a NaN activation also lands here: the comparison is written to catch it)
    if (!(vmax <= 65504.f)) ctl->range_flag = 1;
  } else if (warp == SA_WORKERS / 32) {
    // The issuing lane's warp-mates wait at the warp barrier, not in a polling loop: lanes of one warp that poll while
    // another lane of it issues take turns with that lane, and every blocked poll then stalls the issue.
    if (lane == 0) {
      // The stream position at the start of a pass is pass x NSTREAM, a multiple of the slot count: chunk c of any pass sits
      // in slot c % SLOTS, and only the barrier parities depend on the pass.
      const uint32_t idesc = make_idesc_f16(H);
      const uint32_t ahi_lo = desc_lo(smem_addr(sh.a_hi), 128u), alo_lo = desc_lo(smem_addr(sh.a_lo), 128u);
      const uint32_t a_hiword = desc_hi((uint32_t)(H / 8) * 128u), b_hiword = desc_hi((uint32_t)(SA_KC / 8) * 128u);
      const uint32_t ring_lo = desc_lo(smem_addr(sh.ring), 128u);
      const uint32_t round0 = pass * (NSTREAM / SA_SLOTS);           // trips around the ring before this pass
      bool alive = true;
#pragma unroll
      for (int kc = 0; kc < NKC; ++kc) {
        if (!alive) break;
        if (!tc_wait(&ctl->a_ready[kc], pass & 1, abort_flag)) { alive = false; break; }
        tc_fence_after();
        const uint32_t a_off = (uint32_t)kc * (SA_KC / 8) * 8u;     // in 16-byte units: 8 per core matrix, 4 core matrices per chunk
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          const int c = 2 * kc + part, s = c % SA_SLOTS;
          if (!tc_wait(&ctl->full[s], (round0 + c / SA_SLOTS) & 1, abort_flag)) { alive = false; break; }
          tc_fence_after();
          const uint32_t b_lo = ring_lo + (uint32_t)s * (CHUNK_BYTES / 16);
#pragma unroll
          for (int j = 0; j < SA_KC / 16; ++j) {
            umma_ss(tmem, ahi_lo + a_off + 16u * j, a_hiword, b_lo + 16u * j, b_hiword, idesc, (c | j) != 0);
            if (part == 0) umma_ss(tmem, alo_lo + a_off + 16u * j, a_hiword, b_lo + 16u * j, b_hiword, idesc, 1u);
          }
          umma_commit(&ctl->empty[s]);
        }
      }
      umma_commit(&ctl->acc_full);
    }
    __syncwarp();
  } else {
    // copy lane: keeps the ring full -- chunk g of the stream follows chunk g - SLOTS into its slot once that one is consumed
    if (lane == 0) {
#pragma unroll 1
      for (uint32_t c = 0; c < NSTREAM; ++c, ++copied) {
        const uint32_t sp = copied % SA_SLOTS;
        if (!tc_wait(&ctl->empty[sp], ((copied / SA_SLOTS) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(&ctl->full[sp], CHUNK_BYTES);
        const uint16_t* src = ((copied / NSTREAM) & 1u) ? parts1 : parts0;
        bulk_copy_g2s(sh.ring + (size_t)sp * CHUNK_BYTES, reinterpret_cast<const uint8_t*>(src) + (size_t)(copied % NSTREAM) * CHUNK_BYTES,
                      CHUNK_BYTES, &ctl->full[sp]);
      }
    }
    __syncwarp();
  }
  // after a timeout the abort flag is up: the pass runs to its end on meaningless numbers (every thread keeps to the same
  // barriers) and the caller leaves
  tc_wait_elect(&ctl->acc_full, pass & 1, abort_flag);
  tc_fence_after();
  // drain: two threads per row (the two column halves); h2 = relu(acc / scale + b2), head partial sums in column order
  if (tid < SA_WORKERS) {
    const int q = warp & 3, half = warp >> 2, r = q * 32 + lane;
    float pa[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t t_row = tmem + ((uint32_t)(q * 32) << 16);
#pragma unroll 2
    for (int c0 = half * (H / 2); c0 < (half + 1) * (H / 2); c0 += 16) {
      uint32_t v[16];
      tmem_ld16(t_row + (uint32_t)c0, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float h2 = fmaxf(fmaf(__uint_as_float(v[i]), inv_scale, mw.b2[c0 + i]), 0.f);
        const float4 w = *reinterpret_cast<const float4*>(mw.W3t + (size_t)(c0 + i) * 4);   // a row of W3t (Ap = 4)
        pa[0] = fmaf(w.x, h2, pa[0]); pa[1] = fmaf(w.y, h2, pa[1]); pa[2] = fmaf(w.z, h2, pa[2]); pa[3] = fmaf(w.w, h2, pa[3]);
      }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
      if (a < Aout) sh.part[((size_t)half * 4 + a) * SA_TE + r] = pa[a];
  }
  __syncthreads();
  if (tid < SA_TE)
    for (int a = 0; a < Aout; ++a)
      sh.out[a * SA_TE + tid] = (mw.b3[a] + sh.part[(size_t)a * SA_TE + tid]) + sh.part[((size_t)4 + a) * SA_TE + tid];
  __syncthreads();
  return *abort_flag == 0;
}

template <int ENV, int H>
__global__ void __launch_bounds__(SA_NT, 1) actor_split_tc_kernel(const ActorParams p, const uint16_t* __restrict__ w2parts,
                                                                 const float* __restrict__ w2scale) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr int D = ENV == TJ_ENV_CARTPOLE ? 4 : 6;
  constexpr int A_BYTES = SA_TE * H * 2;                      // one FP16 part of the A operand
  constexpr uint32_t CHUNK_BYTES = H * SA_KC * 2;             // one chunk of one part of W2
  constexpr uint32_t NSTREAM = 2 * (H / SA_KC);
  SaShared sh;
  sh.a_hi = smem_raw;
  sh.a_lo = sh.a_hi + A_BYTES;
  sh.ring = sh.a_lo + A_BYTES;
  float* wsm = reinterpret_cast<float*>(sh.ring + SA_SLOTS * CHUNK_BYTES);
  const size_t staged = p.w_total - (p.off_b2 - p.off_W2t);   // everything but the H x H matrix
  sh.xs = wsm + staged;                                       // [8][TE]
  sh.out = sh.xs + (size_t)8 * SA_TE;                         // [4][TE]
  sh.part = sh.out + (size_t)4 * SA_TE;                       // [2][4][TE]
  sh.ctl = reinterpret_cast<SaCtl*>(sh.part + 2 * (size_t)4 * SA_TE);
  SaCtl* ctl = sh.ctl;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int n_tiles = (p.N + SA_TE - 1) / SA_TE;
  const bool on_policy = p.C == 0;

  if (tid == 0) {
    for (int s = 0; s < SA_SLOTS; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    for (int k = 0; k < SA_MAX_KC; ++k) mbar_init(&ctl->a_ready[k], SA_WORKERS / 32);
    mbar_init(&ctl->wbar, 1);
    mbar_init(&ctl->acc_full, 1);
    ctl->abort_flag = 0;
    ctl->range_flag = 0;
  }
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&ctl->tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const MlpWeights mw = stage_mlp_weights<1>(p, p.W, wsm, &ctl->wbar, tid == 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;
  bool ok = tc_wait_elect(&ctl->wbar, 0, abort_flag);
  ok = __syncthreads_and(ok);
  const float inv_scale = w2scale[1];                         // 1 / (activation scale x weight scale)

  uint32_t copied = 0, pass = 0;                               // chunk stream position (copy lane), forward passes
  if (tid == SA_WORKERS + 32 && ok) {
    for (; copied < SA_SLOTS; ++copied) {
      mbar_expect_tx(&ctl->full[copied], CHUNK_BYTES);
      bulk_copy_g2s(sh.ring + (size_t)copied * CHUNK_BYTES, reinterpret_cast<const uint8_t*>(w2parts) + (size_t)(copied % NSTREAM) * CHUNK_BYTES,
                    CHUNK_BYTES, &ctl->full[copied]);
    }
  }

  unsigned long long n_episodes = 0;
  double ret_sum = 0.0;
  for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
    const int e = tile * SA_TE + tid;
    const bool owner = tid < SA_TE && e < p.N;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    int ep = 0;
    float ep_ret = 0.f;
    if (owner) {
      s = reinterpret_cast<const float4*>(p.state)[e];
      ep = p.ep_step[e];
      ep_ret = p.ep_return[e];
    }
    for (int step = 0; step < p.n_steps && ok; ++step) {
      const unsigned long long t = (unsigned long long)p.t0 + step;
      float obs[6];
      sa_observe<ENV>(s, obs);
      if (tid < SA_TE) {
#pragma unroll
        for (int k = 0; k < D; ++k) sh.xs[k * SA_TE + tid] = owner ? obs[k] : 0.f;
      }
      __syncthreads();
      ok = sa_forward<D, H>(p.Hp, p.Aout, mw, sh, w2parts, w2parts, inv_scale, tmem, pass++, copied, abort_flag);
      ok = __syncthreads_and(ok);
      if (!ok) break;
      if (owner) {
        auto logit = [&](int i) { return sh.out[i * SA_TE + tid]; };
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
          float* so = p.seg_obs + i * D;
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
          s = (ENV == TJ_ENV_CARTPOLE) ? sa_reset4(p.seed, (uint32_t)e, t, -0.05f, 0.1f) : sa_reset4(p.seed, (uint32_t)e, t, -0.1f, 0.2f);
        } else {
          s = sn;
        }
      }
      if (!on_policy && tile == 0 && tid == 0)
        p.block_ver[((p.cursor0 + (unsigned long long)step * p.N) % (unsigned long long)p.C) / p.N] = p.version;
      // last step of a segment: bootstrap value of the state each env is now in
      if (on_policy && (int)(t % (unsigned long long)p.T) == p.T - 1) {
        float o2[6];
        sa_observe<ENV>(s, o2);
        __syncthreads();
        if (tid < SA_TE) {
#pragma unroll
          for (int k = 0; k < D; ++k) sh.xs[k * SA_TE + tid] = owner ? o2[k] : 0.f;
        }
        __syncthreads();
        ok = sa_forward<D, H>(p.Hp, p.Aout, mw, sh, w2parts, w2parts, inv_scale, tmem, pass++, copied, abort_flag);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        if (owner) {
          const int slot = (int)((long long)(t / (unsigned long long)p.T) % p.G);
          p.seg_val[((size_t)slot * (p.T + 1) + p.T) * p.N + e] = sh.out[p.A * SA_TE + tid];
        }
      }
      __syncthreads();
    }
    if (owner) {
      reinterpret_cast<float4*>(p.state)[e] = s;
      p.ep_step[e] = ep;
      p.ep_return[e] = ep_ret;
    }
  }
  if (tid < SA_TE && n_episodes) {
    atomicAdd(&p.stats->episodes, n_episodes);
    atomicAdd(&p.stats->return_sum, ret_sum);
  }
  // the copies still in flight must land before the block gives its shared memory back
  if (tid == SA_WORKERS + 32) {
    for (uint32_t g = pass * NSTREAM; g < copied; ++g)
      if (!tc_wait(&ctl->full[g % SA_SLOTS], (g / SA_SLOTS) & 1, abort_flag)) break;
    if (ctl->abort_flag) atomicExch(&p.stats->error, 4ull);
    else if (ctl->range_flag) atomicExch(&p.stats->error, 5ull);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

// TD error (Algorithm 1, TD-error line; Huber loss on it) for a context in this weight mode: a tile of 128 sampled rows per
// block, the online network on obs (pass 0), the target network on next_obs (pass 1), both with the split-operand hidden
// layer above; the small parameters are staged twice, the chunk stream alternates between the two split matrices.
// Outputs and the per-block loss partial as in the FP32 TD kernel (one partial per 128 rows, summed in row order).
template <int D, int H>
__global__ void __launch_bounds__(SA_NT, 1) td_split_tc_kernel(const TdParams p, const uint16_t* __restrict__ parts_online,
                                                              const float* __restrict__ scale_online,
                                                              const uint16_t* __restrict__ parts_target,
                                                              const float* __restrict__ scale_target) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr int A_BYTES = SA_TE * H * 2;
  constexpr uint32_t CHUNK_BYTES = H * SA_KC * 2;
  constexpr uint32_t NSTREAM = 2 * (H / SA_KC);
  SaShared sh;
  sh.a_hi = smem_raw;
  sh.a_lo = sh.a_hi + A_BYTES;
  sh.ring = sh.a_lo + A_BYTES;
  float* wsm = reinterpret_cast<float*>(sh.ring + SA_SLOTS * CHUNK_BYTES);
  const size_t staged = p.w_total - (p.off_b2 - p.off_W2t);
  sh.xs = wsm + staged;
  sh.out = sh.xs + (size_t)8 * SA_TE;
  sh.part = sh.out + (size_t)4 * SA_TE;
  sh.ctl = reinterpret_cast<SaCtl*>(sh.part + 2 * (size_t)4 * SA_TE);
  SaCtl* ctl = sh.ctl;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int j0 = blockIdx.x * SA_TE, n_here = min(SA_TE, p.n - j0);
  if (tid == 0) {
    for (int s = 0; s < SA_SLOTS; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    for (int k = 0; k < SA_MAX_KC; ++k) mbar_init(&ctl->a_ready[k], SA_WORKERS / 32);
    mbar_init(&ctl->wbar, 1);
    mbar_init(&ctl->acc_full, 1);
    ctl->abort_flag = 0;
    ctl->range_flag = 0;
  }
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&ctl->tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  MlpWeights mw = stage_mlp_weights<1>(p, p.Wonline, wsm, &ctl->wbar, tid == 0);
  for (int i = tid; i < SA_TE * D; i += SA_NT) {
    const int el = i / D, k = i % D;
    sh.xs[k * SA_TE + el] = el < n_here ? p.obs[(size_t)(j0 + el) * D + k] : 0.f;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;
  bool ok = tc_wait_elect(&ctl->wbar, 0, abort_flag);
  ok = __syncthreads_and(ok);
  uint32_t copied = 0;
  if (tid == SA_WORKERS + 32 && ok) {
    for (; copied < SA_SLOTS; ++copied) {
      mbar_expect_tx(&ctl->full[copied], CHUNK_BYTES);
      bulk_copy_g2s(sh.ring + (size_t)copied * CHUNK_BYTES, reinterpret_cast<const uint8_t*>(parts_online) + (size_t)copied * CHUNK_BYTES,
                    CHUNK_BYTES, &ctl->full[copied]);
    }
  }
  uint32_t passes = 0;
  float qsel = 0.f;
  if (ok) {
    ok = sa_forward<D, H>(p.Hp, p.A, mw, sh, parts_online, parts_target, scale_online[1], tmem, 0u, copied, abort_flag);
    passes = 1;
    ok = __syncthreads_and(ok);
  }
  if (ok) {
    if (tid < n_here) {
      int a = p.act[j0 + tid];
      a = a < 0 ? 0 : (a >= p.A ? p.A - 1 : a);
      qsel = sh.out[a * SA_TE + tid];
    }
    __syncthreads();   // every thread is done with the online parameters and outputs: the staging buffer may be refilled
    mw = stage_mlp_weights<1>(p, p.Wtarget, wsm, &ctl->wbar, tid == 0);
    for (int i = tid; i < SA_TE * D; i += SA_NT) {
      const int el = i / D, k = i % D;
      sh.xs[k * SA_TE + el] = el < n_here ? p.next_obs[(size_t)(j0 + el) * D + k] : 0.f;
    }
    ok = tc_wait_elect(&ctl->wbar, 1, abort_flag);
    ok = __syncthreads_and(ok);
  }
  if (ok) {
    ok = sa_forward<D, H>(p.Hp, p.A, mw, sh, parts_online, parts_target, scale_target[1], tmem, 1u, copied, abort_flag);
    passes = 2;
    ok = __syncthreads_and(ok);
  }
  const float nan = __int_as_float(0x7FC00000);
  float* hub = sh.part;                       // free again after the pass
  if (tid < SA_TE) {
    float h = 0.f;
    if (tid < n_here) {
      const int j = j0 + tid;
      float delta = nan;
      h = nan;
      if (ok) {
        float qmax = sh.out[tid];
        for (int i = 1; i < p.A; ++i) qmax = fmaxf(qmax, sh.out[i * SA_TE + tid]);
        const float y = p.rew[j] + p.gamma * (p.done[j] ? 0.f : 1.f) * qmax;
        delta = y - qsel;
        const float ad = fabsf(delta);
        h = ad <= p.kappa ? 0.5f * delta * delta : p.kappa * (ad - 0.5f * p.kappa);
      }
      if (p.td_out) p.td_out[j] = delta;        // after a timeout: defined outputs (NaN), never what an earlier call left
      if (p.huber_out) p.huber_out[j] = h;
    }
    hub[tid] = h;
  }
  __syncthreads();
  if (tid == 0) {
    float sum = 0.f;
    for (int i = 0; i < n_here; ++i) sum += hub[i];
    p.partial[blockIdx.x] = sum;
    if (ctl->abort_flag && p.error) atomicExch(p.error, 4ull);
    else if (ctl->range_flag && p.error) atomicExch(p.error, 5ull);
  }
  // the copies still in flight must land before the block gives its shared memory back
  if (tid == SA_WORKERS + 32) {
    for (uint32_t g = passes * NSTREAM; g < copied; ++g)
      if (!tc_wait(&ctl->full[g % SA_SLOTS], (g / SA_SLOTS) & 1, abort_flag)) break;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

// W2 [H][H] (row = neuron) -> scaled FP16 high and low parts as the stream the kernel consumes: for each K chunk kc of 32
// columns first the high parts' chunk, then the low parts', each H rows x 32 columns in the K-major core-matrix layout:
// element (n, k) sits at ((n / 8) * 4 + (k % 32) / 8) * 64 + (n % 8) * 8 + k % 8 inside its chunk.
// scale_out[0] = the power of two the weights were multiplied by, scale_out[1] = 1 / (that x the activation scale).
// One launch of a few large blocks: every block finds the largest |entry| of the matrix itself (64 K floats from L2 at most,
// 64 per thread), so no block waits for another; block 0 records the scale; then each block packs its share.
constexpr int SPLIT_PACK_BLOCKS = 32, SPLIT_PACK_THREADS = 1024;
__global__ void __launch_bounds__(SPLIT_PACK_THREADS) split_pack_kernel(const float* __restrict__ blob, int D, int H, float* __restrict__ scale_out,
                                                                        uint16_t* __restrict__ dst) {
  __shared__ float wmax[32];
  const float* W2 = blob + (size_t)H * D + H;
  float m = 0.f;
  for (int i = threadIdx.x; i < H * H; i += blockDim.x) m = fmaxf(m, fabsf(W2[i]));   // the caller's pointer may be only 4-byte aligned
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, wmax[w]);
  // largest entry into [1024, 2048): far inside FP16's range, low parts of all but the tiniest entries normal
  int e = 0;
  if (m > 0.f && isfinite(m)) e = 10 - (int)floorf(log2f(m));
  e = e < -24 ? -24 : (e > 24 ? 24 : e);
  const float sc = exp2f((float)e);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    scale_out[0] = sc;
    scale_out[1] = 1.0f / (sc * SA_H_SCALE);
  }
  const int chunk_elems = H * SA_KC;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < H * H; i += gridDim.x * blockDim.x) {
    const int kc = i / chunk_elems, within = i % chunk_elems;
    const int core = within / 64, in_core = within % 64;
    const int rg = core / (SA_KC / 8), kg = core % (SA_KC / 8);
    const int n = rg * 8 + in_core / 8, k = kc * SA_KC + kg * 8 + in_core % 8;
    const float v = W2[(size_t)n * H + k] * sc;
    const __half hi = __float2half_rn(v);
    const __half lo = __float2half_rn(v - __half2float(hi));
    dst[(size_t)(2 * kc) * chunk_elems + within] = __half_as_ushort(hi);
    dst[(size_t)(2 * kc + 1) * chunk_elems + within] = __half_as_ushort(lo);
  }
}

template <int ENV, int H>
cudaError_t launch_split(const ActorParams& p, const uint16_t* w2parts, const float* w2scale, int grid, size_t smem, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(actor_split_tc_kernel<ENV, H>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  actor_split_tc_kernel<ENV, H><<<grid, SA_NT, smem, s>>>(p, w2parts, w2scale);
  return cudaGetLastError();
}

template <int ENV>
cudaError_t launch_split_env(const ActorParams& p, const uint16_t* w2parts, const float* w2scale, int grid, size_t smem, cudaStream_t s) {
  switch (p.H) {
    case 64: return launch_split<ENV, 64>(p, w2parts, w2scale, grid, smem, s);
    case 128: return launch_split<ENV, 128>(p, w2parts, w2scale, grid, smem, s);
    case 192: return launch_split<ENV, 192>(p, w2parts, w2scale, grid, smem, s);
    case 256: return launch_split<ENV, 256>(p, w2parts, w2scale, grid, smem, s);
    default: return cudaErrorInvalidConfiguration;
  }
}

}  // namespace

bool split_actor_supported(int env_kind, int D, int H, int Aout) {
  const bool env_ok = (env_kind == TJ_ENV_CARTPOLE && D == 4) || (env_kind == TJ_ENV_ACROBOT && D == 6);
  return env_ok && H >= 64 && H <= 256 && H % 64 == 0 && Aout <= 4;   // Aout <= 4: rows of the head matrix are one float4
}

size_t split_weight_halfs(int H) { return (size_t)2 * H * H; }

cudaError_t launch_pack_split_weights(const float* blob, int D, int H, uint16_t* dst, float* scale, cudaStream_t s) {
  split_pack_kernel<<<SPLIT_PACK_BLOCKS, SPLIT_PACK_THREADS, 0, s>>>(blob, D, H, scale, dst);
  return cudaGetLastError();
}

cudaError_t launch_actor_split(int env_kind, const ActorParams& p, const uint16_t* w2parts, const float* w2scale, int sm_count,
                               cudaStream_t s) {
  if (p.N <= 0) return cudaSuccess;
  if (!split_actor_supported(env_kind, p.D, p.H, p.Aout)) return cudaErrorInvalidConfiguration;
  const size_t staged = p.w_total - (p.off_b2 - p.off_W2t);
  const size_t smem = (size_t)2 * SA_TE * p.H * 2 + (size_t)SA_SLOTS * p.H * SA_KC * 2 +
                      (staged + (size_t)(8 + 4 + 8) * SA_TE) * sizeof(float) + sizeof(SaCtl) + 64;
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  const int n_tiles = (p.N + SA_TE - 1) / SA_TE;
  const int grid = n_tiles < sm_count ? n_tiles : sm_count;
  return env_kind == TJ_ENV_CARTPOLE ? launch_split_env<TJ_ENV_CARTPOLE>(p, w2parts, w2scale, grid, smem, s)
                                     : launch_split_env<TJ_ENV_ACROBOT>(p, w2parts, w2scale, grid, smem, s);
}

template <int D>
static cudaError_t launch_td_split_d(const TdParams& p, const uint16_t* po, const float* so, const uint16_t* pt, const float* st, int grid,
                                     size_t smem, cudaStream_t s) {
#define TJ_TD_SPLIT_CASE(HH)                                                                                                      \
  case HH: {                                                                                                                      \
    cudaError_t e = cudaFuncSetAttribute(td_split_tc_kernel<D, HH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);      \
    if (e != cudaSuccess) return e;                                                                                               \
    td_split_tc_kernel<D, HH><<<grid, SA_NT, smem, s>>>(p, po, so, pt, st);                                                        \
    return cudaGetLastError();                                                                                                    \
  }
  switch (p.H) {
    TJ_TD_SPLIT_CASE(64)
    TJ_TD_SPLIT_CASE(128)
    TJ_TD_SPLIT_CASE(192)
    TJ_TD_SPLIT_CASE(256)
    default: return cudaErrorInvalidConfiguration;
  }
#undef TJ_TD_SPLIT_CASE
}

int td_split_grid(int n) { return (n + SA_TE - 1) / SA_TE; }

cudaError_t launch_td_split(const TdParams& p, const uint16_t* parts_online, const float* scale_online, const uint16_t* parts_target,
                            const float* scale_target, cudaStream_t s) {
  if (p.n <= 0) return cudaSuccess;
  if (!(p.D == 4 || p.D == 6) || p.A > 4 || p.Ap != 4) return cudaErrorInvalidConfiguration;
  const size_t staged = p.w_total - (p.off_b2 - p.off_W2t);
  const size_t smem = (size_t)2 * SA_TE * p.H * 2 + (size_t)SA_SLOTS * p.H * SA_KC * 2 +
                      (staged + (size_t)(8 + 4 + 8) * SA_TE) * sizeof(float) + sizeof(SaCtl) + 64;
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  const int grid = td_split_grid(p.n);
  return p.D == 4 ? launch_td_split_d<4>(p, parts_online, scale_online, parts_target, scale_target, grid, smem, s)
                  : launch_td_split_d<6>(p, parts_online, scale_online, parts_target, scale_target, grid, smem, s);
}

}  // namespace tj
