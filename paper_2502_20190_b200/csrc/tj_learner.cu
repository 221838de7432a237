// Learner-side kernels: parameter publish (repack), eligible-block list, staleness-bounded sampling with
// gather, TD error / Huber loss, and the GAE reverse scan.
#include <mutex>

#include "tj_async.cuh"
#include "tj_device.cuh"
#include "tj_internal.h"
#include "tj_mlp.cuh"

namespace tj {

namespace {

__device__ __forceinline__ float bf16_round_rne(float x) {
  uint32_t u = __float_as_uint(x);
  if ((u & 0x7F800000u) == 0x7F800000u) return x;
  u += 0x7FFFu + ((u >> 16) & 1u);
  return __uint_as_float(u & 0xFFFF0000u);
}

// blob [W1 HxD, b1 H, W2 HxH, b2 H, W3 AxH, b3 A (, Wv H, bv 1)] -> transposed, padded kernel layout
__global__ void pack_weights_kernel(const float* __restrict__ blob, float* __restrict__ dst, WeightLayout L,
                                    int value_head, int bf16) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= L.total) return;
  const int D = L.D, H = L.H, A = L.A;
  const float* W1 = blob;
  const float* b1 = W1 + (size_t)H * D;
  const float* W2 = b1 + H;
  const float* b2 = W2 + (size_t)H * H;
  const float* W3 = b2 + H;
  const float* b3 = W3 + (size_t)A * H;
  const float* Wv = b3 + A;
  const float* bv = Wv + H;
  float v = 0.f;
  bool is_weight = false;
  if (i >= L.off_W1t && i < L.off_W1t + (size_t)D * L.Hp) {
    const size_t j = i - L.off_W1t;
    const int k = (int)(j / L.Hp), n = (int)(j % L.Hp);
    if (n < H) { v = W1[(size_t)n * D + k]; is_weight = true; }
  } else if (i >= L.off_b1 && i < L.off_b1 + L.Hp) {
    const int n = (int)(i - L.off_b1);
    if (n < H) v = b1[n];
  } else if (i >= L.off_W2t && i < L.off_W2t + (size_t)H * L.Hp) {
    const size_t j = i - L.off_W2t;
    const int k = (int)(j / L.Hp), n = (int)(j % L.Hp);
    if (n < H) { v = W2[(size_t)n * H + k]; is_weight = true; }
  } else if (i >= L.off_b2 && i < L.off_b2 + L.Hp) {
    const int n = (int)(i - L.off_b2);
    if (n < H) v = b2[n];
  } else if (i >= L.off_W3t && i < L.off_W3t + (size_t)H * L.Ap) {
    const size_t j = i - L.off_W3t;
    const int k = (int)(j / L.Ap), n = (int)(j % L.Ap);
    if (n < A) { v = W3[(size_t)n * H + k]; is_weight = true; }
    else if (value_head && n == A) { v = Wv[k]; is_weight = true; }
  } else if (i >= L.off_b3 && i < L.off_b3 + L.Ap) {
    const int n = (int)(i - L.off_b3);
    if (n < A) v = b3[n];
    else if (value_head && n == A) v = bv[0];
  }
  if (bf16 && is_weight) v = bf16_round_rne(v);
  dst[i] = v;
}

__global__ void transpose_pad_kernel(const float* __restrict__ src, float* __restrict__ dst, int rows, int cols,
                                     int ld_dst) {
  // dst[c][r] = src[r][c], dst rows padded to ld_dst with zeros
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)cols * ld_dst) return;
  const int c = (int)(i / ld_dst), r = (int)(i % ld_dst);
  dst[i] = r < rows ? src[(size_t)r * cols + c] : 0.f;
}

// Ascending list of ring blocks (one block = the N records of one actor step, all with one version) whose
// version is at most `bound` behind the learner.  One thread block, stable compaction by chunks.
__global__ void eligible_kernel(const int* __restrict__ block_ver, int n_blocks, long long v_learner, long long bound,
                                int* __restrict__ elig_list, int* __restrict__ elig_count) {
  __shared__ int warp_tot[32];
  __shared__ int base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) base = 0;
  __syncthreads();
  for (int c0 = 0; c0 < n_blocks; c0 += blockDim.x) {
    const int b = c0 + tid;
    const int flag = (b < n_blocks && v_learner - (long long)block_ver[b] <= bound) ? 1 : 0;
    const unsigned m = __ballot_sync(0xffffffffu, flag);
    const int before = __popc(m & ((1u << lane) - 1u));
    if (lane == 0) warp_tot[warp] = __popc(m);
    __syncthreads();
    int woff = 0, tot = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
      if (w < warp) woff += warp_tot[w];
      tot += warp_tot[w];
    }
    if (flag) elig_list[base + woff + before] = b;
    __syncthreads();
    if (tid == 0) base += tot;
    __syncthreads();
  }
  if (tid == 0) *elig_count = base;
}

// One warp per draw: slot = E[mulhi(x0, |E|)] with E enumerated block by block, then the record is copied
// word for word into the dense minibatch arrays.
__global__ void sample_gather_kernel(const SampleParams p) {
  const int warp = (int)(((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  if (warp >= p.B) return;
  const int j = warp;
  const unsigned long long nE = (unsigned long long)(*p.elig_count) * (unsigned long long)p.N;
  const uint4 w = stream_words(p.seed, STREAM_SAMPLE, 0, (uint32_t)j, (unsigned long long)p.k);
  const uint32_t r = __umulhi(w.x, (uint32_t)nE);
  const int slot = p.elig_list[r / (uint32_t)p.N] * p.N + (int)(r % (uint32_t)p.N);
  const float* rec = p.ring + (size_t)slot * p.rec_words;
  const int D = p.D;
  for (int i = lane; i < p.rec_words; i += 32) {
    const float v = rec[i];
    if (i < D) p.obs[(size_t)j * D + i] = v;
    else if (i < 2 * D) p.next_obs[(size_t)j * D + (i - D)] = v;
    else if (i == 2 * D) p.act[j] = __float_as_int(v);
    else if (i == 2 * D + 1) p.rew[j] = v;
    else if (i == 2 * D + 2) p.done[j] = __float_as_int(v);
    else {
      const int ver = __float_as_int(v);
      p.ver[j] = ver;
      long long stale = p.v_learner - (long long)ver;
      if (stale < 0) stale = 0;
      atomicAdd(&p.stats->hist[stale > 32 ? 32 : stale], 1ull);
      atomicMax(&p.stats->max_stale, (unsigned long long)stale);
    }
  }
  if (lane == 0 && p.idx_out) p.idx_out[j] = slot;
}

// The same gather with 128-bit accesses (obs_dim a multiple of 4, 16-byte aligned outputs): LPD lanes share one
// draw and copy the record's 16-byte chunks -- obs, next_obs, then the (act, rew, done, ver) tail.
template <int LPD>
__global__ void sample_gather_vec_kernel(const SampleParams p) {
  const int lane = threadIdx.x & 31, sub = lane % LPD;
  const int j = (int)((((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * (32 / LPD)) + lane / LPD;
  if (j >= p.B) return;
  const unsigned long long nE = (unsigned long long)(*p.elig_count) * (unsigned long long)p.N;
  const uint4 w = stream_words(p.seed, STREAM_SAMPLE, 0, (uint32_t)j, (unsigned long long)p.k);
  const uint32_t r = __umulhi(w.x, (uint32_t)nE);
  const int slot = p.elig_list[r / (uint32_t)p.N] * p.N + (int)(r % (uint32_t)p.N);
  const float4* rec = reinterpret_cast<const float4*>(p.ring + (size_t)slot * p.rec_words);
  const int dq = p.D / 4;                         // chunks per observation
  float4* obs = reinterpret_cast<float4*>(p.obs + (size_t)j * p.D);
  float4* nxt = reinterpret_cast<float4*>(p.next_obs + (size_t)j * p.D);
  for (int c = sub; c <= 2 * dq; c += LPD) {
    const float4 v = __ldcs(rec + c);             // sampled rows are not reused: streaming load
    if (c < dq) obs[c] = v;
    else if (c < 2 * dq) nxt[c - dq] = v;
    else {
      const int ver = __float_as_int(v.w);
      p.act[j] = __float_as_int(v.x);
      p.rew[j] = v.y;
      p.done[j] = __float_as_int(v.z);
      p.ver[j] = ver;
      long long stale = p.v_learner - (long long)ver;
      if (stale < 0) stale = 0;
      atomicAdd(&p.stats->hist[stale > 32 ? 32 : stale], 1ull);
      atomicMax(&p.stats->max_stale, (unsigned long long)stale);
    }
  }
  if (sub == 0 && p.idx_out) p.idx_out[j] = slot;
}

// TD error on a tile of TE samples: online forward on obs, target forward on next_obs.
// STAGE as in the actor kernel (stage_mlp_weights); the staging buffer is filled twice (online, then target parameters).
// A staging wait that ran out: latch the context's error word and leave defined outputs (NaN) for this block's rows and
// its partial sum, so that neither the caller nor the loss reduction reads what an earlier call left there.
__device__ __forceinline__ void td_give_up(const TdParams& p, int n_here, int j0) {
  const float nan = __int_as_float(0x7FC00000);
  if (threadIdx.x == 0) {
    if (p.error) atomicExch(p.error, 3ull);
    p.partial[blockIdx.x] = nan;
  }
  if ((int)threadIdx.x < n_here) {
    if (p.td_out) p.td_out[j0 + threadIdx.x] = nan;
    if (p.huber_out) p.huber_out[j0 + threadIdx.x] = nan;
  }
}

template <int TE, int NT, int EPT, int NPT, int STAGE>
__global__ void __launch_bounds__(NT) td_kernel(const TdParams p) {
  extern __shared__ __align__(128) float smem[];
  __shared__ __align__(8) uint64_t wbar;
  const size_t staged = STAGE == 2 ? p.w_total : (STAGE == 1 ? p.w_total - (p.off_b2 - p.off_W2t) : 0);
  const int Dx = (p.D + 3) & ~3;
  float* wsm = smem;
  float* xs = wsm + staged;
  float* h1 = xs + (size_t)Dx * TE;
  float* h2 = h1 + (size_t)p.Hp * TE;
  float* out = h2 + (size_t)p.Hp * TE;
  float* qsel = out + (size_t)p.Ap * TE;
  float* hub = qsel + TE;
  const int tid = threadIdx.x, j0 = blockIdx.x * TE, n_here = min(TE, p.n - j0), D = p.D;
  if (STAGE > 0) {
    if (tid == 0) mbar_init(&wbar, 1);
    __syncthreads();
  }
  MlpWeights mw = stage_mlp_weights<STAGE>(p, p.Wonline, wsm, &wbar, tid == 0);

  for (int i = tid; i < TE * D; i += NT) {
    const int el = i / D, k = i % D;
    xs[k * TE + el] = el < n_here ? p.obs[(size_t)(j0 + el) * D + k] : 0.f;
  }
  if (STAGE > 0 && !mbar_wait_bounded(&wbar, 0)) { td_give_up(p, n_here, j0); return; }
  __syncthreads();
  mlp_forward_tile<TE, NT, EPT, (STAGE > 0), (STAGE == 2), NPT>(mw, D, p.H, p.Hp, p.A, p.Ap, xs, h1, h2, out);
  if (tid < n_here) {
    int a = p.act[j0 + tid];
    a = a < 0 ? 0 : (a >= p.A ? p.A - 1 : a);
    qsel[tid] = out[a * TE + tid];
  }
  __syncthreads();  // every thread is done with the online parameters: the buffer may be refilled
  mw = stage_mlp_weights<STAGE>(p, p.Wtarget, wsm, &wbar, tid == 0);
  for (int i = tid; i < TE * D; i += NT) {
    const int el = i / D, k = i % D;
    xs[k * TE + el] = el < n_here ? p.next_obs[(size_t)(j0 + el) * D + k] : 0.f;
  }
  if (STAGE > 0 && !mbar_wait_bounded(&wbar, 1)) { td_give_up(p, n_here, j0); return; }
  __syncthreads();
  mlp_forward_tile<TE, NT, EPT, (STAGE > 0), (STAGE == 2), NPT>(mw, D, p.H, p.Hp, p.A, p.Ap, xs, h1, h2, out);
  if (tid < TE) {
    float h = 0.f;
    if (tid < n_here) {
      const int j = j0 + tid;
      float qmax = out[tid];
      for (int i = 1; i < p.A; ++i) qmax = fmaxf(qmax, out[i * TE + tid]);
      const float y = p.rew[j] + p.gamma * (p.done[j] ? 0.f : 1.f) * qmax;
      const float delta = y - qsel[tid];
      const float ad = fabsf(delta);
      h = ad <= p.kappa ? 0.5f * delta * delta : p.kappa * (ad - 0.5f * p.kappa);
      if (p.td_out) p.td_out[j] = delta;
      if (p.huber_out) p.huber_out[j] = h;
    }
    hub[tid] = h;
  }
  __syncthreads();
  if (tid == 0) {
    float sum = 0.f;
    for (int i = 0; i < n_here; ++i) sum += hub[i];
    p.partial[blockIdx.x] = sum;
  }
}

// fixed-order sum of the per-block partial losses: one warp fetches 16 x 32 partials with independent coalesced loads
// (a single thread walking the array pays one memory latency per element, a warp fetching one chunk per iteration one per
// chunk), then lane 0 adds them in index order -- the same sum, term by term
__global__ void td_finish_kernel(const float* __restrict__ partial, int n_partial, int n, float* __restrict__ loss_out) {
  if (blockIdx.x != 0 || threadIdx.x >= 32) return;
  const int lane = threadIdx.x;
  float sum = 0.f;
  for (int base = 0; base < n_partial; base += 16 * 32) {
    float mine[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const int i = base + c * 32 + lane;
      mine[c] = i < n_partial ? partial[i] : 0.f;
    }
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const int left = n_partial - (base + c * 32);
      const int cnt = left < 0 ? 0 : (left < 32 ? left : 32);
      for (int l = 0; l < cnt; ++l) sum += __shfl_sync(0xffffffffu, mine[c], l);
    }
  }
  if (lane == 0) *loss_out = sum / (float)n;
}

// GAE: one thread per environment walks its column backwards; a warp reads 32 consecutive environments, so
// every access is a full 128-byte line.  The recurrence is serial in t, but its inputs are not: each thread
// fetches the next GAE_U time steps' rewards, values and done flags before it needs them, which keeps enough
// loads in flight to stream at HBM speed.
constexpr int GAE_U = 8;
__global__ void __launch_bounds__(128) gae_kernel(const float* __restrict__ rew, const float* __restrict__ val,
                                                  const uint8_t* __restrict__ done, int T, int N, float gamma,
                                                  float lambda, float* __restrict__ adv, float* __restrict__ ret) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= N) return;
  float next_adv = 0.f;
  float v_next = __ldcs(val + (size_t)T * N + e);
  const float gl = gamma * lambda;
  int t = T - 1;
  for (; t >= GAE_U - 1; t -= GAE_U) {
    float r[GAE_U], v[GAE_U];
    uint8_t d[GAE_U];
#pragma unroll
    for (int u = 0; u < GAE_U; ++u) {
      const size_t i = (size_t)(t - u) * N + e;
      r[u] = __ldcs(rew + i);
      v[u] = __ldcs(val + i);
      d[u] = __ldcs(done + i);
    }
#pragma unroll
    for (int u = 0; u < GAE_U; ++u) {
      const size_t i = (size_t)(t - u) * N + e;
      const float nd = d[u] ? 0.f : 1.f;
      const float delta = r[u] + gamma * nd * v_next - v[u];
      const float a = delta + gl * nd * next_adv;
      __stcs(adv + i, a);
      __stcs(ret + i, a + v[u]);
      next_adv = a;
      v_next = v[u];
    }
  }
  for (; t >= 0; --t) {
    const size_t i = (size_t)t * N + e;
    const float nd = done[i] ? 0.f : 1.f;
    const float v = val[i];
    const float delta = rew[i] + gamma * nd * v_next - v;
    const float a = delta + gl * nd * next_adv;
    adv[i] = a;
    ret[i] = a + v;
    next_adv = a;
    v_next = v;
  }
}

constexpr int kTdTile = 16;
constexpr int kTdThreads = 128;

}  // namespace

cudaError_t launch_pack_weights(const float* blob, float* dst, const WeightLayout& L, int value_head, int bf16,
                                cudaStream_t s) {
  pack_weights_kernel<<<(unsigned)((L.total + 255) / 256), 256, 0, s>>>(blob, dst, L, value_head, bf16);
  return cudaGetLastError();
}

cudaError_t launch_transpose_pad(const float* src, float* dst, int rows, int cols, int ld_dst, cudaStream_t s) {
  const size_t n = (size_t)cols * ld_dst;
  transpose_pad_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(src, dst, rows, cols, ld_dst);
  return cudaGetLastError();
}

cudaError_t launch_eligible(const int* block_ver, int n_blocks, long long v_learner, long long bound, int* elig_list,
                            int* elig_count, cudaStream_t s) {
  eligible_kernel<<<1, 1024, 0, s>>>(block_ver, n_blocks, v_learner, bound, elig_list, elig_count);
  return cudaGetLastError();
}

cudaError_t launch_sample_gather(const SampleParams& p, cudaStream_t s) {
  const int warps_per_block = 8;
  const bool aligned = ((reinterpret_cast<uintptr_t>(p.obs) | reinterpret_cast<uintptr_t>(p.next_obs)) & 15) == 0;
  if (p.D % 4 == 0 && aligned) {
    if (p.rec_words <= 32) {      // a few chunks per record: four lanes per draw, eight draws per warp
      const int draws_per_block = warps_per_block * 8;
      sample_gather_vec_kernel<4><<<(p.B + draws_per_block - 1) / draws_per_block, warps_per_block * 32, 0, s>>>(p);
    } else {
      sample_gather_vec_kernel<32><<<(p.B + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, s>>>(p);
    }
    return cudaGetLastError();
  }
  sample_gather_kernel<<<(p.B + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, s>>>(p);
  return cudaGetLastError();
}

int td_grid(int n) { return (n + kTdTile - 1) / kTdTile; }

template <int TE, int NT, int EPT, int NPT, int STAGE>
cudaError_t launch_td_stage(const TdParams& p, size_t smem, int grid, cudaStream_t s) {
  auto kernel = td_kernel<TE, NT, EPT, NPT, STAGE>;
  if (smem > 48 * 1024) {
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
  }
  kernel<<<grid, NT, smem, s>>>(p);
  return cudaGetLastError();
}

// tile: 16 rows x 128 threads with 4 x 4 register tiles; wide layers (hidden >= 192) 32 rows x 128 threads, 8 x 8
template <int TE, int NT, int EPT, int NPT>
cudaError_t launch_td_tile(const TdParams& p, cudaStream_t s, int* grid_out) {
  const int Dx = (p.D + 3) & ~3;
  const size_t acts = (size_t)Dx * TE + 2 * (size_t)p.Hp * TE + (size_t)p.Ap * TE + 2 * TE;
  const size_t limit = 226 * 1024;
  const size_t smem2 = (acts + p.w_total) * sizeof(float);
  const size_t smem1 = (acts + p.w_total - (p.off_b2 - p.off_W2t)) * sizeof(float);
  const size_t smem0 = acts * sizeof(float);
  const int grid = (p.n + TE - 1) / TE;
  *grid_out = grid;
  if (smem2 <= 112 * 1024) return launch_td_stage<TE, NT, EPT, NPT, 2>(p, smem2, grid, s);
  if (smem1 <= limit) return launch_td_stage<TE, NT, EPT, NPT, 1>(p, smem1, grid, s);
  if (smem0 <= limit) return launch_td_stage<TE, NT, EPT, NPT, 0>(p, smem0, grid, s);
  return cudaErrorInvalidConfiguration;
}

cudaError_t launch_td(const TdParams& p, cudaStream_t s) {
  int grid = 0;
  cudaError_t err = p.H >= 192 ? launch_td_tile<32, 128, 8, 8>(p, s, &grid) : launch_td_tile<kTdTile, kTdThreads, 4, 4>(p, s, &grid);
  if (err != cudaSuccess) return err;
  if (p.loss_out) {
    td_finish_kernel<<<1, 32, 0, s>>>(p.partial, grid, p.n, p.loss_out);
    err = cudaGetLastError();
  }
  return err;
}

// Scratch for tj_td_error_static: it is part of the library image, so every GPU that loads the library
// holds these 32 KB until the process exits and nobody has to allocate it.
constexpr int kStaticTdPartials = 8192;
static __device__ __align__(256) float g_td_static_partial[kStaticTdPartials];

int td_static_max_rows() { return 65536; }

cudaError_t launch_td_static(const TdParams& p_in, int device, cudaStream_t s, bool* too_large) {
  *too_large = p_in.n > td_static_max_rows() || td_grid(p_in.n) > kStaticTdPartials;
  if (*too_large) return cudaSuccess;
  // In host code the array's name is only a stand-in; the device address has to be asked for, once per device, with
  // that device current.  The table is keyed by the context's device and filled under a lock, so first calls from
  // several threads (one context each) do not race.
  static float* addr_by_device[64] = {};
  static std::mutex addr_lock;
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (device < 0 || device >= 64 || dev != device) return cudaErrorInvalidDevice;
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> hold(addr_lock);
    if (!addr_by_device[device]) {
      float* q = nullptr;
      e = cudaGetSymbolAddress(reinterpret_cast<void**>(&q), g_td_static_partial);
      if (e != cudaSuccess) return e;
      addr_by_device[device] = q;
    }
    scratch = addr_by_device[device];
  }
  TdParams p = p_in;
  p.partial = scratch;
  return launch_td(p, s);
}

cudaError_t launch_td_finish(const float* partial, int n_partial, int n, float* loss_out, cudaStream_t s) {
  td_finish_kernel<<<1, 32, 0, s>>>(partial, n_partial, n, loss_out);
  return cudaGetLastError();
}

cudaError_t launch_gae(const float* rew, const float* val, const uint8_t* done, int T, int N, float gamma, float lambda,
                       float* adv, float* ret, cudaStream_t s) {
  gae_kernel<<<(N + 127) / 128, 128, 0, s>>>(rew, val, done, T, N, gamma, lambda, adv, ret);
  return cudaGetLastError();
}

}  // namespace tj
