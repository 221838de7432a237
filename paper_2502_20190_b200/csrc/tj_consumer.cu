// On-policy consumer kernels (App. C, synchronous mode; Table 2's PPO batch settings): per-segment advantage normalisation
// and shuffled minibatches of segment rows.
#include "tj_device.cuh"
#include "tj_internal.h"

namespace tj {

namespace {

constexpr int NORM_THREADS = 256;
constexpr int NORM_MAX_BLOCKS = 1024;

// fixed-order block sum in double: lanes by shuffles, then the warps' sums in index order
__device__ __forceinline__ double block_sum(double v, double* warp_sums) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) warp_sums[warp] = v;
  __syncthreads();
  double s = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < NORM_THREADS / 32; ++w) s += warp_sums[w];
  __syncthreads();
  return s;   // valid in thread 0
}

// the sum of the per-block partials in index order (every block computes the same value the same way)
__device__ __forceinline__ double sum_partials(const double* partial, int n_blocks, double* shared_out) {
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int b = 0; b < n_blocks; ++b) s += partial[b];
    *shared_out = s;
  }
  __syncthreads();
  return *shared_out;
}

// pass 1: partial[b] = sum of x over the block's slice (slices are contiguous, fixed by n and the grid)
__global__ void __launch_bounds__(NORM_THREADS) norm_sum_kernel(const float* __restrict__ x, long long n, double* __restrict__ partial) {
  __shared__ double ws[NORM_THREADS / 32];
  const long long per = (n + gridDim.x - 1) / gridDim.x, lo = per * blockIdx.x, hi = lo + per < n ? lo + per : n;
  double v = 0.0;
  for (long long i = lo + threadIdx.x; i < hi; i += NORM_THREADS) v += (double)x[i];
  const double s = block_sum(v, ws);
  if (threadIdx.x == 0) partial[blockIdx.x] = s;
}

// pass 2: partial2[b] = sum of (x - mean)^2 over the block's slice
__global__ void __launch_bounds__(NORM_THREADS) norm_sqdev_kernel(const float* __restrict__ x, long long n, const double* __restrict__ partial,
                                                                double* __restrict__ partial2) {
  __shared__ double ws[NORM_THREADS / 32];
  __shared__ double tot;
  const double mean = sum_partials(partial, gridDim.x, &tot) / (double)n;
  const long long per = (n + gridDim.x - 1) / gridDim.x, lo = per * blockIdx.x, hi = lo + per < n ? lo + per : n;
  double v = 0.0;
  for (long long i = lo + threadIdx.x; i < hi; i += NORM_THREADS) {
    const double d = (double)x[i] - mean;
    v += d * d;
  }
  const double s = block_sum(v, ws);
  if (threadIdx.x == 0) partial2[blockIdx.x] = s;
}

// pass 3: out = (x - mean) / (sqrt(var) + eps)
__global__ void __launch_bounds__(NORM_THREADS) norm_apply_kernel(const float* __restrict__ x, long long n, const double* __restrict__ partial,
                                                                const double* __restrict__ partial2, double eps, float* __restrict__ out) {
  __shared__ double tot, tot2;
  const double mean = sum_partials(partial, gridDim.x, &tot) / (double)n;
  const double var = sum_partials(partial2, gridDim.x, &tot2) / (double)n;
  const double inv = 1.0 / (sqrt(var) + eps);
  const long long per = (n + gridDim.x - 1) / gridDim.x, lo = per * blockIdx.x, hi = lo + per < n ? lo + per : n;
  for (long long i = lo + threadIdx.x; i < hi; i += NORM_THREADS) out[i] = (float)(((double)x[i] - mean) * inv);
}

// Keyed bijection of [0, R): four Feistel rounds on 2 * hb bits with the SHUFFLE stream's first word as the round function,
// then cycle walking.  A permutation's cycle through a value below R returns below R, so the walk ends; the cap only
// guards the loop formally (it equals the size of the Feistel domain).
__device__ __forceinline__ unsigned long long feistel4(uint2 seed, unsigned long long shuffle_id, int hb, unsigned long long x) {
  const unsigned long long mask = (1ull << hb) - 1ull;
  unsigned long long left = x >> hb, right = x & mask;
#pragma unroll
  for (uint32_t round = 0; round < 4; ++round) {
    const uint4 w = stream_words(seed, STREAM_SHUFFLE, round, (uint32_t)right, shuffle_id);
    const unsigned long long nr = left ^ ((unsigned long long)w.x & mask);
    left = right;
    right = nr;
  }
  return (left << hb) | right;
}

__device__ __forceinline__ long long shuffle_index(uint2 seed, unsigned long long shuffle_id, int hb, long long R, long long i) {
  unsigned long long y = feistel4(seed, shuffle_id, hb, (unsigned long long)i);
  for (unsigned long long guard = 0; y >= (unsigned long long)R && guard < (1ull << (2 * hb)); ++guard) y = feistel4(seed, shuffle_id, hb, y);
  return (long long)y;
}

// one thread per minibatch row: position first + j of the shuffled order -> source row -> dense copies
__global__ void segment_minibatch_kernel(const MinibatchParams p) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= p.n) return;
  const long long src = shuffle_index(p.seed, p.shuffle_id, p.hb, p.R, p.first + j);
  const int D = p.D;
  if ((D & 3) == 0) {
    const float4* s4 = reinterpret_cast<const float4*>(p.seg_obs + (size_t)src * D);
    float4* d4 = reinterpret_cast<float4*>(p.obs + (size_t)j * D);
    for (int c = 0; c < D / 4; ++c) d4[c] = s4[c];
  } else {
    for (int c = 0; c < D; ++c) p.obs[(size_t)j * D + c] = p.seg_obs[(size_t)src * D + c];
  }
  p.act[j] = p.seg_act[src];
  p.logp[j] = p.seg_logp[src];
  p.adv[j] = p.adv_in[src];
  p.ret[j] = p.ret_in[src];
  if (p.row) p.row[j] = (int)src;
}

}  // namespace

int shuffle_half_bits(long long R) {
  int bits = 0;
  while (bits < 62 && (1ll << bits) < R) ++bits;
  const int hb = (bits + 1) / 2;
  return hb < 1 ? 1 : hb;
}

size_t normalize_scratch_doubles() { return 2 * NORM_MAX_BLOCKS; }

cudaError_t launch_normalize(const float* x, long long n, double eps, float* out, double* scratch, cudaStream_t s) {
  long long blocks = (n + 4 * NORM_THREADS - 1) / (4 * NORM_THREADS);
  if (blocks > NORM_MAX_BLOCKS) blocks = NORM_MAX_BLOCKS;
  if (blocks < 1) blocks = 1;
  double* p1 = scratch;
  double* p2 = scratch + NORM_MAX_BLOCKS;
  norm_sum_kernel<<<(unsigned)blocks, NORM_THREADS, 0, s>>>(x, n, p1);
  norm_sqdev_kernel<<<(unsigned)blocks, NORM_THREADS, 0, s>>>(x, n, p1, p2);
  norm_apply_kernel<<<(unsigned)blocks, NORM_THREADS, 0, s>>>(x, n, p1, p2, eps, out);
  return cudaGetLastError();
}

cudaError_t launch_segment_minibatch(const MinibatchParams& p, cudaStream_t s) {
  if (p.n <= 0) return cudaSuccess;
  segment_minibatch_kernel<<<(p.n + 127) / 128, 128, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tj
