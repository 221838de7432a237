// Measured FP32 fused-multiply-add rate of the device the library runs on: the denominator for the FP32 policy kernels'
// arithmetic roofline (Sec. 3.3 of the paper sizes actors and learners from measured rates; here the same idea gives
// the rate the FP32 path is held against).  One thread block per SM slot, every thread running eight independent FMA
// chains from registers; nothing but one result word per thread leaves the SM.
#include "tj_internal.h"

namespace tj {

namespace {

constexpr int CAL_THREADS = 256, CAL_CHAINS = 8, CAL_INNER = 64;

__global__ void __launch_bounds__(CAL_THREADS) fma_rate_kernel(float* __restrict__ sink, int outer, float a, float b) {
  float x[CAL_CHAINS];
#pragma unroll
  for (int i = 0; i < CAL_CHAINS; ++i) x[i] = (float)(threadIdx.x + i) * 1e-3f;
  for (int o = 0; o < outer; ++o) {
#pragma unroll
    for (int r = 0; r < CAL_INNER; ++r) {
#pragma unroll
      for (int i = 0; i < CAL_CHAINS; ++i) x[i] = fmaf(x[i], a, b);
    }
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < CAL_CHAINS; ++i) s += x[i];
  sink[(size_t)blockIdx.x * CAL_THREADS + threadIdx.x] = s;
}

}  // namespace

size_t fma_rate_sink_floats(int sm_count) { return (size_t)sm_count * 8 * CAL_THREADS; }

// flops of one launch; the launch itself
double launch_fma_rate(float* sink, int sm_count, int outer, cudaStream_t s, cudaError_t* err) {
  const int grid = sm_count * 8;     // 2,048 resident threads per SM
  fma_rate_kernel<<<grid, CAL_THREADS, 0, s>>>(sink, outer, 0.999f, 1e-3f);
  *err = cudaGetLastError();
  return 2.0 * (double)grid * CAL_THREADS * CAL_CHAINS * CAL_INNER * (double)outer;
}

}  // namespace tj
