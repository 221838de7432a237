// FP32 dense layer for a tile of TE environments (or samples) held in shared memory.
//
// Activations are stored k-major, x[k][e], so that the four environments a thread owns are one 128-bit
// shared-memory load and the four output neurons it owns are one 128-bit load from the transposed weight
// matrix Wt[k][i].  Every output is accumulated as  acc = bias;  acc = fma(Wt[k][i], x[k][e], acc)  for
// k = 0, 1, 2, ...: one rounding order, independent of the tiling, so results do not depend on launch shape.
#pragma once
#include <cuda_runtime.h>

namespace tj {

constexpr int kThreads = 256;

enum { ACT_NONE = 0, ACT_RELU = 1, ACT_TANH = 2 };

template <int ACT>
__device__ __forceinline__ float activate(float v) {
  if (ACT == ACT_RELU) return v > 0.0f ? v : 0.0f;
  if (ACT == ACT_TANH) return tanhf(v);
  return v;
}

// y[i][e] = act(bias + sum_k Wt[k][i] x[k][e]) for i < round_up4(n_out), e < TE.
//   Wt: [K][ldw] (global, zero padded to ldw = round_up4(n_out)),  x: [K][TE] shared,  y: [round_up4(n_out)][TE] shared
//   ENV_BIAS = false: bias = b[i];  true: bias = b[bias_row[e] * ldw + i] (a per-environment row of b)
template <int TE, int ACT, bool ENV_BIAS>
__device__ __forceinline__ void dense_layer(const float* __restrict__ Wt, const float* __restrict__ b, int ldw, int K,
                                            int n_out, const float* __restrict__ x, float* __restrict__ y,
                                            const int* __restrict__ bias_row) {
  constexpr int EG = TE / 4, NG = kThreads / EG;
  const int eg = threadIdx.x % EG, ng = threadIdx.x / EG;
  for (int i0 = ng * 4; i0 < n_out; i0 += NG * 4) {
    float acc[4][4];  // [neuron][env]
    if (ENV_BIAS) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 bb = __ldg(reinterpret_cast<const float4*>(b + (size_t)bias_row[eg * 4 + e] * ldw + i0));
        acc[0][e] = bb.x; acc[1][e] = bb.y; acc[2][e] = bb.z; acc[3][e] = bb.w;
      }
    } else {
      const float4 bb = __ldg(reinterpret_cast<const float4*>(b + i0));
#pragma unroll
      for (int e = 0; e < 4; ++e) { acc[0][e] = bb.x; acc[1][e] = bb.y; acc[2][e] = bb.z; acc[3][e] = bb.w; }
    }
    const float* xp = x + eg * 4;
    const float* wp = Wt + i0;
#pragma unroll 4
    for (int k = 0; k < K; ++k) {
      const float4 xv = *reinterpret_cast<const float4*>(xp + k * TE);
      const float4 wv = __ldg(reinterpret_cast<const float4*>(wp + (size_t)k * ldw));
      const float xe[4] = {xv.x, xv.y, xv.z, xv.w};
      const float wn[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[n][e] = fmaf(wn[n], xe[e], acc[n][e]);
    }
#pragma unroll
    for (int n = 0; n < 4; ++n) {
      float4 o;
      o.x = activate<ACT>(acc[n][0]); o.y = activate<ACT>(acc[n][1]);
      o.z = activate<ACT>(acc[n][2]); o.w = activate<ACT>(acc[n][3]);
      *reinterpret_cast<float4*>(y + (size_t)(i0 + n) * TE + eg * 4) = o;
    }
  }
}

// Policy forward for the tile: x [D][TE] -> h1 -> h2 -> out [Ap][TE]; ends with a barrier.
template <int TE>
__device__ __forceinline__ void mlp_forward_tile(const float* __restrict__ W, size_t off_W1t, size_t off_b1,
                                                 size_t off_W2t, size_t off_b2, size_t off_W3t, size_t off_b3, int D,
                                                 int H, int Hp, int Aout, int Ap, const float* x, float* h1, float* h2,
                                                 float* out) {
  dense_layer<TE, ACT_RELU, false>(W + off_W1t, W + off_b1, Hp, D, H, x, h1, nullptr);
  __syncthreads();
  dense_layer<TE, ACT_RELU, false>(W + off_W2t, W + off_b2, Hp, H, H, h1, h2, nullptr);
  __syncthreads();
  dense_layer<TE, ACT_NONE, false>(W + off_W3t, W + off_b3, Ap, H, Aout, h2, out, nullptr);
  __syncthreads();
}

}  // namespace tj
