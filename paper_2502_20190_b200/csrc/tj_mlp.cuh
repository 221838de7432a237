// FP32 dense layers for a tile of TE environments (or samples) held in shared memory.
//
// Activations are stored k-major, x[k][e], so that the four environments a thread owns are one 128-bit
// shared-memory load and the four output neurons it owns are one 128-bit load from the transposed weight
// matrix Wt[k][i].  Every output is accumulated as  acc = bias;  acc = fma(Wt[k][i], x[k][e], acc)  for
// k = 0, 1, 2, ...: one rounding order, independent of the tiling, so results do not depend on launch shape.
#pragma once
#include <cuda_runtime.h>

#include "tj_async.cuh"

namespace tj {

enum { ACT_NONE = 0, ACT_RELU = 1, ACT_TANH = 2 };

template <int ACT>
__device__ __forceinline__ float activate(float v) {
  if (ACT == ACT_RELU) return v > 0.0f ? v : 0.0f;
  if (ACT == ACT_TANH) return tanhf(v);
  return v;
}

// weights either sit in shared memory (plain load) or in global memory (read-only path)
template <bool W_SMEM>
__device__ __forceinline__ float4 load_w4(const float* p) {
  if (W_SMEM) return *reinterpret_cast<const float4*>(p);
  return __ldg(reinterpret_cast<const float4*>(p));
}
template <bool W_SMEM>
__device__ __forceinline__ float load_w1(const float* p) {
  if (W_SMEM) return *p;
  return __ldg(p);
}

// y[i][e] = act(bias + sum_k Wt[k][i] x[k][e]) for i < round_up4(n_out), e < TE.
//   Wt: [K][ldw] (zero padded to ldw = round_up4(n_out)),  x: [K][TE] shared,  y: [round_up4(n_out)][TE] shared
//   ENV_BIAS = false: bias = b[i];  true: bias = b[bias_row[e] * ldw + i] (a per-environment row of b, global)
//   W_SMEM / B_SMEM: whether Wt / b sit in shared memory (else global, read-only path)
//   EPT: environments per thread (4 or 8).  A thread owns EPT environments x 4 neurons; with 8 environments each
//   weight fetched feeds twice as many FMAs, which is what shared-memory (or L2) bandwidth asks for.
//   NPT: neurons per thread (4 or 8): 8 x 8 register tiles do 64 FMAs per two activation and two weight loads.
template <int TE, int NT, int EPT, int ACT, bool ENV_BIAS, bool W_SMEM, bool B_SMEM = W_SMEM, int NPT = 4>
__device__ __forceinline__ void dense_layer(const float* __restrict__ Wt, const float* __restrict__ b, int ldw, int K,
                                            int n_out, const float* __restrict__ x, float* __restrict__ y,
                                            const int* __restrict__ bias_row) {
  constexpr int EG = TE / EPT, NG = NT / EG, XV = EPT / 4, WV = NPT / 4;
  const int eg = threadIdx.x % EG, ng = threadIdx.x / EG;
  for (int i0 = ng * NPT; i0 < n_out; i0 += NG * NPT) {
    float acc[NPT][EPT];  // [neuron][env]
    bool wv_ok[WV];       // a thread's second group of four neurons may lie beyond the padded width
#pragma unroll
    for (int u = 0; u < WV; ++u) wv_ok[u] = i0 + 4 * u < ldw;
#pragma unroll
    for (int u = 0; u < WV; ++u) {
      if (ENV_BIAS) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
          float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
          if (wv_ok[u]) bb = __ldg(reinterpret_cast<const float4*>(b + (size_t)bias_row[eg * EPT + e] * ldw + i0 + 4 * u));
          acc[4 * u][e] = bb.x; acc[4 * u + 1][e] = bb.y; acc[4 * u + 2][e] = bb.z; acc[4 * u + 3][e] = bb.w;
        }
      } else {
        float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
        if (wv_ok[u]) bb = load_w4<B_SMEM>(b + i0 + 4 * u);
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
          acc[4 * u][e] = bb.x; acc[4 * u + 1][e] = bb.y; acc[4 * u + 2][e] = bb.z; acc[4 * u + 3][e] = bb.w;
        }
      }
    }
    const float* xp = x + eg * EPT;
    const float* wp = Wt + i0;
#pragma unroll 8
    for (int k = 0; k < K; ++k) {
      float xe[EPT], wn[NPT];
#pragma unroll
      for (int v = 0; v < XV; ++v) {
        const float4 xv = *reinterpret_cast<const float4*>(xp + k * TE + 4 * v);
        xe[4 * v] = xv.x; xe[4 * v + 1] = xv.y; xe[4 * v + 2] = xv.z; xe[4 * v + 3] = xv.w;
      }
#pragma unroll
      for (int u = 0; u < WV; ++u) {
        float4 wv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (wv_ok[u]) wv = load_w4<W_SMEM>(wp + (size_t)k * ldw + 4 * u);
        wn[4 * u] = wv.x; wn[4 * u + 1] = wv.y; wn[4 * u + 2] = wv.z; wn[4 * u + 3] = wv.w;
      }
#pragma unroll
      for (int n = 0; n < NPT; ++n)
#pragma unroll
        for (int e = 0; e < EPT; ++e) acc[n][e] = fmaf(wn[n], xe[e], acc[n][e]);
    }
#pragma unroll
    for (int n = 0; n < NPT; ++n) {
      if (!wv_ok[n / 4]) continue;
#pragma unroll
      for (int v = 0; v < XV; ++v) {
        float4 o;
        o.x = activate<ACT>(acc[n][4 * v]); o.y = activate<ACT>(acc[n][4 * v + 1]);
        o.z = activate<ACT>(acc[n][4 * v + 2]); o.w = activate<ACT>(acc[n][4 * v + 3]);
        *reinterpret_cast<float4*>(y + (size_t)(i0 + n) * TE + eg * EPT + 4 * v) = o;
      }
    }
  }
}

// Narrow output layer (a few actions): one thread per (environment, output), same FMA chain.
template <int TE, int NT, bool W_SMEM>
__device__ __forceinline__ void head_layer(const float* __restrict__ Wt, const float* __restrict__ b, int ldw, int K,
                                           int n_out, const float* __restrict__ x, float* __restrict__ y) {
  for (int idx = threadIdx.x; idx < TE * n_out; idx += NT) {
    const int e = idx % TE, a = idx / TE;
    float acc = load_w1<W_SMEM>(b + a);
    const float* xp = x + e;
    const float* wp = Wt + a;
#pragma unroll 8
    for (int k = 0; k < K; ++k) acc = fmaf(load_w1<W_SMEM>(wp + (size_t)k * ldw), xp[k * TE], acc);
    y[a * TE + e] = acc;
  }
}

// Where each part of the packed parameters is read from (shared or global memory).
struct MlpWeights {
  const float *W1t, *b1, *W2t, *b2, *W3t, *b3;
};

// Queue the bulk copies of the staged parameter ranges (one thread, `issue`) and name where each part is read from.
// STAGE 0: everything from global memory; 1: all but the H x H matrix staged in shared memory; 2: all staged.
// P is a parameter struct with the packed layout's offsets (off_W1t .. off_b3, w_total); W the packed parameters.
template <int STAGE, typename P>
__device__ __forceinline__ MlpWeights stage_mlp_weights(const P& p, const float* W, float* wsm, uint64_t* bar, bool issue) {
  MlpWeights w;
  if (STAGE == 0) {
    w.W1t = W + p.off_W1t; w.b1 = W + p.off_b1; w.W2t = W + p.off_W2t; w.b2 = W + p.off_b2;
    w.W3t = W + p.off_W3t; w.b3 = W + p.off_b3;
    return w;
  }
  const size_t gap = STAGE == 1 ? p.off_b2 - p.off_W2t : 0;
  if (issue) {
    if (STAGE == 2) {
      mbar_expect_tx(bar, (uint32_t)(p.w_total * sizeof(float)));
      bulk_copy_chunks(wsm, W, p.w_total * sizeof(float), bar);
    } else {
      const size_t head = p.off_W2t, tail = p.w_total - p.off_b2;
      mbar_expect_tx(bar, (uint32_t)((head + tail) * sizeof(float)));
      bulk_copy_chunks(wsm, W, head * sizeof(float), bar);
      bulk_copy_chunks(wsm + head, W + p.off_b2, tail * sizeof(float), bar);
    }
  }
  w.W1t = wsm + p.off_W1t; w.b1 = wsm + p.off_b1;
  w.W2t = STAGE == 2 ? wsm + p.off_W2t : W + p.off_W2t;
  w.b2 = wsm + p.off_b2 - gap; w.W3t = wsm + p.off_W3t - gap; w.b3 = wsm + p.off_b3 - gap;
  return w;
}

// Policy forward for the tile: x [D][TE] -> h1 -> h2 -> out [Ap][TE]; ends with a barrier.
// SMALL_SMEM: W1t, the biases and W3t are in shared memory;  W2_SMEM: W2t is too.
template <int TE, int NT, int EPT, bool SMALL_SMEM, bool W2_SMEM, int NPT = 4>
__device__ __forceinline__ void mlp_forward_tile(const MlpWeights& w, int D, int H, int Hp, int Aout, int Ap,
                                                 const float* x, float* h1, float* h2, float* out) {
  dense_layer<TE, NT, EPT, ACT_RELU, false, SMALL_SMEM, SMALL_SMEM, NPT>(w.W1t, w.b1, Hp, D, H, x, h1, nullptr);
  __syncthreads();
  dense_layer<TE, NT, EPT, ACT_RELU, false, W2_SMEM, SMALL_SMEM, NPT>(w.W2t, w.b2, Hp, H, H, h1, h2, nullptr);
  __syncthreads();
  if (Aout <= 8) head_layer<TE, NT, SMALL_SMEM>(w.W3t, w.b3, Ap, H, Aout, h2, out);
  else dense_layer<TE, NT, EPT, ACT_NONE, false, SMALL_SMEM>(w.W3t, w.b3, Ap, H, Aout, h2, out, nullptr);
  __syncthreads();
}

}  // namespace tj
