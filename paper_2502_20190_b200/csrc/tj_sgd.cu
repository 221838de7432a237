// Learner update (Algorithm 1: theta <- theta + alpha * delta * grad V(s; theta)) as one minibatch semi-gradient step on
// the mean Huber loss of the TD error, FP32, on parameter blobs in the publish layout
// [W1 H x D, b1, W2 H x H, b2, W3 A x H, b3] (row-major out x in):
//   forward   h1, h2 of the online network kept, q = Q(s, a; theta), q' = max_a Q(s', a; theta_target),
//             delta = r + gamma (1 - done) q' - q, g = -clip(delta, -kappa, kappa) / n  (= dL/dq)
//   backward  dh2 = g W3[a] (h2 > 0), dh1 = (W2^T dh2) (h1 > 0)
//   update    W3[a] -= lr sum_j g_j h2_j, W2 -= lr dh2^T h1, W1 -= lr dh1^T x, biases likewise
// Every sum runs in a fixed order (rows ascending), so a step is reproducible bit for bit.
#include "tj_internal.h"

namespace tj {

namespace {

constexpr int SG_ROWS = 16;       // minibatch rows per thread block in the forward and backward kernels
constexpr int SG_THREADS = 256;

// one dense layer for SG_ROWS rows at once: out[i][r] = (relu)(b[i] + sum_k W[i][k] in[k][r]); activations live in shared
// memory k-major, so a step of the inner loop is one weight times 16 broadcast values
template <bool RELU>
__device__ __forceinline__ void sg_dense(const float* __restrict__ W, const float* __restrict__ b, int n_out, int n_in,
                                         const float* in, float* out) {
  for (int i = threadIdx.x; i < n_out; i += SG_THREADS) {
    float acc[SG_ROWS];
    const float bi = b[i];
#pragma unroll
    for (int r = 0; r < SG_ROWS; ++r) acc[r] = bi;
    const float* w = W + (size_t)i * n_in;
    for (int k = 0; k < n_in; ++k) {
      const float wk = __ldg(w + k);
      const float4* a = reinterpret_cast<const float4*>(in + (size_t)k * SG_ROWS);
#pragma unroll
      for (int r4 = 0; r4 < SG_ROWS / 4; ++r4) {
        const float4 v = a[r4];
        acc[4 * r4 + 0] = fmaf(wk, v.x, acc[4 * r4 + 0]);
        acc[4 * r4 + 1] = fmaf(wk, v.y, acc[4 * r4 + 1]);
        acc[4 * r4 + 2] = fmaf(wk, v.z, acc[4 * r4 + 2]);
        acc[4 * r4 + 3] = fmaf(wk, v.w, acc[4 * r4 + 3]);
      }
    }
#pragma unroll
    for (int r = 0; r < SG_ROWS; ++r) out[(size_t)i * SG_ROWS + r] = RELU ? fmaxf(acc[r], 0.f) : acc[r];
  }
}

// shared memory: xs [D][16] | a1 [H][16] | a2 [H][16] | qs [A][16]
__global__ void __launch_bounds__(SG_THREADS) sgd_forward_kernel(const SgdParams p) {
  extern __shared__ __align__(16) float sg_sm[];
  const int D = p.D, H = p.H, A = p.A;
  float* xs = sg_sm;
  float* a1 = xs + (size_t)D * SG_ROWS;
  float* a2 = a1 + (size_t)H * SG_ROWS;
  float* qs = a2 + (size_t)H * SG_ROWS;
  __shared__ float qsel[SG_ROWS], hub[SG_ROWS];
  const int row0 = blockIdx.x * SG_ROWS;
  const float *W1 = p.theta, *b1 = W1 + (size_t)H * D, *W2 = b1 + H, *b2 = W2 + (size_t)H * H, *W3 = b2 + H, *b3 = W3 + (size_t)A * H;
  const float *T1 = p.theta_target, *tb1 = T1 + (size_t)H * D, *T2 = tb1 + H, *tb2 = T2 + (size_t)H * H, *T3 = tb2 + H,
              *tb3 = T3 + (size_t)A * H;
  // ---- online network on obs; h1 and h2 are kept for the backward pass
  for (int i = threadIdx.x; i < D * SG_ROWS; i += SG_THREADS) {
    const int k = i / SG_ROWS, r = i % SG_ROWS;
    xs[i] = row0 + r < p.n ? p.obs[(size_t)(row0 + r) * D + k] : 0.f;
  }
  __syncthreads();
  sg_dense<true>(W1, b1, H, D, xs, a1);
  __syncthreads();
  sg_dense<true>(W2, b2, H, H, a1, a2);
  __syncthreads();
  sg_dense<false>(W3, b3, A, H, a2, qs);
  for (int i = threadIdx.x; i < H * SG_ROWS; i += SG_THREADS) {
    const int k = i / SG_ROWS, r = i % SG_ROWS;
    if (row0 + r < p.n) {
      p.h1[(size_t)(row0 + r) * H + k] = a1[i];
      p.h2[(size_t)(row0 + r) * H + k] = a2[i];
    }
  }
  __syncthreads();
  if (threadIdx.x < SG_ROWS && row0 + threadIdx.x < p.n) {
    int a = p.act[row0 + threadIdx.x];
    a = a < 0 ? 0 : (a >= A ? A - 1 : a);
    qsel[threadIdx.x] = qs[(size_t)a * SG_ROWS + threadIdx.x];
  }
  __syncthreads();
  // ---- target network on next_obs
  for (int i = threadIdx.x; i < D * SG_ROWS; i += SG_THREADS) {
    const int k = i / SG_ROWS, r = i % SG_ROWS;
    xs[i] = row0 + r < p.n ? p.next_obs[(size_t)(row0 + r) * D + k] : 0.f;
  }
  __syncthreads();
  sg_dense<true>(T1, tb1, H, D, xs, a1);
  __syncthreads();
  sg_dense<true>(T2, tb2, H, H, a1, a2);
  __syncthreads();
  sg_dense<false>(T3, tb3, A, H, a2, qs);
  __syncthreads();
  if (threadIdx.x < SG_ROWS) {
    const int r = threadIdx.x, j = row0 + r;
    float h = 0.f;
    if (j < p.n) {
      float qmax = qs[r];
      for (int i = 1; i < A; ++i) qmax = fmaxf(qmax, qs[(size_t)i * SG_ROWS + r]);
      const float y = p.rew[j] + p.gamma * (p.done[j] ? 0.f : 1.f) * qmax;
      const float delta = y - qsel[r], ad = fabsf(delta);
      h = ad <= p.kappa ? 0.5f * delta * delta : p.kappa * (ad - 0.5f * p.kappa);
      p.g[j] = -fminf(fmaxf(delta, -p.kappa), p.kappa) / (float)p.n;
    }
    hub[r] = h;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int r = 0; r < SG_ROWS; ++r) s += hub[r];
    p.partial[blockIdx.x] = s;
  }
}

// backward through the activations, SG_ROWS rows per block: shared memory d2 [H][16]
__global__ void __launch_bounds__(SG_THREADS) sgd_backward_kernel(const SgdParams p) {
  extern __shared__ __align__(16) float sg_sm[];
  const int D = p.D, H = p.H, A = p.A;
  float* d2 = sg_sm;
  __shared__ float gs[SG_ROWS];
  __shared__ int as[SG_ROWS];
  const int row0 = blockIdx.x * SG_ROWS;
  const float* W2 = p.theta + (size_t)H * D + H;
  const float* W3 = W2 + (size_t)H * H + H;
  if (threadIdx.x < SG_ROWS) {
    const int j = row0 + threadIdx.x;
    int a = j < p.n ? p.act[j] : 0;
    as[threadIdx.x] = a < 0 ? 0 : (a >= A ? A - 1 : a);
    gs[threadIdx.x] = j < p.n ? p.g[j] : 0.f;
  }
  __syncthreads();
  // dh2[r][i] = g_r W3[a_r][i] where h2 > 0
  for (int idx = threadIdx.x; idx < H * SG_ROWS; idx += SG_THREADS) {
    const int r = idx / H, i = idx % H, j = row0 + r;
    float v = 0.f;
    if (j < p.n && p.h2[(size_t)j * H + i] > 0.f) v = gs[r] * W3[(size_t)as[r] * H + i];
    d2[(size_t)i * SG_ROWS + r] = v;
    if (j < p.n) p.dh2[(size_t)j * H + i] = v;
  }
  __syncthreads();
  // dh1[r][k] = sum_i W2[i][k] dh2[r][i] where h1 > 0 (threads along k: the weight loads are coalesced)
  for (int k = threadIdx.x; k < H; k += SG_THREADS) {
    float acc[SG_ROWS];
#pragma unroll
    for (int r = 0; r < SG_ROWS; ++r) acc[r] = 0.f;
    for (int i = 0; i < H; ++i) {
      const float w = __ldg(W2 + (size_t)i * H + k);
      const float4* a = reinterpret_cast<const float4*>(d2 + (size_t)i * SG_ROWS);
#pragma unroll
      for (int r4 = 0; r4 < SG_ROWS / 4; ++r4) {
        const float4 v = a[r4];
        acc[4 * r4 + 0] = fmaf(w, v.x, acc[4 * r4 + 0]);
        acc[4 * r4 + 1] = fmaf(w, v.y, acc[4 * r4 + 1]);
        acc[4 * r4 + 2] = fmaf(w, v.z, acc[4 * r4 + 2]);
        acc[4 * r4 + 3] = fmaf(w, v.w, acc[4 * r4 + 3]);
      }
    }
#pragma unroll
    for (int r = 0; r < SG_ROWS; ++r) {
      const int j = row0 + r;
      if (j < p.n) p.dh1[(size_t)j * H + k] = p.h1[(size_t)j * H + k] > 0.f ? acc[r] : 0.f;
    }
  }
}

// C[m][n] -= lr * sum_j A[j][m] * Bm[j][n]   (C row-major M x N; A n_rows x M with row stride lda; Bm n_rows x N, stride ldb)
// 32 x 32 tile per block, 256 threads, each 2 x 2; rows j in ascending order
__global__ void __launch_bounds__(256) sgd_update_matrix_kernel(float* __restrict__ Cm, int M, int N, const float* __restrict__ Am,
                                                                int lda, const float* __restrict__ Bm, int ldb, int n_rows,
                                                                float lr) {
  __shared__ float As[32][33], Bs[32][33];
  const int m0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
  for (int j0 = 0; j0 < n_rows; j0 += 32) {
    for (int i = threadIdx.x; i < 32 * 32; i += 256) {
      const int jj = i >> 5, c = i & 31, j = j0 + jj;
      As[jj][c] = (j < n_rows && m0 + c < M) ? Am[(size_t)j * lda + m0 + c] : 0.f;
      Bs[jj][c] = (j < n_rows && n0 + c < N) ? Bm[(size_t)j * ldb + n0 + c] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int jj = 0; jj < 32; ++jj) {
      const float a0 = As[jj][ty], a1 = As[jj][ty + 16], b0 = Bs[jj][tx], b1 = Bs[jj][tx + 16];
      acc[0][0] = fmaf(a0, b0, acc[0][0]);
      acc[0][1] = fmaf(a0, b1, acc[0][1]);
      acc[1][0] = fmaf(a1, b0, acc[1][0]);
      acc[1][1] = fmaf(a1, b1, acc[1][1]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 2; ++u)
#pragma unroll
    for (int v = 0; v < 2; ++v) {
      const int m = m0 + ty + 16 * u, n = n0 + tx + 16 * v;
      if (m < M && n < N) Cm[(size_t)m * N + n] -= lr * acc[u][v];
    }
}

// b[m] -= lr * sum_j A[j][m]
__global__ void sgd_update_bias_kernel(float* __restrict__ b, int M, const float* __restrict__ Am, int lda, int n_rows, float lr) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= M) return;
  float s = 0.f;
  for (int j = 0; j < n_rows; ++j) s += Am[(size_t)j * lda + m];
  b[m] -= lr * s;
}

// head: W3[a][i] -= lr * sum_{j: a_j = a} g_j h2[j][i];  b3[a] -= lr * sum_{j: a_j = a} g_j.   grid (ceil(H/128), A)
__global__ void sgd_update_head_kernel(const SgdParams p, float lr) {
  const int H = p.H, A = p.A, a = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
  float* W3 = p.theta + (size_t)H * p.D + H + (size_t)H * H + H;
  float* b3 = W3 + (size_t)A * H;
  float s = 0.f, sb = 0.f;
  for (int j = 0; j < p.n; ++j) {
    int aj = p.act[j];
    aj = aj < 0 ? 0 : (aj >= A ? A - 1 : aj);
    if (aj != a) continue;
    const float g = p.g[j];
    sb += g;
    if (i < H) s = fmaf(g, p.h2[(size_t)j * H + i], s);
  }
  if (i < H) W3[(size_t)a * H + i] -= lr * s;
  if (i == 0) b3[a] -= lr * sb;
}

}  // namespace

size_t sgd_scratch_floats(int max_rows, int H) {
  const size_t rows = ((size_t)max_rows + SG_ROWS - 1) / SG_ROWS * SG_ROWS;
  return 4 * rows * (size_t)H + rows + rows / SG_ROWS + 64;
}

int sgd_partial_count(int n) { return (n + SG_ROWS - 1) / SG_ROWS; }

bool sgd_supported(int D, int H, int A) {
  const size_t smem = ((size_t)D + 2 * (size_t)H + A) * SG_ROWS * sizeof(float);
  return H >= 1 && D >= 1 && A >= 1 && smem <= 200 * 1024;
}

cudaError_t launch_sgd_step(const SgdParams& p, float lr, cudaStream_t s) {
  const int D = p.D, H = p.H, A = p.A;
  const int grid = sgd_partial_count(p.n);
  const size_t smem_f = ((size_t)D + 2 * (size_t)H + A) * SG_ROWS * sizeof(float);
  const size_t smem_b = (size_t)H * SG_ROWS * sizeof(float);
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(sgd_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_f)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(sgd_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_b)) != cudaSuccess) return e;
  sgd_forward_kernel<<<grid, SG_THREADS, smem_f, s>>>(p);
  sgd_backward_kernel<<<grid, SG_THREADS, smem_b, s>>>(p);
  float* W1 = p.theta;
  float* b1 = W1 + (size_t)H * D;
  float* W2 = b1 + H;
  float* b2 = W2 + (size_t)H * H;
  // the backward pass has read W2 and W3; now the parameters may change
  sgd_update_head_kernel<<<dim3((H + 127) / 128, A), 128, 0, s>>>(p, lr);
  sgd_update_matrix_kernel<<<dim3((H + 31) / 32, (H + 31) / 32), 256, 0, s>>>(W2, H, H, p.dh2, H, p.h1, H, p.n, lr);
  sgd_update_bias_kernel<<<(H + 127) / 128, 128, 0, s>>>(b2, H, p.dh2, H, p.n, lr);
  sgd_update_matrix_kernel<<<dim3((D + 31) / 32, (H + 31) / 32), 256, 0, s>>>(W1, H, D, p.dh1, H, p.obs, D, p.n, lr);
  sgd_update_bias_kernel<<<(H + 127) / 128, 128, 0, s>>>(b1, H, p.dh1, H, p.n, lr);
  return cudaGetLastError();
}

}  // namespace tj
