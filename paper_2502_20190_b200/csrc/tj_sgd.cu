// Learner update (Algorithm 1: theta <- theta + alpha * delta * grad V(s; theta)) as one minibatch semi-gradient step on
// the mean Huber loss of the TD error, FP32, on parameter blobs in the publish layout
// [W1 H x D, b1, W2 H x H, b2, W3 A x H, b3] (row-major out x in):
//   forward   h1, h2 of the online network kept, q = Q(s, a; theta), q' = max_a Q(s', a; theta_target),
//             delta = r + gamma (1 - done) q' - q, g = -clip(delta, -kappa, kappa) / n  (= dL/dq)
//   backward  dh2 = g W3[a] (h2 > 0), dh1 = (W2^T dh2) (h1 > 0)
//   update    W3[a] -= lr sum_j g_j h2_j, W2 -= lr dh2^T h1, W1 -= lr dh1^T x, biases likewise
// Every sum runs in a fixed order (rows ascending), so a step is reproducible bit for bit.
#include "tj_internal.h"
#include "tj_tc.cuh"

namespace tj {

namespace {

constexpr int SG_ROWS = 16;       // minibatch rows per thread block in the forward and backward kernels
constexpr int SG_THREADS = 256;

constexpr int SG_KT = 32;         // K columns of the weight tile staged in shared memory

// one dense layer for SG_ROWS rows at once: out[i][r] = (relu)(b[i] + sum_k W[i][k] in[k][r]); activations live in shared
// memory k-major, so a step of the inner loop is one weight times 16 broadcast values.  The weights (row-major out x in)
// pass through a 256 x 32 shared-memory tile so that the global loads run along k, 128 contiguous bytes per row.
template <bool RELU>
__device__ __forceinline__ void sg_dense(const float* __restrict__ W, const float* __restrict__ b, int n_out, int n_in,
                                         const float* in, float* out, float* wt) {
  for (int i0 = 0; i0 < n_out; i0 += SG_THREADS) {
    const int i = i0 + threadIdx.x;
    float acc[SG_ROWS];
    const float bi = i < n_out ? b[i] : 0.f;
#pragma unroll
    for (int r = 0; r < SG_ROWS; ++r) acc[r] = bi;
    for (int k0 = 0; k0 < n_in; k0 += SG_KT) {
      __syncthreads();
      for (int t = threadIdx.x; t < SG_THREADS * SG_KT; t += SG_THREADS) {
        const int ii = t / SG_KT, kk = t % SG_KT;
        wt[ii * (SG_KT + 1) + kk] = (i0 + ii < n_out && k0 + kk < n_in) ? __ldg(W + (size_t)(i0 + ii) * n_in + k0 + kk) : 0.f;
      }
      __syncthreads();
      const int kn = n_in - k0 < SG_KT ? n_in - k0 : SG_KT;
      for (int kk = 0; kk < kn; ++kk) {
        const float wk = wt[threadIdx.x * (SG_KT + 1) + kk];
        const float4* a = reinterpret_cast<const float4*>(in + (size_t)(k0 + kk) * SG_ROWS);
#pragma unroll
        for (int r4 = 0; r4 < SG_ROWS / 4; ++r4) {
          const float4 v = a[r4];
          acc[4 * r4 + 0] = fmaf(wk, v.x, acc[4 * r4 + 0]);
          acc[4 * r4 + 1] = fmaf(wk, v.y, acc[4 * r4 + 1]);
          acc[4 * r4 + 2] = fmaf(wk, v.z, acc[4 * r4 + 2]);
          acc[4 * r4 + 3] = fmaf(wk, v.w, acc[4 * r4 + 3]);
        }
      }
    }
    if (i < n_out) {
#pragma unroll
      for (int r = 0; r < SG_ROWS; ++r) out[(size_t)i * SG_ROWS + r] = RELU ? fmaxf(acc[r], 0.f) : acc[r];
    }
  }
}

// shared memory: xs [D][16] | a1 [H][16] | a2 [H][16] | qs [A][16] | weight tile [256][33]
__global__ void __launch_bounds__(SG_THREADS) sgd_forward_kernel(const SgdParams p) {
  extern __shared__ __align__(16) float sg_sm[];
  const int D = p.D, H = p.H, A = p.A;
  float* xs = sg_sm;
  float* a1 = xs + (size_t)D * SG_ROWS;
  float* a2 = a1 + (size_t)H * SG_ROWS;
  float* qs = a2 + (size_t)H * SG_ROWS;
  float* wt = qs + (size_t)A * SG_ROWS;
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
  sg_dense<true>(W1, b1, H, D, xs, a1, wt);
  __syncthreads();
  sg_dense<true>(W2, b2, H, H, a1, a2, wt);
  __syncthreads();
  sg_dense<false>(W3, b3, A, H, a2, qs, wt);
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
  sg_dense<true>(T1, tb1, H, D, xs, a1, wt);
  __syncthreads();
  sg_dense<true>(T2, tb2, H, H, a1, a2, wt);
  __syncthreads();
  sg_dense<false>(T3, tb3, A, H, a2, qs, wt);
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
      const float gj = -fminf(fmaxf(delta, -p.kappa), p.kappa) / (float)p.n;
      int a = p.act[j];
      a = a < 0 ? 0 : (a >= A ? A - 1 : a);
      for (int i = 0; i < A; ++i) p.g[(size_t)j * A + i] = i == a ? gj : 0.f;
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

// ---------------------------------------------------------------------------------------------------------------------
// Wide networks and large minibatches: the layers as tiled FP32 matrix products (a weight element is reused for 128 rows
// instead of 16).  C[m][n] = epi(sum_k A[m][k] Bop[k][n]): A row-major M x K.  B_KN false: B is N x K row-major (a weight
// matrix as the forward pass uses it, Bop = B^T); true: B is K x N row-major (the same matrix in the backward pass).
// 128 x 64 tile per block (32 x 64 for the heads, whose few outputs would leave most SMs idle with tall tiles), 16 k per
// step, each thread 8 x 4 (2 x 4); k ascending, one accumulator per output: a fixed order.
constexpr int GM_BM = 128, GM_BN = 64, GM_BK = 16, GM_THREADS = 256;

template <bool B_KN, int EPI, int BM>
__device__ __forceinline__ void sg_gemm_body(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
                                             float* __restrict__ C, int ldc, int M, int N, int K,
                                             const float* __restrict__ bias, const float* __restrict__ mask, int ldm) {
  __shared__ __align__(16) float As[GM_BK][BM + 4];
  __shared__ __align__(16) float Bs[GM_BK][GM_BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  constexpr int RM = BM / 16;   // rows per thread
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * GM_BN;
  const bool vecA = (lda & 3) == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0;
  const bool vecB = (ldb & 3) == 0 && (reinterpret_cast<uintptr_t>(B) & 15) == 0;
  float acc[RM][4];
#pragma unroll
  for (int i = 0; i < RM; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  // four consecutive k of one row (of A, or of an N x K B): a 16-byte load where the row allows it
  auto load_k4 = [](const float* base, int ld, int row, int n_rows, int k, int K, bool vec) -> float4 {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row < n_rows && k < K) {
      const float* src = base + (size_t)row * ld + k;
      if (vec && k + 3 < K) {
        v = __ldg(reinterpret_cast<const float4*>(src));
      } else {
        v.x = __ldg(src);
        if (k + 1 < K) v.y = __ldg(src + 1);
        if (k + 2 < K) v.z = __ldg(src + 2);
        if (k + 3 < K) v.w = __ldg(src + 3);
      }
    }
    return v;
  };
  // the next k-step's operands travel from global memory to registers while this one is multiplied
  constexpr int NA = (BM * 4 + GM_THREADS - 1) / GM_THREADS;
  float4 ra[NA], rb;
  auto fetch = [&](int k0) {
#pragma unroll
    for (int u = 0; u < NA; ++u) {
      const int i = tid + u * GM_THREADS;
      if (i < BM * 4) ra[u] = load_k4(A, lda, m0 + (i >> 2), M, k0 + (i & 3) * 4, K, vecA);
    }
    if (!B_KN) {
      rb = load_k4(B, ldb, n0 + (tid >> 2), N, k0 + (tid & 3) * 4, K, vecB);
    } else {
      const int k = k0 + (tid >> 4), n = n0 + (tid & 15) * 4;
      rb = make_float4(0.f, 0.f, 0.f, 0.f);
      if (k < K && n < N) {
        const float* src = B + (size_t)k * ldb + n;
        if (vecB && n + 3 < N) {
          rb = __ldg(reinterpret_cast<const float4*>(src));
        } else {
          rb.x = __ldg(src);
          if (n + 1 < N) rb.y = __ldg(src + 1);
          if (n + 2 < N) rb.z = __ldg(src + 2);
          if (n + 3 < N) rb.w = __ldg(src + 3);
        }
      }
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < K; k0 += GM_BK) {
#pragma unroll
    for (int u = 0; u < NA; ++u) {
      const int i = tid + u * GM_THREADS, r = i >> 2, kq = (i & 3) * 4;
      if (i >= BM * 4) break;
      As[kq][r] = ra[u].x; As[kq + 1][r] = ra[u].y; As[kq + 2][r] = ra[u].z; As[kq + 3][r] = ra[u].w;
    }
    if (!B_KN) {
      const int r = tid >> 2, kq = (tid & 3) * 4;
      Bs[kq][r] = rb.x; Bs[kq + 1][r] = rb.y; Bs[kq + 2][r] = rb.z; Bs[kq + 3][r] = rb.w;
    } else {
      *reinterpret_cast<float4*>(&Bs[tid >> 4][(tid & 15) * 4]) = rb;
    }
    __syncthreads();
    if (k0 + GM_BK < K) fetch(k0 + GM_BK);
#pragma unroll
    for (int kk = 0; kk < GM_BK; ++kk) {
      float av[RM];
      if constexpr (RM == 8) {
        const float4 a0 = *reinterpret_cast<const float4*>(&As[kk][ty * 8]);
        const float4 a1 = *reinterpret_cast<const float4*>(&As[kk][ty * 8 + 4]);
        av[0] = a0.x; av[1] = a0.y; av[2] = a0.z; av[3] = a0.w;
        av[RM - 4] = a1.x; av[RM - 3] = a1.y; av[RM - 2] = a1.z; av[RM - 1] = a1.w;
      } else {
#pragma unroll
        for (int i = 0; i < RM; ++i) av[i] = As[kk][ty * RM + i];
      }
      const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < RM; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < RM; ++i) {
    const int m = m0 + ty * RM + i;
    if (m >= M) break;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) break;
      float v = acc[i][j];
      if (EPI == GM_BIAS_RELU) v = fmaxf(v + __ldg(bias + n), 0.f);
      else if (EPI == GM_BIAS) v = v + __ldg(bias + n);
      else v = __ldg(mask + (size_t)m * ldm + n) > 0.f ? v : 0.f;
      C[(size_t)m * ldc + n] = v;
    }
  }
}

template <bool B_KN, int EPI, int BM>
__global__ void __launch_bounds__(GM_THREADS) sg_gemm_kernel(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
                                                             float* __restrict__ C, int ldc, int M, int N, int K,
                                                             const float* __restrict__ bias, const float* __restrict__ mask, int ldm) {
  sg_gemm_body<B_KN, EPI, BM>(A, lda, B, ldb, C, ldc, M, N, K, bias, mask, ldm);
}

// the same product for two operand sets of one shape in one launch (the two networks' heads): blockIdx.z picks the set
struct GemmPair { const float* A[2]; const float* B[2]; float* C[2]; const float* bias[2]; };
template <bool B_KN, int EPI, int BM>
__global__ void __launch_bounds__(GM_THREADS) sg_gemm_pair_kernel(const GemmPair pr, int lda, int ldb, int ldc, int M, int N, int K) {
  const int z = blockIdx.z;
  sg_gemm_body<B_KN, EPI, BM>(pr.A[z], lda, pr.B[z], ldb, pr.C[z], ldc, M, N, K, pr.bias[z], nullptr, 0);
}

// The heads of both networks for wide hidden layers: out[row][a] = bias[a] + sum_k h[row][k] W[a][k], a < A <= 16, H a
// multiple of 128.  A 32-row FMA tile pads the few outputs to 64 columns and pays a block barrier per 16 k; here a warp takes
// a row at a time: lane l reads the 16-byte pieces l, l + 32, ... of the row (coalesced), multiplies them with the head's
// weights (in shared memory, laid out so that consecutive lanes read consecutive 16-byte words) into 16 partial outputs, and
// the 16 x 32 partials are summed by a fixed halving exchange (16 shuffles).  blockIdx.y picks the network.
constexpr int HD_ROWS = 64;   // rows per block: eight per warp
__global__ void __launch_bounds__(256) sg_heads_kernel(const GemmPair pr, int n_rows, int H, int A, int ldc) {
  extern __shared__ __align__(16) float4 hd_w[];       // [(j * 4 + kk) * 4 + aq][lane]: W[aq * 4 .. + 3][4 (32 j + lane) + kk]
  const int z = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float* __restrict__ W = pr.B[z];
  const float* __restrict__ hrows = pr.A[z];
  const float* __restrict__ bias = pr.bias[z];
  float* __restrict__ out = pr.C[z];
  const int nj = H / 128;
  for (int i = tid; i < nj * 16 * 32; i += blockDim.x) {
    const int l = i & 31, aq = (i >> 5) & 3, kk = (i >> 7) & 3, j = i >> 9;
    const int k = 4 * (32 * j + l) + kk, a = aq * 4;
    float4 w;
    w.x = a < A ? W[(size_t)a * H + k] : 0.f;
    w.y = a + 1 < A ? W[(size_t)(a + 1) * H + k] : 0.f;
    w.z = a + 2 < A ? W[(size_t)(a + 2) * H + k] : 0.f;
    w.w = a + 3 < A ? W[(size_t)(a + 3) * H + k] : 0.f;
    hd_w[i] = w;
  }
  __syncthreads();
  const int a_mine = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
  const float b_mine = a_mine < A ? bias[a_mine] : 0.f;
  for (int r = warp; r < HD_ROWS; r += 8) {
    const int row = blockIdx.x * HD_ROWS + r;
    if (row >= n_rows) break;
    float v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = 0.f;
    for (int j = 0; j < nj; ++j) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(hrows + (size_t)row * H) + 32 * j + lane);
      const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
#pragma unroll
        for (int aq = 0; aq < 4; ++aq) {
          const float4 w = hd_w[((j * 4 + kk) * 4 + aq) * 32 + lane];
          v[aq * 4] = fmaf(xs[kk], w.x, v[aq * 4]); v[aq * 4 + 1] = fmaf(xs[kk], w.y, v[aq * 4 + 1]);
          v[aq * 4 + 2] = fmaf(xs[kk], w.z, v[aq * 4 + 2]); v[aq * 4 + 3] = fmaf(xs[kk], w.w, v[aq * 4 + 3]);
        }
    }
    // halving exchange: after the step with distance d a lane keeps the half of its values that its bit d selects
#define TJ_HD_STEP(D, CNT)                                                                     \
    {                                                                                             \
      const bool upper = (lane & (D)) != 0;                                                       \
      _Pragma("unroll") for (int i = 0; i < (CNT); ++i) {                                         \
        const float keep = upper ? v[i + (CNT)] : v[i], send = upper ? v[i] : v[i + (CNT)];      \
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, (D));                                   \
      }                                                                                           \
    }
    TJ_HD_STEP(16, 8)
    TJ_HD_STEP(8, 4)
    TJ_HD_STEP(4, 2)
    TJ_HD_STEP(2, 1)
#undef TJ_HD_STEP
    const float total = v[0] + __shfl_xor_sync(0xffffffffu, v[0], 1);
    if ((lane & 1) == 0 && a_mine < A) out[(size_t)row * ldc + a_mine] = total + b_mine;
  }
}

template <bool B_KN, int EPI, int BM = GM_BM>
void sg_gemm(const float* A, int lda, const float* B, int ldb, float* C, int ldc, int M, int N, int K, const float* bias,
             const float* mask, int ldm, cudaStream_t s) {
  sg_gemm_kernel<B_KN, EPI, BM><<<dim3((N + GM_BN - 1) / GM_BN, (M + BM - 1) / BM), GM_THREADS, 0, s>>>(A, lda, B, ldb, C, ldc, M, N, K,
                                                                                                     bias, mask, ldm);
}

// ---------------------------------------------------------------------------------------------------------------------
// The same product on the tensor cores, FP32-faithful: every operand is split into a TF32 high part (the top 19 bits) and
// the remainder, and C accumulates A_hi B_hi + A_lo B_hi + A_hi B_lo in FP32 (the dropped A_lo B_lo term is 2^-22 of the
// product, and the tensor core reads each remainder with 11 significant bits: another 2^-22 each).  A: M x K row-major, B: N x K row-major (a weight matrix as the forward pass uses it), K a multiple of 4, rows
// 16-byte aligned.  One 128 x 128 tile per block, accumulator in tensor memory (128 columns); per step of 16 k the
// threads split the step's operands into one of two shared-memory stages (K-major core matrices of 8 rows x 16 bytes)
// while the tensor core works on the other, and the operands of the following TG_PF steps are on their way from global
// memory to registers.  65 KB of shared memory: two blocks per SM cover each other's waits.
constexpr int TG_M = 128, TG_N = 128, TG_K = 16, TG_THREADS = 256, TG_PF = 3;
constexpr int TG_OPER_BYTES = TG_M * TG_K * 4;            // one operand part of one stage: 8 KB
constexpr int TG_STAGE_BYTES = 4 * TG_OPER_BYTES;         // A_hi | A_lo | B_hi | B_lo
constexpr int TG_SMEM_BYTES = 2 * TG_STAGE_BYTES + 1024;  // + alignment slack

template <int EPI>
__global__ void __launch_bounds__(TG_THREADS, 2) sg_gemm_tc_kernel(const float* __restrict__ A, int lda, const float* __restrict__ B,
                                                                   int ldb, float* __restrict__ C, int ldc, int M, int N, int K,
                                                                   const float* __restrict__ bias, const float* __restrict__ mask,
                                                                   int ldm, unsigned long long* __restrict__ error) {
  extern __shared__ uint8_t tg_raw[];
  uint8_t* stage0 = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tg_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t done[2];
  __shared__ uint32_t tmem_base;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m0 = blockIdx.y * TG_M, n0 = blockIdx.x * TG_N;
  if (tid == 0) {
    mbar_init(&done[0], 1);
    mbar_init(&done[1], 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_base)), "r"(128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base;

  // loader mapping: a warp instruction covers eight rows x four 16-byte pieces (64 contiguous bytes per row); warp w
  // owns rows 16 w .. 16 w + 15 of both operands' tiles, a thread two pieces of each
  static_assert(TG_K == 16, "the loader maps four 16-byte pieces to a row");
  const int r8 = lane >> 2, kq = lane & 3;
  // TG_PF register sets: the operands of the next TG_PF steps are in flight from global memory at any time
  float4 ra[TG_PF][2], rb[TG_PF][2];
  auto fetch = [&](int k0, float4 (&fa)[2], float4 (&fb)[2]) {
    const int k = k0 + kq * 4;
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      const int rr = warp * 16 + g * 8 + r8;
      fa[g] = (m0 + rr < M && k < K) ? __ldg(reinterpret_cast<const float4*>(A + (size_t)(m0 + rr) * lda + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
      fb[g] = (n0 + rr < N && k < K) ? __ldg(reinterpret_cast<const float4*>(B + (size_t)(n0 + rr) * ldb + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto split_store = [](uint8_t* hi_dst, uint8_t* lo_dst, const float4 v) {
    float4 hi, lo;
    hi.x = __uint_as_float(__float_as_uint(v.x) & 0xFFFFE000u); lo.x = v.x - hi.x;
    hi.y = __uint_as_float(__float_as_uint(v.y) & 0xFFFFE000u); lo.y = v.y - hi.y;
    hi.z = __uint_as_float(__float_as_uint(v.z) & 0xFFFFE000u); lo.z = v.z - hi.z;
    hi.w = __uint_as_float(__float_as_uint(v.w) & 0xFFFFE000u); lo.w = v.w - hi.w;
    *reinterpret_cast<float4*>(hi_dst) = hi;
    *reinterpret_cast<float4*>(lo_dst) = lo;
  };
  const int nk = (K + TG_K - 1) / TG_K;
  const uint32_t idesc = make_idesc_tf32(TG_N);
  constexpr uint32_t SBO = (TG_K / 4) * 128u;     // eight rows further: one row group of K/4 core matrices
  bool ok = true;
  // one step: registers -> split -> stage i & 1, the tensor core's products on it, the load of step i + TG_PF.  Returns
  // false (for every thread alike) when a wait ran out.
  auto step = [&](int i, float4 (&fa)[2], float4 (&fb)[2]) -> bool {
    const int s = i & 1;
    uint8_t* st = stage0 + (size_t)s * TG_STAGE_BYTES;
    // the tensor core must be done with this stage (its use two steps ago).  One warp polls the barrier, the others
    // sleep at the block barrier: polls from every warp would take shared-memory cycles from the tensor core, whose
    // TF32 operand reads (8 KB per instruction) already need most of them
    if (i >= 2) {
      if (warp == 1) ok = tc_wait_elect(&done[s], (uint32_t)(((i >> 1) - 1) & 1), &abort_flag);
      if (__syncthreads_or(!ok)) return false;
    }
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      const int rr = warp * 16 + g * 8 + r8;
      const size_t off = (size_t)(rr >> 3) * SBO + (size_t)(rr & 7) * 16 + (size_t)kq * 128;
      split_store(st + off, st + TG_OPER_BYTES + off, fa[g]);
      split_store(st + 2 * TG_OPER_BYTES + off, st + 3 * TG_OPER_BYTES + off, fb[g]);
    }
    fence_async_smem();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t a_hi = smem_addr(st), a_lo = a_hi + TG_OPER_BYTES, b_hi = a_hi + 2 * TG_OPER_BYTES, b_lo = a_hi + 3 * TG_OPER_BYTES;
#pragma unroll
      for (int j = 0; j < TG_K / 8; ++j) {
        const uint32_t o = (uint32_t)j * 256u;
        umma_tf32(tmem, make_desc(a_hi + o, 128u, SBO), make_desc(b_hi + o, 128u, SBO), idesc, (i | j) != 0);
        umma_tf32(tmem, make_desc(a_lo + o, 128u, SBO), make_desc(b_hi + o, 128u, SBO), idesc, true);
        umma_tf32(tmem, make_desc(a_hi + o, 128u, SBO), make_desc(b_lo + o, 128u, SBO), idesc, true);
      }
      umma_commit(&done[s]);
    }
    if (i + TG_PF < nk) fetch((i + TG_PF) * TG_K, fa, fb);
    return true;
  };
#pragma unroll
  for (int pf = 0; pf < TG_PF; ++pf)
    if (pf < nk) fetch(pf * TG_K, ra[pf], rb[pf]);
  bool running = true;
  for (int i = 0; i < nk && running; i += TG_PF) {
#pragma unroll
    for (int pf = 0; pf < TG_PF; ++pf)
      if (running && i + pf < nk) running = step(i + pf, ra[pf], rb[pf]);
  }
  // every product is complete once the last commit has arrived (a commit covers all earlier ones of its thread)
  if (running && warp == 1) ok = tc_wait_elect(&done[(nk - 1) & 1], (uint32_t)(((nk - 1) >> 1) & 1), &abort_flag);
  ok = !__syncthreads_or(!ok || !running);
  if (ok) {
    tc_fence_after();
    const int q = warp & 3, hsel = warp >> 2;      // TMEM lane quarter of this warp, column half
    const int m = m0 + q * 32 + lane;
    const uint32_t t_acc = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(hsel * 64);
    uint32_t v[64];
#pragma unroll
    for (int g = 0; g < 4; ++g) tmem_ld16(t_acc + (uint32_t)(g * 16), v + 16 * g);
    tmem_ld_wait();
    if (m < M) {
      const bool vec = (ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(C) & 15) == 0;
#pragma unroll
      for (int c4 = 0; c4 < 16; ++c4) {
        const int n = n0 + hsel * 64 + c4 * 4;
        if (n >= N) break;
        float o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float x = __uint_as_float(v[c4 * 4 + j]);
          if (n + j < N) {
            if (EPI == GM_BIAS_RELU) x = fmaxf(x + __ldg(bias + n + j), 0.f);
            else if (EPI == GM_BIAS) x = x + __ldg(bias + n + j);
            else x = __ldg(mask + (size_t)m * ldm + n + j) > 0.f ? x : 0.f;
          }
          o[j] = x;
        }
        float* dst = C + (size_t)m * ldc + n;
        if (vec && n + 3 < N) {
          *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[1], o[2], o[3]);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (n + j < N) dst[j] = o[j];
        }
      }
    }
  } else if (tid == 0) {
    atomicExch(error, 3ull);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128u) : "memory");
}

// dst[c][r] = src[r][c] for an n x n matrix (32 x 32 tiles through shared memory, both sides coalesced)
__global__ void __launch_bounds__(256) sg_transpose_kernel(const float* __restrict__ src, float* __restrict__ dst, int n) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < 32; i += 8)
    if (r0 + i < n && c0 + tx < n) tile[i][tx] = src[(size_t)(r0 + i) * n + c0 + tx];
  __syncthreads();
  for (int i = ty; i < 32; i += 8)
    if (c0 + i < n && r0 + tx < n) dst[(size_t)(c0 + i) * n + r0 + tx] = tile[tx][i];
}

// shapes the tensor-core product takes: 16-byte rows on both operands and enough 128 x 128 tiles to occupy most SMs (with
// fewer, the 128 x 64 FMA tiles spread the work over more blocks and finish sooner)
static bool tc_gemm_ok(const float* A, int lda, const float* B, int ldb, int M, int N, int K) {
  const long long tiles = (long long)((M + TG_M - 1) / TG_M) * ((N + TG_N - 1) / TG_N);
  return (K & 3) == 0 && (lda & 3) == 0 && (ldb & 3) == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0 &&
         (reinterpret_cast<uintptr_t>(B) & 15) == 0 && K >= 32 && tiles >= 96;
}

// forward-layout product (B is N x K): tensor cores where the shape allows, the FMA tiles otherwise
template <int EPI>
cudaError_t sg_layer(const float* A, int lda, const float* B, int ldb, float* C, int ldc, int M, int N, int K, const float* bias,
                     const float* mask, int ldm, unsigned long long* error, cudaStream_t s) {
  if (tc_gemm_ok(A, lda, B, ldb, M, N, K)) {
    cudaError_t e = cudaFuncSetAttribute(sg_gemm_tc_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, TG_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    sg_gemm_tc_kernel<EPI><<<dim3((N + TG_N - 1) / TG_N, (M + TG_M - 1) / TG_M), TG_THREADS, TG_SMEM_BYTES, s>>>(A, lda, B, ldb, C, ldc, M, N, K,
                                                                                                         bias, mask, ldm, error);
  } else {
    sg_gemm<false, EPI>(A, lda, B, ldb, C, ldc, M, N, K, bias, mask, ldm, s);
  }
  return cudaGetLastError();
}

// TD error, Huber loss and its gradient at the outputs from the two networks' Q values: q (in) and g (out) share p.g
// ([n][A]: a row is read, then overwritten by its own thread), qt [n][A]; loss partials per SG_ROWS rows as in the
// fused forward kernel
__global__ void __launch_bounds__(32) sgd_loss_kernel(const SgdParams p, const float* __restrict__ qt) {
  __shared__ float hub[SG_ROWS];
  const int r = threadIdx.x, j = blockIdx.x * SG_ROWS + r, A = p.A;
  if (r < SG_ROWS) {
    float h = 0.f;
    if (j < p.n) {
      int a = p.act[j];
      a = a < 0 ? 0 : (a >= A ? A - 1 : a);
      float* gr = p.g + (size_t)j * A;
      const float qsel = gr[a];
      const float* tr = qt + (size_t)j * A;
      float qmax = tr[0];
      for (int i = 1; i < A; ++i) qmax = fmaxf(qmax, tr[i]);
      const float y = p.rew[j] + p.gamma * (p.done[j] ? 0.f : 1.f) * qmax;
      const float delta = y - qsel, ad = fabsf(delta);
      h = ad <= p.kappa ? 0.5f * delta * delta : p.kappa * (ad - 0.5f * p.kappa);
      const float gj = -fminf(fmaxf(delta, -p.kappa), p.kappa) / (float)p.n;
      for (int i = 0; i < A; ++i) gr[i] = i == a ? gj : 0.f;
    }
    hub[r] = h;
  }
  __syncwarp();
  if (r == 0) {
    float s = 0.f;
    for (int i = 0; i < SG_ROWS; ++i) s += hub[i];
    p.partial[blockIdx.x] = s;
  }
}

// On-policy forward (PPO): trunk, policy head and value head of the one network; per row the clipped surrogate, the value
// loss and the entropy, and their gradients at the outputs: g[j][0..A) for the logits, g[j][A] for the value.
// shared memory: xs [D][16] | a1 [H][16] | a2 [H][16] | qs [A + 1][16] | weight tile [256][33]
__global__ void __launch_bounds__(SG_THREADS) ppo_forward_kernel(const SgdParams p) {
  extern __shared__ __align__(16) float sg_sm[];
  const int D = p.D, H = p.H, A = p.A;
  float* xs = sg_sm;
  float* a1 = xs + (size_t)D * SG_ROWS;
  float* a2 = a1 + (size_t)H * SG_ROWS;
  float* qs = a2 + (size_t)H * SG_ROWS;
  float* wt = qs + (size_t)(A + 1) * SG_ROWS;
  __shared__ float part[5][SG_ROWS];
  const int row0 = blockIdx.x * SG_ROWS;
  const float *W1 = p.theta, *b1 = W1 + (size_t)H * D, *W2 = b1 + H, *b2 = W2 + (size_t)H * H, *W3 = b2 + H, *b3 = W3 + (size_t)A * H,
              *Wv = b3 + A, *bv = Wv + H;
  for (int i = threadIdx.x; i < D * SG_ROWS; i += SG_THREADS) {
    const int k = i / SG_ROWS, r = i % SG_ROWS;
    xs[i] = row0 + r < p.n ? p.obs[(size_t)(row0 + r) * D + k] : 0.f;
  }
  __syncthreads();
  sg_dense<true>(W1, b1, H, D, xs, a1, wt);
  __syncthreads();
  sg_dense<true>(W2, b2, H, H, a1, a2, wt);
  __syncthreads();
  sg_dense<false>(W3, b3, A, H, a2, qs, wt);
  sg_dense<false>(Wv, bv, 1, H, a2, qs + (size_t)A * SG_ROWS, wt);
  for (int i = threadIdx.x; i < H * SG_ROWS; i += SG_THREADS) {
    const int k = i / SG_ROWS, r = i % SG_ROWS;
    if (row0 + r < p.n) {
      p.h1[(size_t)(row0 + r) * H + k] = a1[i];
      p.h2[(size_t)(row0 + r) * H + k] = a2[i];
    }
  }
  __syncthreads();
  if (threadIdx.x < SG_ROWS) {
    const int r = threadIdx.x, j = row0 + r;
    float l_tot = 0.f, l_pi = 0.f, l_v = 0.f, l_h = 0.f, l_c = 0.f;
    if (j < p.n) {
      int a = p.act[j];
      a = a < 0 ? 0 : (a >= A ? A - 1 : a);
      float lmax = qs[r];
      for (int i = 1; i < A; ++i) lmax = fmaxf(lmax, qs[(size_t)i * SG_ROWS + r]);
      float Z = 0.f;
      for (int i = 0; i < A; ++i) Z += expf(qs[(size_t)i * SG_ROWS + r] - lmax);
      const float logZ = lmax + logf(Z);
      float ent = 0.f;
      for (int i = 0; i < A; ++i) {
        const float lp = qs[(size_t)i * SG_ROWS + r] - logZ;
        ent -= expf(lp) * lp;
      }
      const float logp = qs[(size_t)a * SG_ROWS + r] - logZ;
      const float ratio = expf(logp - p.logp_old[j]), Aj = p.adv[j];
      const float rc = fminf(fmaxf(ratio, 1.f - p.clip_eps), 1.f + p.clip_eps);
      const float t1 = ratio * Aj, t2 = rc * Aj;
      const bool unclipped = t1 <= t2;
      const float val = qs[(size_t)A * SG_ROWS + r], dv = val - p.ret[j];
      l_pi = -(unclipped ? t1 : t2);
      l_c = unclipped ? 0.f : 1.f;
      l_v = 0.5f * dv * dv;
      l_h = ent;
      l_tot = l_pi + p.c_v * l_v - p.c_e * l_h;
      const float g_logp = unclipped ? -Aj * ratio : 0.f, inv_n = 1.f / (float)p.n;
      float* gr = p.g + (size_t)j * p.ldg;
      for (int i = 0; i < A; ++i) {
        const float lp = qs[(size_t)i * SG_ROWS + r] - logZ, pi = expf(lp);
        const float dlogp = (i == a ? 1.f : 0.f) - pi;
        const float dent = -pi * (lp + ent);
        gr[i] = (g_logp * dlogp - p.c_e * dent) * inv_n;
      }
      gr[A] = p.c_v * dv * inv_n;
    }
    part[0][r] = l_tot; part[1][r] = l_pi; part[2][r] = l_v; part[3][r] = l_h; part[4][r] = l_c;
  }
  __syncthreads();
  if (threadIdx.x < 5) {
    float s = 0.f;
    for (int r = 0; r < SG_ROWS; ++r) s += part[threadIdx.x][r];
    p.stat_partial[(size_t)blockIdx.x * 5 + threadIdx.x] = s;
  }
}

// out[k] = (sum over the blocks of partial k) / n, k = 0..4, blocks in ascending order
__global__ void ppo_finish_kernel(const float* __restrict__ stat_partial, int n_blocks, int n, float* __restrict__ out) {
  const int k = threadIdx.x;
  if (k >= 5) return;
  float s = 0.f;
  for (int b = 0; b < n_blocks; ++b) s += stat_partial[(size_t)b * 5 + k];
  out[k] = s / (float)n;
}

// backward through the activations, SG_ROWS rows per block: shared memory d2 [H][16]
__global__ void __launch_bounds__(SG_THREADS) sgd_backward_kernel(const SgdParams p) {
  extern __shared__ __align__(16) float sg_sm[];
  const int D = p.D, H = p.H, A = p.A;
  float* d2 = sg_sm;
  const int row0 = blockIdx.x * SG_ROWS;
  const float* W2 = p.theta + (size_t)H * D + H;
  const float* W3 = W2 + (size_t)H * H + H;
  const float* Wv = W3 + (size_t)A * H + A;
  // dh2[r][i] = sum_a g[r][a] W3[a][i] (+ g[r][A] Wv[i] with the value head) where h2 > 0; for the Q head g has one
  // non-zero entry per row
  for (int idx = threadIdx.x; idx < H * SG_ROWS; idx += SG_THREADS) {
    const int r = idx / H, i = idx % H, j = row0 + r;
    float v = 0.f;
    if (j < p.n && p.h2[(size_t)j * H + i] > 0.f) {
      const float* gr = p.g + (size_t)j * p.ldg;
      for (int a = 0; a < A; ++a) v = fmaf(gr[a], W3[(size_t)a * H + i], v);
      if (p.value_head) v = fmaf(gr[A], Wv[i], v);
    }
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


// One gradient product of the update: C (M x N, at float offset `off` of the parameter blob) gets (Am rows)^T (Bm rows),
// a bias (Bm == nullptr) a column of ones.  Tiles of all products are numbered in one list: tile_begin is this product's
// first tile.
struct GradProduct {
  const float* Am;
  const float* Bm;
  int off, M, N, lda, ldb, tile_begin;
};
struct GradProducts {
  GradProduct g[8];
  int n, n_tiles;
};

constexpr int GP_TILE = 64, GP_ROWS = 16;   // columns of a gradient tile; minibatch rows staged per step

// One tile (TM x 64, TM = 64 or 128: each thread TM / 16 x 4) of one gradient product over one range of minibatch rows
template <int TM>
__device__ __forceinline__ void grad_tile(float* __restrict__ P, const GradProduct& d, int t, int count, int n_rows, int rows_per_range,
                                          float (*As)[128 + 4], float (*Bs)[GP_TILE + 4]) {
  constexpr int RM = TM / 16, NA = TM / 64;
  const int M = d.M, N = d.N, lda = d.lda, ldb = d.ldb;
  const float* __restrict__ Am = d.Am;
  const float* __restrict__ Bm = d.Bm;
  const int tiles_n = (N + GP_TILE - 1) / GP_TILE;
  const int m0 = (t / tiles_n) * TM, n0 = (t % tiles_n) * GP_TILE;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int j_begin = blockIdx.y * rows_per_range;
  const int j_end = j_begin + rows_per_range < n_rows ? j_begin + rows_per_range : n_rows;
  const bool vecA = (lda & 3) == 0 && (reinterpret_cast<uintptr_t>(Am) & 15) == 0;
  const bool vecB = Bm && (ldb & 3) == 0 && (reinterpret_cast<uintptr_t>(Bm) & 15) == 0;
  // four consecutive columns of row j (zero beyond the row range or the matrix): a 16-byte load where the row allows it
  auto load_c4 = [](const float* base, int ld, int j, int j_end, int c, int C, bool vec) -> float4 {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < j_end && c < C) {
      const float* src = base + (size_t)j * ld + c;
      if (vec && c + 3 < C) {
        v = *reinterpret_cast<const float4*>(src);
      } else {
        v.x = src[0];
        if (c + 1 < C) v.y = src[1];
        if (c + 2 < C) v.z = src[2];
        if (c + 3 < C) v.w = src[3];
      }
    }
    return v;
  };
  float acc[RM][4];
#pragma unroll
  for (int u = 0; u < RM; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) acc[u][v] = 0.f;
  // the next rows travel from global memory to registers while these are multiplied
  const int l_jj = threadIdx.x >> 4, l_c = (threadIdx.x & 15) * 4;
  float4 ra[NA], rb;
  auto fetch = [&](int j0) {
    const int j = j0 + l_jj;
#pragma unroll
    for (int h = 0; h < NA; ++h) ra[h] = load_c4(Am, lda, j, j_end, m0 + h * 64 + l_c, M, vecA);
    if (Bm) {
      rb = load_c4(Bm, ldb, j, j_end, n0 + l_c, N, vecB);
    } else {
      const float one = j < j_end ? 1.f : 0.f;
      rb = make_float4(n0 + l_c < N ? one : 0.f, n0 + l_c + 1 < N ? one : 0.f, n0 + l_c + 2 < N ? one : 0.f, n0 + l_c + 3 < N ? one : 0.f);
    }
  };
  if (j_begin < j_end) fetch(j_begin);
  for (int j0 = j_begin; j0 < j_end; j0 += GP_ROWS) {
#pragma unroll
    for (int h = 0; h < NA; ++h) *reinterpret_cast<float4*>(&As[l_jj][h * 64 + l_c]) = ra[h];
    *reinterpret_cast<float4*>(&Bs[l_jj][l_c]) = rb;
    __syncthreads();
    if (j0 + GP_ROWS < j_end) fetch(j0 + GP_ROWS);
#pragma unroll
    for (int jj = 0; jj < GP_ROWS; ++jj) {
      float av[RM];
#pragma unroll
      for (int h = 0; h < RM / 4; ++h) {
        const float4 a = *reinterpret_cast<const float4*>(&As[jj][ty * RM + h * 4]);
        av[h * 4] = a.x; av[h * 4 + 1] = a.y; av[h * 4 + 2] = a.z; av[h * 4 + 3] = a.w;
      }
      const float4 b = *reinterpret_cast<const float4*>(&Bs[jj][tx * 4]);
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int u = 0; u < RM; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(av[u], bv[v], acc[u][v]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < RM; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int m = m0 + ty * RM + u, n = n0 + tx * 4 + v;
      if (m < M && n < N) P[(size_t)blockIdx.y * count + d.off + (size_t)m * N + n] = acc[u][v];
    }
}

// Every gradient product of one update in a single launch: thread block (tile, range) sums, over its range of minibatch
// rows, one tile of one product (128 x 64 where the product has at least 128 rows, else 64 x 64) and writes it to
// P[range][off + m * N + n] -- a partial gradient laid out like the parameter blob itself, `count` floats per range.
// No atomics: the apply kernel adds the ranges in order.
__global__ void __launch_bounds__(256) sgd_grad_partial_kernel(float* __restrict__ P, const GradProducts gp, int count, int n_rows,
                                                               int rows_per_range) {
  __shared__ __align__(16) float As[GP_ROWS][128 + 4], Bs[GP_ROWS][GP_TILE + 4];
  int q = 0;
  while (q + 1 < gp.n && (int)blockIdx.x >= gp.g[q + 1].tile_begin) ++q;
  const GradProduct& d = gp.g[q];
  const int t = blockIdx.x - d.tile_begin;
  if (d.M >= 128) grad_tile<128>(P, d, t, count, n_rows, rows_per_range, As, Bs);
  else grad_tile<64>(P, d, t, count, n_rows, rows_per_range, As, Bs);
}

// C[i] -= lr * (P[0][i] + P[1][i] + ...), the partial sums added in range order
__global__ void sgd_apply_kernel(float* __restrict__ Cm, const float* __restrict__ P, int count, int n_ranges, float lr) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float s = 0.f;
  for (int z = 0; z < n_ranges; ++z) s += P[(size_t)z * count + i];
  Cm[i] -= lr * s;
}

// the same gradient through Adam (Table 2's optimiser): m <- b1 m + (1-b1) g, v <- b2 v + (1-b2) g^2,
// theta <- theta - lr (m / c1) / (sqrt(v / c2) + eps) with the bias corrections c1 = 1 - b1^t, c2 = 1 - b2^t from the host
__global__ void sgd_apply_adam_kernel(float* __restrict__ Cm, float* __restrict__ m, float* __restrict__ v,
                                      const float* __restrict__ P, int count, int n_ranges, float lr, float beta1, float beta2,
                                      float eps, float c1, float c2) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float g = 0.f;
  for (int z = 0; z < n_ranges; ++z) g += P[(size_t)z * count + i];
  const float mi = fmaf(beta1, m[i], (1.f - beta1) * g);
  const float vi = fmaf(beta2, v[i], (1.f - beta2) * g * g);
  m[i] = mi;
  v[i] = vi;
  Cm[i] -= lr * (mi / c1) / (sqrtf(vi / c2) + eps);
}

}  // namespace

size_t sgd_scratch_floats(int max_rows, int D, int H) {
  const size_t rows = ((size_t)max_rows + SG_ROWS - 1) / SG_ROWS * SG_ROWS;
  // h1, h2, dh1, dh2, g [rows][<= 16 actions + value], loss partials (1 + 5 per 16 rows), and per row range one partial
  // gradient of the whole parameter blob (at most 16 actions and a value head); W2 transposed
  const size_t blob = (size_t)H * D + H + (size_t)H * H + H + 17 * (size_t)H + 17;
  // + split copies of W1 (x 2 networks), W2 (x 2) and W2^T for the tensor-core products
  return 4 * rows * (size_t)H + rows * 17 + 6 * (rows / SG_ROWS) + 64 + (size_t)H * H + (size_t)SG_SPLITS * blob +
         2 * tc_pack_floats(H, D) + 3 * tc_pack_floats(H, H) + 64;
}

int sgd_partial_count(int n) { return (n + SG_ROWS - 1) / SG_ROWS; }

bool sgd_supported(int D, int H, int A) {
  const size_t smem = (((size_t)D + 2 * (size_t)H + A) * SG_ROWS + (size_t)SG_THREADS * (SG_KT + 1)) * sizeof(float);
  return H >= 1 && D >= 1 && A >= 1 && A <= 16 && smem <= 200 * 1024;
}

namespace {
// the tiled path pays off once a layer is a real matrix product; below that the fused per-16-rows kernels launch less
bool use_tiled(const SgdParams& p) { return !p.value_head && p.H >= 128 && p.n >= 512; }
// wide layers with enough 128 x 256 tiles: the pre-split tensor-core products (both hidden layers must qualify)
bool use_tc2(const SgdParams& p) {
  return use_tiled(p) && p.wpack && tc_gemm2_ok(p.obs, p.D, p.n, p.H, p.D) && tc_gemm2_ok(p.next_obs, p.D, p.n, p.H, p.D) &&
         tc_gemm2_ok(p.h1, p.H, p.n, p.H, p.H);
}

// the backward pass and every parameter update: C -= lr * (gradient rows)^T (input rows), a bias with a column of ones
cudaError_t backward_and_update(const SgdParams& p, float lr, const AdamParams* adam, cudaStream_t s) {
  const int D = p.D, H = p.H, A = p.A;
  const int grid = sgd_partial_count(p.n);
  const size_t smem_b = (size_t)H * SG_ROWS * sizeof(float);
  cudaError_t e;
  if (use_tiled(p)) {
    // dh2 = (g W3) where h2 > 0; dh1 = (dh2 W2) where h1 > 0
    const float* W2m = p.theta + (size_t)H * D + H;
    const float* W3m = W2m + (size_t)H * H + H;
    sg_gemm<true, GM_MASK>(p.g, p.ldg, W3m, H, p.dh2, H, p.n, H, A, nullptr, p.h2, H, s);
    if (use_tc2(p)) {
      // W2^T was split with the other weight matrices at the start of the step
      TcGemmBatch b{};
      b.g[0] = TcGemm{p.dh2, H, p.wpack + 2 * tc_pack_floats(H, D) + 2 * tc_pack_floats(H, H), p.dh1, H, p.n, H, H, nullptr, p.h1, H};
      b.n = 1;
      if ((e = launch_gemm_tc2(b, GM_MASK, p.error, s)) != cudaSuccess) return e;
    } else if (tc_gemm_ok(p.dh2, H, p.w2t, H, p.n, H, H)) {
      // the tensor-core product wants both operands K-major: dh1 = dh2 (W2^T)^T with W2^T written out first
      sg_transpose_kernel<<<dim3((H + 31) / 32, (H + 31) / 32), 256, 0, s>>>(W2m, p.w2t, H);
      if ((e = sg_layer<GM_MASK>(p.dh2, H, p.w2t, H, p.dh1, H, p.n, H, H, nullptr, p.h1, H, p.error, s)) != cudaSuccess) return e;
    } else {
      sg_gemm<true, GM_MASK>(p.dh2, H, W2m, H, p.dh1, H, p.n, H, H, nullptr, p.h1, H, s);
    }
  } else {
    if ((e = cudaFuncSetAttribute(sgd_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_b)) != cudaSuccess) return e;
    sgd_backward_kernel<<<grid, SG_THREADS, smem_b, s>>>(p);
  }
  float* W1 = p.theta;
  float* b1 = W1 + (size_t)H * D;
  float* W2 = b1 + H;
  float* b2 = W2 + (size_t)H * H;
  float* W3 = b2 + H;
  float* b3 = W3 + (size_t)A * H;
  float* Wv = b3 + A;
  float* bv = Wv + H;
  // the backward pass has read W2 and the heads; now the parameters may change: all products in one or two launches, then
  // one pass over the whole blob.  Products whose input width is a multiple of 128 go to the tensor cores (with their bias
  // gradient), the others to the FMA tiles.
  GradProducts gp{};
  auto add = [&](float* C, int M, int N, const float* Am, int lda, const float* Bm, int ldb) {
    GradProduct& d = gp.g[gp.n++];
    d.Am = Am;
    d.Bm = Bm;
    d.off = (int)(C - p.theta);
    d.M = M;
    d.N = N;
    d.lda = lda;
    d.ldb = ldb;
    d.tile_begin = gp.n_tiles;
    const int tm = M >= 128 ? 128 : 64;   // as the kernel picks it
    gp.n_tiles += ((M + tm - 1) / tm) * ((N + GP_TILE - 1) / GP_TILE);
  };
  TcWgradBatch tb{};
  const bool tc_grads = use_tc2(p);
  // one product and its bias: C [M][N] = G^T X, bias [M] = column sums of G
  auto product = [&](float* C, float* bias, int M, int N, const float* G, int ldg, const float* X, int ldx) {
    if (tc_grads && tc_wgrad_ok(N, p.n)) {
      TcWgrad& d = tb.g[tb.n++];
      d = TcWgrad{G, ldg, X, ldx, M, N, (int)(C - p.theta), (int)(bias - p.theta), tb.n_tiles};
      tb.n_tiles += tc_wgrad_tiles(M, N);
    } else {
      add(C, M, N, G, ldg, X, ldx);
      add(bias, M, 1, G, ldg, nullptr, 0);
    }
  };
  product(W1, b1, H, D, p.dh1, H, p.obs, D);
  product(W2, b2, H, H, p.dh2, H, p.h1, H);
  product(W3, b3, A, H, p.g, p.ldg, p.h2, H);
  if (p.value_head) product(Wv, bv, 1, H, p.g + A, p.ldg, p.h2, H);
  // row ranges: with tensor-core tiles about one thread block per SM in all (a block costs a fixed ~10 us beside its rows);
  // otherwise 128 rows or more per range
  int n_ranges;
  if (tb.n_tiles > 0) {
    n_ranges = (p.sm_count > 0 ? p.sm_count : 148) / tb.n_tiles;
    if (n_ranges < 1) n_ranges = 1;
  } else {
    n_ranges = (p.n + 127) / 128;
  }
  if (n_ranges > SG_SPLITS) n_ranges = SG_SPLITS;
  const int rows_per_range = ((p.n + n_ranges - 1) / n_ranges + 31) / 32 * 32;
  n_ranges = (p.n + rows_per_range - 1) / rows_per_range;
  const int count = (int)((p.value_head ? bv + 1 : b3 + A) - p.theta);
  if (tb.n && (e = launch_wgrad_tc(tb, p.grad_partial, count, p.n, rows_per_range, n_ranges, p.error, s)) != cudaSuccess) return e;
  if (gp.n_tiles > 0) sgd_grad_partial_kernel<<<dim3(gp.n_tiles, n_ranges), 256, 0, s>>>(p.grad_partial, gp, count, p.n, rows_per_range);
  if (adam)
    sgd_apply_adam_kernel<<<(count + 255) / 256, 256, 0, s>>>(p.theta, adam->m, adam->v, p.grad_partial, count, n_ranges, lr, adam->beta1,
                                                              adam->beta2, adam->eps, adam->c1, adam->c2);
  else
    sgd_apply_kernel<<<(count + 255) / 256, 256, 0, s>>>(p.theta, p.grad_partial, count, n_ranges, lr);
  return cudaGetLastError();
}
}  // namespace

// launches of the backward pass and the update: dh2 and dh1 (with W2's transpose on the tensor-core path) or the fused
// backward kernel, the grouped gradient products, the apply pass
static int backward_launches(const SgdParams& p) {
  if (!use_tiled(p)) return 3;
  if (use_tc2(p)) return 2 + 2 + (tc_wgrad_ok(p.D, p.n) ? 0 : 1);   // hidden-width products always qualify; W1's by obs_dim
  return (tc_gemm_ok(p.dh2, p.H, p.w2t, p.H, p.n, p.H, p.H) ? 3 : 2) + 2;
}

int sgd_step_launches(const SgdParams& p) { return (use_tiled(p) ? (use_tc2(p) ? 5 : 7) : 1) + backward_launches(p); }

int ppo_step_launches(const SgdParams& p, bool with_stats) { return 1 + (with_stats ? 1 : 0) + backward_launches(p); }

cudaError_t launch_sgd_step(const SgdParams& p, float lr, const AdamParams* adam, cudaStream_t s) {
  if (use_tiled(p)) {
    const int n = p.n, D = p.D, H = p.H, A = p.A;
    const float *W1 = p.theta, *b1 = W1 + (size_t)H * D, *W2 = b1 + H, *b2 = W2 + (size_t)H * H, *W3 = b2 + H, *b3 = W3 + (size_t)A * H;
    const float *T1 = p.theta_target, *tb1 = T1 + (size_t)H * D, *T2 = tb1 + H, *tb2 = T2 + (size_t)H * H, *T3 = tb2 + H,
                *tb3 = T3 + (size_t)A * H;
    // online network: h1, h2 kept, Q values into g; target network: its activations borrow dh1 / dh2 (free until the
    // backward pass), its Q values then take dh1's place
    cudaError_t e;
    if (use_tc2(p)) {
      // both networks' weight matrices (and W2^T for the backward pass) split once, then each layer of both networks in one launch
      float* pk_W1 = p.wpack;
      float* pk_T1 = pk_W1 + tc_pack_floats(H, D);
      float* pk_W2 = pk_T1 + tc_pack_floats(H, D);
      float* pk_T2 = pk_W2 + tc_pack_floats(H, H);
      float* pk_W2t = pk_T2 + tc_pack_floats(H, H);
      TcPackJobs jobs{};
      jobs.j[jobs.n++] = TcPackJob{W1, D, 0, H, D, pk_W1};
      jobs.j[jobs.n++] = TcPackJob{T1, D, 0, H, D, pk_T1};
      jobs.j[jobs.n++] = TcPackJob{W2, H, 0, H, H, pk_W2};
      jobs.j[jobs.n++] = TcPackJob{T2, H, 0, H, H, pk_T2};
      jobs.j[jobs.n++] = TcPackJob{W2, H, 1, H, H, pk_W2t};
      if ((e = launch_pack_tf32_operands(jobs, s)) != cudaSuccess) return e;
      TcGemmBatch l1{};
      l1.g[0] = TcGemm{p.obs, D, pk_W1, p.h1, H, n, H, D, b1, nullptr, 0};
      l1.g[1] = TcGemm{p.next_obs, D, pk_T1, p.dh1, H, n, H, D, tb1, nullptr, 0};
      l1.n = 2;
      if ((e = launch_gemm_tc2(l1, GM_BIAS_RELU, p.error, s)) != cudaSuccess) return e;
      TcGemmBatch l2{};
      l2.g[0] = TcGemm{p.h1, H, pk_W2, p.h2, H, n, H, H, b2, nullptr, 0};
      l2.g[1] = TcGemm{p.dh1, H, pk_T2, p.dh2, H, n, H, H, tb2, nullptr, 0};
      l2.n = 2;
      if ((e = launch_gemm_tc2(l2, GM_BIAS_RELU, p.error, s)) != cudaSuccess) return e;
      // both heads in one launch: Q of the online network into g, of the target network into dh1's place
      GemmPair heads{{p.h2, p.dh2}, {W3, T3}, {p.g, p.dh1}, {b3, tb3}};
      const size_t hd_smem = (size_t)H * 16 * sizeof(float);
      if (H % 128 == 0 && A <= 16 && hd_smem <= 96 * 1024) {
        if ((e = cudaFuncSetAttribute(sg_heads_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hd_smem)) != cudaSuccess) return e;
        sg_heads_kernel<<<dim3((n + HD_ROWS - 1) / HD_ROWS, 2), 256, hd_smem, s>>>(heads, n, H, A, A);
      } else {
        sg_gemm_pair_kernel<false, GM_BIAS, 32><<<dim3((A + GM_BN - 1) / GM_BN, (n + 31) / 32, 2), GM_THREADS, 0, s>>>(heads, H, H, A, n, A, H);
      }
    } else {
      if ((e = sg_layer<GM_BIAS_RELU>(p.obs, D, W1, D, p.h1, H, n, H, D, b1, nullptr, 0, p.error, s)) != cudaSuccess) return e;
      if ((e = sg_layer<GM_BIAS_RELU>(p.h1, H, W2, H, p.h2, H, n, H, H, b2, nullptr, 0, p.error, s)) != cudaSuccess) return e;
      sg_gemm<false, GM_BIAS, 32>(p.h2, H, W3, H, p.g, A, n, A, H, b3, nullptr, 0, s);
      if ((e = sg_layer<GM_BIAS_RELU>(p.next_obs, D, T1, D, p.dh1, H, n, H, D, tb1, nullptr, 0, p.error, s)) != cudaSuccess) return e;
      if ((e = sg_layer<GM_BIAS_RELU>(p.dh1, H, T2, H, p.dh2, H, n, H, H, tb2, nullptr, 0, p.error, s)) != cudaSuccess) return e;
      sg_gemm<false, GM_BIAS, 32>(p.dh2, H, T3, H, p.dh1, A, n, A, H, tb3, nullptr, 0, s);
    }
    sgd_loss_kernel<<<sgd_partial_count(n), 32, 0, s>>>(p, p.dh1);
    return backward_and_update(p, lr, adam, s);
  }
  const size_t smem_f = (((size_t)p.D + 2 * (size_t)p.H + p.A) * SG_ROWS + (size_t)SG_THREADS * (SG_KT + 1)) * sizeof(float);
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(sgd_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_f)) != cudaSuccess) return e;
  sgd_forward_kernel<<<sgd_partial_count(p.n), SG_THREADS, smem_f, s>>>(p);
  return backward_and_update(p, lr, adam, s);
}

cudaError_t launch_ppo_step(const SgdParams& p, float lr, const AdamParams* adam, float* stats_out, cudaStream_t s) {
  const size_t smem_f = (((size_t)p.D + 2 * (size_t)p.H + p.A + 1) * SG_ROWS + (size_t)SG_THREADS * (SG_KT + 1)) * sizeof(float);
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(ppo_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_f)) != cudaSuccess) return e;
  ppo_forward_kernel<<<sgd_partial_count(p.n), SG_THREADS, smem_f, s>>>(p);
  if (stats_out) ppo_finish_kernel<<<1, 32, 0, s>>>(p.stat_partial, sgd_partial_count(p.n), p.n, stats_out);
  return backward_and_update(p, lr, adam, s);
}

}  // namespace tj
