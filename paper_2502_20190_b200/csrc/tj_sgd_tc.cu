// FP32-faithful matrix products of the learner update on the tensor cores (Algorithm 1, update line: the forward layers of
// both networks and the backward pass's dh1 are dense contractions over 128-512 inputs for thousands of rows).
//
// C[M][N] = epilogue(A[M][K] B[N][K]^T): every operand is split into a TF32 high part (the top 19 bits) and the remainder,
// and C accumulates A_hi B_hi + A_lo B_hi + A_hi B_lo in FP32 in tensor memory (the dropped A_lo B_lo term is 2^-22 of the
// product, and the tensor core reads each remainder with 11 significant bits: another 2^-22 each).
//
// One 128 x 256 tile per thread block, ten warps:
//   eight worker warps bring A from global memory sixteen columns at a time, split it and write the two parts into one of
//     four shared-memory stages (K-major core matrices of 8 rows x 16 bytes), one mbarrier arrival per warp and stage;
//   a copy lane streams B, which `launch_pack_tf32_operands` has split and laid out ONCE per update in exactly the order
//     and layout the tile consumes (32 KB per 16 columns: high part, low part), into a four-slot ring with bulk copies;
//   an issuing lane fires the six MMAs (two K = 8 steps x three products, N = 256) of a chunk as soon as its A stage and
//     B slot are there, and commits free both; nobody else in its warp polls;
//   the workers then drain the accumulator (bias + ReLU, or the backward pass's ReLU mask) to global memory.
// Two problems (the online and the target network's layer) can share a launch: blockIdx.z picks the set.
// Every wait is bounded; a timeout latches the error word, waits for the copies in flight and frees the tensor memory.
#include "tj_internal.h"
#include "tj_tc.cuh"

namespace tj {

namespace {

constexpr int T2_M = 128, T2_N = 256, T2_K = 16;
constexpr int T2_WORKERS = 256, T2_THREADS = T2_WORKERS + 64, T2_PF = 3;
constexpr int T2_ASTAGES = 3, T2_BSLOTS = 4;
constexpr int T2_STG_LD = 36;                              // floats per row of a warp's 32 x 32 staging block (144 bytes)
constexpr int T2_STG_BYTES = (T2_WORKERS / 32) * 32 * T2_STG_LD * 4;   // 36 KB: one block per worker warp
constexpr int T2_A_PART = T2_M * T2_K * 4;                 // 8 KB: one part of an A stage
constexpr int T2_A_STAGE = 2 * T2_A_PART;
constexpr int T2_B_PART = T2_N * T2_K * 4;                 // 16 KB: one part of a B chunk
constexpr int T2_B_SLOT = 2 * T2_B_PART;
constexpr uint32_t T2_SBO = (T2_K / 4) * 128u;             // eight rows further: one row group of K/4 core matrices

struct T2Ctl {
  uint64_t a_ready[T2_ASTAGES], a_free[T2_ASTAGES], b_full[T2_BSLOTS], b_empty[T2_BSLOTS], acc_full;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int T2_SMEM_BYTES = T2_ASTAGES * T2_A_STAGE + T2_BSLOTS * T2_B_SLOT + T2_STG_BYTES + (int)sizeof(T2Ctl) + 1024;

// A thread owns a row of the accumulator, and a row written straight to global memory costs one 16-byte sector per lane and
// store instruction (8,192 separate sectors per 128 x 256 tile: about 24 K cycles).  So every warp passes its 32 rows x 32
// columns through a staging block of its own: lane r writes row r, then lane l reads the 16-byte piece l % 8 of rows
// l / 8 + 4 i, so that one store instruction writes four rows of 128 contiguous bytes.  Only warp-level synchronisation.
__device__ __forceinline__ void stage_rows(float* stg, int lane, const uint32_t (&v)[32]) {
  __syncwarp();                                   // the block's previous readers are done
  float* row = stg + lane * T2_STG_LD;
#pragma unroll
  for (int c4 = 0; c4 < 8; ++c4) *reinterpret_cast<uint4*>(row + c4 * 4) = make_uint4(v[c4 * 4], v[c4 * 4 + 1], v[c4 * 4 + 2], v[c4 * 4 + 3]);
  __syncwarp();
}
__device__ __forceinline__ float4 staged_piece(const float* stg, int lane, int i) {
  return *reinterpret_cast<const float4*>(stg + ((lane >> 3) + 4 * i) * T2_STG_LD + (lane & 7) * 4);
}

__global__ void __launch_bounds__(T2_THREADS, 1) sg_gemm_tc2_kernel(const TcGemmBatch batch, int epi, unsigned long long* __restrict__ error) {
  extern __shared__ uint8_t t2_raw[];
  uint8_t* a_stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(t2_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* b_slots = a_stages + T2_ASTAGES * T2_A_STAGE;
  float* stg_all = reinterpret_cast<float*>(b_slots + T2_BSLOTS * T2_B_SLOT);
  T2Ctl* ctl = reinterpret_cast<T2Ctl*>(b_slots + T2_BSLOTS * T2_B_SLOT + T2_STG_BYTES);
  const TcGemm& g = batch.g[blockIdx.z];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m0 = blockIdx.y * T2_M, n0 = blockIdx.x * T2_N;
  const int M = g.M, N = g.N, K = g.K, lda = g.lda;
  const int nk = K / T2_K;
  // Blocks that share a tile of B walk the K chunks in rotated order, so that they do not all ask L2 for the same 32 KB at
  // the same moment; step i of this block is chunk (i + rot) mod nk.  The order of a block's sums depends on its row tile only.
  const int rot = (int)((blockIdx.y * 5u + blockIdx.z * 3u) % (unsigned)nk);
  if (tid == 0) {
    for (int i = 0; i < T2_ASTAGES; ++i) { mbar_init(&ctl->a_ready[i], T2_WORKERS / 32); mbar_init(&ctl->a_free[i], 1); }
    for (int i = 0; i < T2_BSLOTS; ++i) { mbar_init(&ctl->b_full[i], 1); mbar_init(&ctl->b_empty[i], 1); }
    mbar_init(&ctl->acc_full, 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&ctl->tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  if (tid < T2_WORKERS) {
    // loader mapping: a warp instruction covers eight rows x four 16-byte pieces (64 contiguous bytes per row); warp w
    // owns rows 16 w .. 16 w + 15 of the tile, a thread two pieces
    const float* __restrict__ A = g.A;
    const int r8 = lane >> 2, kq = lane & 3;
    float4 ra[T2_PF][2];
    auto fetch = [&](int i, float4 (&fa)[2]) {
      const int c = i + rot < nk ? i + rot : i + rot - nk;
      const int k = c * T2_K + kq * 4;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rr = warp * 16 + h * 8 + r8;
        fa[h] = (m0 + rr < M) ? __ldg(reinterpret_cast<const float4*>(A + (size_t)(m0 + rr) * lda + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
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
    bool ok = true;
    auto step = [&](int i, float4 (&fa)[2]) {
      const int st = i % T2_ASTAGES;
      uint8_t* base = a_stages + (size_t)st * T2_A_STAGE;
      if (i >= T2_ASTAGES) ok = tc_wait_elect(&ctl->a_free[st], (uint32_t)(((i / T2_ASTAGES) - 1) & 1), abort_flag);
      if (!ok) return;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rr = warp * 16 + h * 8 + r8;
        const size_t off = (size_t)(rr >> 3) * T2_SBO + (size_t)(rr & 7) * 16 + (size_t)kq * 128;
        split_store(base + off, base + T2_A_PART + off, fa[h]);
      }
      fence_async_smem();
      mbar_arrive_warp(&ctl->a_ready[st]);
      if (i + T2_PF < nk) fetch(i + T2_PF, fa);
    };
#pragma unroll
    for (int pf = 0; pf < T2_PF; ++pf)
      if (pf < nk) fetch(pf, ra[pf]);
    for (int i = 0; i < nk && ok; i += T2_PF) {
#pragma unroll
      for (int pf = 0; pf < T2_PF; ++pf)
        if (ok && i + pf < nk) step(i + pf, ra[pf]);
    }
  } else if (warp == T2_WORKERS / 32) {
    if (lane == 0) {
      // descriptors as 32-bit halves: the high word is a constant of the layout, the low word the address in 16-byte units
      const uint32_t idesc = make_idesc_tf32(T2_N), hiword = desc_hi(T2_SBO);
      const uint32_t a0 = desc_lo(smem_addr(a_stages), 128u), b0 = desc_lo(smem_addr(b_slots), 128u);
      for (int i = 0; i < nk; ++i) {
        const int st = i % T2_ASTAGES, sl = i % T2_BSLOTS;
        if (!tc_wait(&ctl->a_ready[st], (uint32_t)((i / T2_ASTAGES) & 1), abort_flag)) break;
        if (!tc_wait(&ctl->b_full[sl], (uint32_t)((i / T2_BSLOTS) & 1), abort_flag)) break;
        tc_fence_after();
        const uint32_t a_hi = a0 + (uint32_t)st * (T2_A_STAGE / 16), a_lo = a_hi + T2_A_PART / 16;
        const uint32_t b_hi = b0 + (uint32_t)sl * (T2_B_SLOT / 16), b_lo = b_hi + T2_B_PART / 16;
#pragma unroll
        for (int j = 0; j < T2_K / 8; ++j) {
          const uint32_t o = (uint32_t)j * 16u;      // eight columns further: two core matrices = 256 bytes
          umma_ss_tf32(tmem, a_hi + o, hiword, b_hi + o, hiword, idesc, (i | j) != 0);
          umma_ss_tf32(tmem, a_lo + o, hiword, b_hi + o, hiword, idesc, 1u);
          umma_ss_tf32(tmem, a_hi + o, hiword, b_lo + o, hiword, idesc, 1u);
        }
        umma_commit(&ctl->a_free[st]);
        umma_commit(&ctl->b_empty[sl]);
      }
      umma_commit(&ctl->acc_full);
    }
    __syncwarp();
  } else {
    if (lane == 0) {
      const uint8_t* src = reinterpret_cast<const uint8_t*>(g.Bpack) + (size_t)blockIdx.x * nk * T2_B_SLOT;
      int issued = 0;
      for (int i = 0; i < nk; ++i, ++issued) {
        const int sl = i % T2_BSLOTS;
        if (i >= T2_BSLOTS && !tc_wait(&ctl->b_empty[sl], (uint32_t)(((i / T2_BSLOTS) - 1) & 1), abort_flag)) break;
        mbar_expect_tx(&ctl->b_full[sl], (uint32_t)T2_B_SLOT);
        const int c = i + rot < nk ? i + rot : i + rot - nk;
        bulk_copy_g2s(b_slots + (size_t)sl * T2_B_SLOT, src + (size_t)c * T2_B_SLOT, (uint32_t)T2_B_SLOT, &ctl->b_full[sl]);
      }
      // after a timeout elsewhere the last copies may still be on their way: they must land before the block leaves
      if (*abort_flag)
        for (int i = issued > T2_BSLOTS ? issued - T2_BSLOTS : 0; i < issued; ++i)
          if (!tc_wait(&ctl->b_full[i % T2_BSLOTS], (uint32_t)((i / T2_BSLOTS) & 1), abort_flag)) break;
    }
    __syncwarp();
  }

  // after a timeout the abort flag is up and the tile is not written
  tc_wait_elect(&ctl->acc_full, 0u, abort_flag);
  __syncthreads();
  const bool good = *abort_flag == 0;
  if (good && tid < T2_WORKERS) {
    tc_fence_after();
    const int q = warp & 3, half = warp >> 2;      // TMEM lane quarter of this warp, column half
    const uint32_t t_acc = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * (T2_N / 2));
    float* __restrict__ C = g.C;
    const float* __restrict__ bias = g.bias;
    const float* __restrict__ mask = g.mask;
    float* stg = stg_all + warp * (32 * T2_STG_LD);
#pragma unroll 1
    for (int c0 = 0; c0 < T2_N / 2; c0 += 32) {
      uint32_t v[32];
      tmem_ld16(t_acc + (uint32_t)c0, v);
      tmem_ld16(t_acc + (uint32_t)c0 + 16u, v + 16);
      tmem_ld_wait();
      stage_rows(stg, lane, v);
      const int n = n0 + half * (T2_N / 2) + c0 + (lane & 7) * 4;
      float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (epi == GM_BIAS_RELU) bv = __ldg(reinterpret_cast<const float4*>(bias + n));
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int m = m0 + q * 32 + (lane >> 3) + 4 * i;
        float4 o = staged_piece(stg, lane, i);
        if (m < M) {
          if (epi == GM_BIAS_RELU) {
            o.x = fmaxf(o.x + bv.x, 0.f); o.y = fmaxf(o.y + bv.y, 0.f); o.z = fmaxf(o.z + bv.z, 0.f); o.w = fmaxf(o.w + bv.w, 0.f);
          } else {
            const float4 k = __ldg(reinterpret_cast<const float4*>(mask + (size_t)m * g.ldm + n));
            o.x = k.x > 0.f ? o.x : 0.f; o.y = k.y > 0.f ? o.y : 0.f; o.z = k.z > 0.f ? o.z : 0.f; o.w = k.w > 0.f ? o.w : 0.f;
          }
          *reinterpret_cast<float4*>(C + (size_t)m * g.ldc + n) = o;
        }
      }
    }
  } else if (!good && tid == 0) {
    atomicExch(error, 3ull);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

// Weight-gradient products on the same tensor-core path: dW[m][n] = sum over minibatch rows r of G[r][m] X[r][n] (G the
// gradient rows of a layer, X its input rows).  The contraction runs over the rows, so both operands are K-major only after a
// transposition, which the workers do on the way from global memory to shared memory: a thread reads one feature of four
// consecutive rows (a warp 32 consecutive features of a row per load: coalesced), which is exactly one 16-byte word of the
// K-major core-matrix layout, splits it and stores both parts.  One thread block = one 128 x 256 (or 128 x 128) tile of one
// product over one range of rows; it writes its sums to P[range][off + m * N + n], a partial gradient laid out like the
// parameter blob, and the apply kernel adds the ranges in order (no atomics, one fixed order).  A product with fewer than 128
// gradient columns (the head: one column per action) reads zeros beyond them.  The first column tile of a product also
// writes the bias gradient, the column sums of G over the range: its loaders hold those values anyway.
constexpr int WG_STAGES = 3;
constexpr int WG_A_PART = T2_M * T2_K * 4, WG_B_PART = T2_N * T2_K * 4;          // 8 KB, 16 KB
constexpr int WG_STAGE = 2 * WG_A_PART + 2 * WG_B_PART;                          // A_hi | A_lo | B_hi | B_lo: 48 KB
struct WgCtl {
  uint64_t ready[WG_STAGES], free_[WG_STAGES], acc_full;
  uint32_t tmem_base;
  int abort_flag;
  float bias_part[T2_WORKERS];     // per loader thread: its feature's sum over the row groups it read
};
constexpr int WG_SMEM_BYTES = WG_STAGES * WG_STAGE + T2_STG_BYTES + (int)sizeof(WgCtl) + 1024;

__global__ void __launch_bounds__(T2_THREADS, 1) sg_wgrad_tc_kernel(const TcWgradBatch batch, float* __restrict__ P, int count, int n_rows,
                                                                    int rows_per_range, unsigned long long* __restrict__ error) {
  extern __shared__ uint8_t wg_raw[];
  uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(wg_raw) + 1023) & ~(uintptr_t)1023);
  float* stg_all = reinterpret_cast<float*>(stages + WG_STAGES * WG_STAGE);
  WgCtl* ctl = reinterpret_cast<WgCtl*>(stages + WG_STAGES * WG_STAGE + T2_STG_BYTES);
  int q = 0;
  while (q + 1 < batch.n && (int)blockIdx.x >= batch.g[q + 1].tile_begin) ++q;
  const TcWgrad& g = batch.g[q];
  const int BN = g.N % T2_N == 0 ? T2_N : 128;                 // columns of this product's tiles
  const int t = blockIdx.x - g.tile_begin, tiles_n = g.N / BN;
  const int m0 = (t / tiles_n) * T2_M, n0 = (t % tiles_n) * BN;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool with_bias = g.bias_off >= 0 && n0 == 0;
  float bsum = 0.f;
  const int j_begin = blockIdx.y * rows_per_range;
  const int j_end = j_begin + rows_per_range < n_rows ? j_begin + rows_per_range : n_rows;
  const int nk = j_end > j_begin ? (j_end - j_begin + T2_K - 1) / T2_K : 0;
  if (tid == 0) {
    for (int i = 0; i < WG_STAGES; ++i) { mbar_init(&ctl->ready[i], T2_WORKERS / 32); mbar_init(&ctl->free_[i], 1); }
    mbar_init(&ctl->acc_full, 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&ctl->tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  if (tid < T2_WORKERS) {
    // task u of a thread: feature (tid + 256 u) mod F of row group (tid + 256 u) / F, F = 128 (A) or BN (B)
    const float* __restrict__ Am = g.Am;
    const float* __restrict__ Bm = g.Bm;
    const int lda = g.lda, ldb = g.ldb;
    const int nb_tasks = BN / 64;                               // 4 or 2 per thread
    float4 ra[2][2], rb[2][4];
    auto load4 = [&](const float* base, int ld, int j, int col) -> float4 {
      float4 v;
      v.x = j < j_end ? __ldg(base + (size_t)j * ld + col) : 0.f;
      v.y = j + 1 < j_end ? __ldg(base + (size_t)(j + 1) * ld + col) : 0.f;
      v.z = j + 2 < j_end ? __ldg(base + (size_t)(j + 2) * ld + col) : 0.f;
      v.w = j + 3 < j_end ? __ldg(base + (size_t)(j + 3) * ld + col) : 0.f;
      return v;
    };
    auto fetch = [&](int i, float4 (&fa)[2], float4 (&fb)[4]) {
      const int j0 = j_begin + i * T2_K;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int task = tid + 256 * u;
        fa[u] = m0 + (task & 127) < g.M ? load4(Am, lda, j0 + (task >> 7) * 4, m0 + (task & 127)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (u < nb_tasks) {
          const int task = tid + 256 * u;
          fb[u] = BN == T2_N ? load4(Bm, ldb, j0 + (task >> 8) * 4, n0 + (task & 255)) : load4(Bm, ldb, j0 + (task >> 7) * 4, n0 + (task & 127));
        }
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
    bool ok = true;
    auto step = [&](int i, float4 (&fa)[2], float4 (&fb)[4]) {
      const int st = i % WG_STAGES;
      uint8_t* base = stages + (size_t)st * WG_STAGE;
      if (i >= WG_STAGES) ok = tc_wait_elect(&ctl->free_[st], (uint32_t)(((i / WG_STAGES) - 1) & 1), abort_flag);
      if (!ok) return;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int task = tid + 256 * u, f = task & 127, kg = task >> 7;
        const size_t off = (size_t)((f >> 3) * 4 + kg) * 128 + (size_t)(f & 7) * 16;
        split_store(base + off, base + WG_A_PART + off, fa[u]);
        bsum += (fa[u].x + fa[u].y) + (fa[u].z + fa[u].w);     // rows beyond the range were read as zeros
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (u < nb_tasks) {
          const int task = tid + 256 * u;
          const int f = BN == T2_N ? (task & 255) : (task & 127), kg = BN == T2_N ? (task >> 8) : (task >> 7);
          const size_t off = (size_t)((f >> 3) * 4 + kg) * 128 + (size_t)(f & 7) * 16;
          split_store(base + 2 * WG_A_PART + off, base + 2 * WG_A_PART + WG_B_PART + off, fb[u]);
        }
      }
      fence_async_smem();
      mbar_arrive_warp(&ctl->ready[st]);
      if (i + 2 < nk) fetch(i + 2, fa, fb);
    };
    if (0 < nk) fetch(0, ra[0], rb[0]);
    if (1 < nk) fetch(1, ra[1], rb[1]);
    for (int i = 0; i < nk && ok; i += 2) {
      step(i, ra[0], rb[0]);
      if (ok && i + 1 < nk) step(i + 1, ra[1], rb[1]);
    }
    ctl->bias_part[tid] = bsum;
  } else if (warp == T2_WORKERS / 32) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc_tf32(BN), hiword = desc_hi(T2_SBO);
      const uint32_t s0 = desc_lo(smem_addr(stages), 128u);
      for (int i = 0; i < nk; ++i) {
        const int st = i % WG_STAGES;
        if (!tc_wait(&ctl->ready[st], (uint32_t)((i / WG_STAGES) & 1), abort_flag)) break;
        tc_fence_after();
        const uint32_t a_hi = s0 + (uint32_t)st * (WG_STAGE / 16), a_lo = a_hi + WG_A_PART / 16, b_hi = a_hi + 2 * (WG_A_PART / 16),
                       b_lo = b_hi + WG_B_PART / 16;
#pragma unroll
        for (int j = 0; j < T2_K / 8; ++j) {
          const uint32_t o = (uint32_t)j * 16u;      // eight rows of the minibatch further: two core matrices = 256 bytes
          umma_ss_tf32(tmem, a_hi + o, hiword, b_hi + o, hiword, idesc, (i | j) != 0);
          umma_ss_tf32(tmem, a_lo + o, hiword, b_hi + o, hiword, idesc, 1u);
          umma_ss_tf32(tmem, a_hi + o, hiword, b_lo + o, hiword, idesc, 1u);
        }
        umma_commit(&ctl->free_[st]);
      }
      umma_commit(&ctl->acc_full);
    }
    __syncwarp();
  }

  tc_wait_elect(&ctl->acc_full, 0u, abort_flag);
  __syncthreads();
  const bool good = *abort_flag == 0;
  if (good && tid < T2_WORKERS) {
    tc_fence_after();
    const int q4 = warp & 3, half = warp >> 2;      // TMEM lane quarter of this warp, column half
    const int cols = BN / 2;
    const uint32_t t_acc = tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(half * cols);
    float* stg = stg_all + warp * (32 * T2_STG_LD);
    float* dst = P + (size_t)blockIdx.y * count + g.off;
#pragma unroll 1
    for (int c0 = 0; c0 < cols; c0 += 32) {
      uint32_t v[32];
      if (nk > 0) {
        tmem_ld16(t_acc + (uint32_t)c0, v);
        tmem_ld16(t_acc + (uint32_t)c0 + 16u, v + 16);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0u;       // an empty range of rows contributes nothing
      }
      stage_rows(stg, lane, v);
      const int n = n0 + half * cols + c0 + (lane & 7) * 4;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int m = m0 + q4 * 32 + (lane >> 3) + 4 * i;
        const float4 o = staged_piece(stg, lane, i);
        if (m < g.M) {
          float* d = dst + (size_t)m * g.N + n;          // the blob's matrices start at any multiple of four bytes
          if ((reinterpret_cast<uintptr_t>(d) & 15) == 0) {
            *reinterpret_cast<float4*>(d) = o;
          } else {
            d[0] = o.x; d[1] = o.y; d[2] = o.z; d[3] = o.w;
          }
        }
      }
    }
    // bias gradient: feature f was read by threads f (row groups 0 and 2 of every chunk) and f + 128 (groups 1 and 3)
    if (with_bias && tid < T2_M && m0 + tid < g.M)
      P[(size_t)blockIdx.y * count + g.bias_off + m0 + tid] = ctl->bias_part[tid] + ctl->bias_part[tid + T2_M];
  } else if (!good && tid == 0) {
    atomicExch(error, 3ull);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

// W (N x K row-major, or K x N when `transpose`) -> TF32 high part and remainder in the order the product kernel streams
// them: per tile of 256 rows and chunk of 16 columns one 32 KB block [high 256 x 16 | low 256 x 16], each part as K-major
// core matrices (8 rows x 4 columns contiguous; element (n, k) at ((n / 8) * 4 + k / 4) * 32 + (n % 8) * 4 + k % 4).
__global__ void __launch_bounds__(256) sg_pack_tf32_kernel(const TcPackJobs jobs) {
  const TcPackJob& jb = jobs.j[blockIdx.y];
  const int total = jb.N * jb.K, nk = jb.K / T2_K;
  constexpr int PER = T2_N * T2_K;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int chunk = i / PER, within = i % PER;
    const int tile = chunk / nk, c = chunk % nk;
    const int core = within / 32, in_core = within % 32;
    const int n = tile * T2_N + (core / 4) * 8 + in_core / 4, k = c * T2_K + (core % 4) * 4 + in_core % 4;
    const float v = jb.transpose ? jb.W[(size_t)k * jb.ld + n] : jb.W[(size_t)n * jb.ld + k];
    const float hi = __uint_as_float(__float_as_uint(v) & 0xFFFFE000u);
    float* d = jb.dst + (size_t)chunk * (2 * PER);
    d[within] = hi;
    d[PER + within] = v - hi;
  }
}

}  // namespace

bool tc_gemm2_ok(const float* A, int lda, int M, int N, int K) {
  const long long tiles = (long long)((M + T2_M - 1) / T2_M) * (N / T2_N);
  return N % T2_N == 0 && K % T2_K == 0 && K >= 2 * T2_K && (lda & 3) == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0 && tiles >= 48;
}

size_t tc_pack_floats(int N, int K) { return (size_t)2 * N * K; }

cudaError_t launch_pack_tf32_operands(const TcPackJobs& jobs, cudaStream_t s) {
  if (jobs.n <= 0) return cudaSuccess;
  sg_pack_tf32_kernel<<<dim3(128, jobs.n), 256, 0, s>>>(jobs);
  return cudaGetLastError();
}

cudaError_t launch_gemm_tc2(const TcGemmBatch& batch, int epi, unsigned long long* error, cudaStream_t s) {
  if (batch.n <= 0) return cudaSuccess;
  const TcGemm& g0 = batch.g[0];
  for (int i = 1; i < batch.n; ++i)
    if (batch.g[i].M != g0.M || batch.g[i].N != g0.N) return cudaErrorInvalidValue;   // one grid for all problems of a launch
  cudaError_t e = cudaFuncSetAttribute(sg_gemm_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, T2_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  sg_gemm_tc2_kernel<<<dim3(g0.N / T2_N, (g0.M + T2_M - 1) / T2_M, batch.n), T2_THREADS, T2_SMEM_BYTES, s>>>(batch, epi, error);
  return cudaGetLastError();
}

bool tc_wgrad_ok(int N, int rows) { return N % 128 == 0 && rows >= 1024; }

int tc_wgrad_tiles(int M, int N) { return ((M + T2_M - 1) / T2_M) * (N / (N % T2_N == 0 ? T2_N : 128)); }

cudaError_t launch_wgrad_tc(const TcWgradBatch& batch, float* P, int count, int n_rows, int rows_per_range, int n_ranges,
                            unsigned long long* error, cudaStream_t s) {
  if (batch.n <= 0 || batch.n_tiles <= 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(sg_wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  sg_wgrad_tc_kernel<<<dim3(batch.n_tiles, n_ranges), T2_THREADS, WG_SMEM_BYTES, s>>>(batch, P, count, n_rows, rows_per_range, error);
  return cudaGetLastError();
}

}  // namespace tj
