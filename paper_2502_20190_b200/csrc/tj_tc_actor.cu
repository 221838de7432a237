// Pipelined tensor-core actor step for the linear-Gaussian workload (obs_dim 128, hidden a multiple of 128 up to 512):
// network, action selection, z = A s, env epilogue, record and reset in one persistent kernel whose roles overlap.
//
// A thread block owns 128 rows (envs) per tile, one row per TMEM lane, and walks tiles persistently.  Roles:
//   warp 0, one lane    producer: streams 32 KB operand chunks (weights, the env matrix) from L2 into a ring of two slots
//   warp 1, one lane    MMA issuer (tcgen05.mma, M = 128, N = 128 per hidden block)
//   warps 4-11          network warps (two threads per row): state rows -> BF16 (layer-1 operand); per 128-neuron block of a
//                       hidden layer: accumulator -> bias, ReLU, BF16 -> next layer's operand; z -> a scratch tile in global
//                       memory
//   warps 12-19         env warps: the FP16 parts of the next tile's state rows and the record's observation; take the head
//                       outputs out of TMEM, select the action, read z back and finish the step (tanh, Philox noise, reward,
//                       done, record, reset or new state, counters), eight rows x four 16-byte pieces per warp instruction
// The env warps work on tile i while the network warps and the tensor pipe are already on tile i + 1.
//
// Per tile the tensor pipe runs ten accumulator blocks that alternate between two 128-column accumulators:
//   layer 1 (4 blocks, A operand = X in shared memory), z (one block), layer 2 (4 blocks, A operand = h1 in tensor
//   memory), head (16 columns).  The epilogue of one block overlaps the MMAs of the next.
// z = A s keeps FP32 accuracy on the FP16 tensor path: state and matrix are each split into a high and a low FP16 part
// (power-of-two scaled so the low parts stay normal numbers), z = hi*hi + lo*hi + hi*lo with FP32 accumulation: 24
// instructions of K = 16, relative error about 2^-22 per term (the dropped lo*lo term and the low parts' rounding).
// Tensor memory (512 columns): [0, H/2) h1 as packed BF16 pairs; [256, 384) and [384, 512) the two accumulators.
// Shared memory: X (BF16 state tile, 32 KB) | U (128 KB: the FP16 high and low parts of the state tile in its first 64 KB
// until z is done, then h2, the head's A operand) | ring (64 KB) | barriers.
// Every wait is bounded: on a timeout the block raises an abort flag, records an error, frees its TMEM and leaves.
#include <cuda_fp16.h>

#include "tj_internal.h"
#include "tj_tc.cuh"

namespace tj {

namespace {

constexpr int PA_M = 128;                  // rows per tile
constexpr int PA_D = 128;                  // observation / state width this kernel is built for
constexpr int PA_NB = 128;                 // neurons per accumulator block
constexpr int PA_KC = 128;                 // K elements per weight chunk (128 x 128 x 2 bytes = 32 KB)
constexpr int PA_W_BYTES = PA_NB * PA_KC * 2;              // bytes of a hidden-layer weight chunk, and of one env-matrix part
constexpr int PA_STAGE_BYTES = PA_W_BYTES;
constexpr int PA_STAGES = 65536 / PA_STAGE_BYTES;
constexpr int PA_X_BYTES = PA_M * PA_D * 2;
constexpr int PA_U_BYTES = 131072;
constexpr int PA_THREADS = 640;            // warps 0-3: producer, MMA issuer, two idle; 4-11 network; 12-19 env
constexpr int PA_GROUP_WARPS = 8;          // warps of the network group and of the env group (one barrier arrival each)
constexpr uint32_t PA_COL_HB = 0, PA_COL_ACC0 = 256, PA_COL_ACC1 = 384;
constexpr int PA_N3 = 16;                  // head width on the tensor cores
constexpr int PA_MAX_GRID = 192;           // thread blocks the z scratch is sized for
constexpr float PA_S_SCALE = 256.0f;       // state values are split after this scaling (|s| < 1.2: far below FP16's range)

struct PaSmem {
  uint64_t full[PA_STAGES], empty[PA_STAGES];
  uint64_t x_ready;        // network -> MMA: X holds the tile's BF16 rows
  uint64_t u_ready;        // env -> MMA: U holds the tile's FP16 high / low parts
  uint64_t acc_full[2];    // MMA -> network: an accumulator block is complete
  uint64_t acc_empty[2];   // network -> MMA: it has been drained (and its result stored)
  uint64_t head_full;      // MMA -> env and network: head outputs complete; U may be rewritten
  uint64_t env_taken;      // env -> MMA: head outputs are in registers
  uint64_t z_stored;       // network -> env: z of the tile is in the scratch tile
  uint64_t act_ready;      // env: the rows' actions are in shared memory
  int act[2][PA_M];        // by tile parity
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__global__ void __launch_bounds__(PA_THREADS, 1) actor_tc_pipelined_kernel(const TcMlpParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr int D = PA_D;
  const int H = p.H;
  uint8_t* xbuf = smem_raw;
  uint8_t* ubuf = xbuf + PA_X_BYTES;
  uint8_t* ring = ubuf + PA_U_BYTES;
  PaSmem* ctl = reinterpret_cast<PaSmem*>(ring + PA_STAGES * PA_STAGE_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_tiles = (p.n + PA_M - 1) / PA_M;
  const int n_hb = H / PA_NB;            // 128-neuron blocks per hidden layer
  // Thread blocks walk the neuron blocks of a layer in rotated order, so that at any moment they stream different
  // parts of the weights from L2 (the arithmetic per neuron is unchanged)
  const int rot = (int)(blockIdx.x % (unsigned)n_hb);
  const int n_kc2 = H / PA_KC;           // K chunks of a layer-2 block (a layer-1 block has one)

  if (tid == 0) {
    for (int s = 0; s < PA_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    mbar_init(&ctl->x_ready, PA_GROUP_WARPS);
    mbar_init(&ctl->u_ready, PA_GROUP_WARPS);
    mbar_init(&ctl->acc_full[0], 1);
    mbar_init(&ctl->acc_full[1], 1);
    mbar_init(&ctl->acc_empty[0], PA_GROUP_WARPS);
    mbar_init(&ctl->acc_empty[1], PA_GROUP_WARPS);
    mbar_init(&ctl->head_full, 1);
    mbar_init(&ctl->env_taken, PA_GROUP_WARPS);
    mbar_init(&ctl->z_stored, PA_GROUP_WARPS);
    mbar_init(&ctl->act_ready, 4);
    ctl->abort_flag = 0;
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&ctl->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;
  const TcEnvParams& ev = p.env;

  if (warp < 4) {
    // registers: 640 threads x 96 at launch = 61,440; 128 x 64 + 256 x 96 + 256 x 112 = 61,440 after the two changes.  The
    // issuing lane's loop is the pace-maker of the whole block: it must not spill, so its warpgroup keeps 64 registers.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- producer
      // order per tile (the order the MMA issuer consumes): layer 1 (one chunk per block), env matrix (high part, low
      // part), layer 2 (H/128 chunks per block), head
      uint32_t it = 0;
      // every block re-reads the same chunks each tile while state rows and records stream through L2 once: the chunks
      // are fetched with an evict-last policy, the streams are written with evict-first stores
      const unsigned long long keep_policy = l2_evict_last_policy();
      const uint32_t head_bytes = (uint32_t)PA_N3 * H * 2;
      const int n1 = n_hb, n2 = n_hb * n_kc2;
      for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x) {
        for (int c = 0; c < n1 + 2 + n2 + 1; ++c, ++it) {
          const uint8_t* src;
          uint32_t bytes = PA_W_BYTES;
          if (c < n1) src = reinterpret_cast<const uint8_t*>(p.wtc) + (size_t)((c + rot) % n_hb) * PA_W_BYTES;
          else if (c < n1 + 2) src = reinterpret_cast<const uint8_t*>(ev.lgA16) + (size_t)(c - n1) * PA_W_BYTES;
          else if (c < n1 + 2 + n2) {
            const int idx = c - n1 - 2;
            src = reinterpret_cast<const uint8_t*>(p.wtc) + (size_t)(n1 + ((idx / n_kc2 + rot) % n_hb) * n_kc2 + idx % n_kc2) * PA_W_BYTES;
          }
          else { src = reinterpret_cast<const uint8_t*>(p.wtc) + (size_t)(n1 + n2) * PA_W_BYTES; bytes = head_bytes; }
          const int s = it % PA_STAGES;
          if (!tc_wait(&ctl->empty[s], ((it / PA_STAGES) & 1) ^ 1, abort_flag)) goto done;
          mbar_expect_tx(&ctl->full[s], bytes);
          bulk_copy_g2s_keep(ring + (size_t)s * PA_STAGE_BYTES, src, bytes, &ctl->full[s], keep_policy);
        }
      }
    } else if (warp == 1 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      // Accumulator uses of a tile: u = 0 .. n_hb-1 layer 1, n_hb z, n_hb+1 .. 2 n_hb layer 2, 2 n_hb + 1 head; use u
      // writes accumulator u & 1 (the count per tile is even, so the pattern repeats).  The network warps drain every use
      // but the head (acc_empty), the env warps take the head (env_taken).
      uint32_t it = 0, tiles = 0, nwait0 = 0, nwait1 = 0;
      const uint32_t idesc_h = make_idesc(PA_NB), idesc16 = make_idesc(PA_N3), idesc_z = make_idesc_f16(D);
      // descriptors as (low, high) words: the high word is fixed per operand shape, the low word steps by 16 per K = 16
      const uint32_t x_lo = desc_lo(smem_addr(xbuf), 128u), u_lo = desc_lo(smem_addr(ubuf), 128u);
      const uint32_t ulo_lo = desc_lo(smem_addr(ubuf) + (uint32_t)PA_X_BYTES, 128u);
      const uint32_t ring_lo = desc_lo(smem_addr(ring), 128u);
      const uint32_t hi_k128 = desc_hi(2048u);                       // operands 128 K-elements wide (X, U, weight chunks)
      const uint32_t hi_head = desc_hi((uint32_t)(H / 8) * 128u);    // operands H K-elements wide (h2, head weights)
      // before use u may overwrite its accumulator, the previous use of that accumulator must have been read out
      auto acquire = [&](int u) -> bool {
        if (u == 0) return true;      // accumulator 0: its last drain was awaited before the previous tile's head
        if (u == 1) return tiles == 0 || tc_wait(&ctl->env_taken, (tiles - 1) & 1, abort_flag);
        return (u & 1) ? tc_wait(&ctl->acc_empty[1], (nwait1++) & 1, abort_flag) : tc_wait(&ctl->acc_empty[0], (nwait0++) & 1, abort_flag);
      };
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tiles) {
        if (!tc_wait(&ctl->x_ready, tiles & 1, abort_flag)) goto done;
        // layer 1: one chunk per 128-neuron block; A operand = X in shared memory
        for (int b = 0; b < n_hb; ++b, ++it) {
          const int u = b;
          if (!acquire(u)) goto done;
          const uint32_t acc = tmem + ((u & 1) ? PA_COL_ACC1 : PA_COL_ACC0);
          const uint32_t s = it % PA_STAGES;
          if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
          tc_fence_after();
          const uint32_t b_lo = ring_lo + s * (PA_STAGE_BYTES / 16);
#pragma unroll
          for (int j = 0; j < PA_KC / 16; ++j) umma_ss(acc, x_lo + j * 16u, hi_k128, b_lo + j * 16u, hi_k128, idesc_h, j != 0);
          umma_commit(&ctl->empty[s]);
          umma_commit((u & 1) ? &ctl->acc_full[1] : &ctl->acc_full[0]);
        }
        // z = A s from the FP16 parts: (s_hi, A_hi) + (s_lo, A_hi) with the first chunk, (s_hi, A_lo) with the second
        {
          const int u = n_hb;
          if (!tc_wait(&ctl->u_ready, tiles & 1, abort_flag)) goto done;
          if (!acquire(u)) goto done;
          const uint32_t acc = tmem + ((u & 1) ? PA_COL_ACC1 : PA_COL_ACC0);
          for (int part = 0; part < 2; ++part, ++it) {
            const uint32_t s = it % PA_STAGES;
            if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
            tc_fence_after();
            const uint32_t b_lo = ring_lo + s * (PA_STAGE_BYTES / 16);
#pragma unroll
            for (int j = 0; j < D / 16; ++j) {
              umma_ss(acc, u_lo + j * 16u, hi_k128, b_lo + j * 16u, hi_k128, idesc_z, (part | j) != 0);
              if (part == 0) umma_ss(acc, ulo_lo + j * 16u, hi_k128, b_lo + j * 16u, hi_k128, idesc_z, 1u);
            }
            umma_commit(&ctl->empty[s]);
          }
          umma_commit((u & 1) ? &ctl->acc_full[1] : &ctl->acc_full[0]);
        }
        // layer 2: per block H / PA_KC chunks; A operand = h1 in tensor memory (8 columns per K = 16); the drain of the last
        // layer-1 block (awaited by the first block here) completes h1
        for (int b = 0; b < n_hb; ++b) {
          const int u = n_hb + 1 + b;
          if (!acquire(u)) goto done;
          const uint32_t acc = tmem + ((u & 1) ? PA_COL_ACC1 : PA_COL_ACC0);
          for (int c = 0; c < n_kc2; ++c, ++it) {
            const uint32_t s = it % PA_STAGES;
            if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
            tc_fence_after();
            const uint32_t b_lo = ring_lo + s * (PA_STAGE_BYTES / 16);
            const uint32_t a_col = tmem + PA_COL_HB + (uint32_t)(c * (PA_KC / 2));
#pragma unroll
            for (int j = 0; j < PA_KC / 16; ++j) umma_ts(acc, a_col + (uint32_t)(j * 8), b_lo + j * 16u, hi_k128, idesc_h, (c | j) != 0);
            umma_commit(&ctl->empty[s]);
          }
          umma_commit((u & 1) ? &ctl->acc_full[1] : &ctl->acc_full[0]);
        }
        // head: 16 outputs, K = H, A operand = h2 in shared memory; accumulator 1.  Both remaining drains complete h2.
        {
          if (!acquire(2 * n_hb + 1)) goto done;
          if (!tc_wait(&ctl->acc_empty[0], (nwait0++) & 1, abort_flag)) goto done;
          const uint32_t s = it % PA_STAGES;
          if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
          tc_fence_after();
          const uint32_t b_lo = ring_lo + s * (PA_STAGE_BYTES / 16);
          for (int j = 0; j < H / 16; ++j) umma_ss(tmem + PA_COL_ACC1, u_lo + j * 16u, hi_head, b_lo + j * 16u, hi_head, idesc16, j != 0);
          umma_commit(&ctl->empty[s]);
          umma_commit(&ctl->head_full);
          ++it;
        }
      }
    }
  } else if (warp < 12) {
    // ------------------------------------------------------------------ network warps
    const int q = warp & 3;                       // TMEM lane quarter this warp may access
    const int hsel = (warp - 4) >> 2;             // which half of a row / of a block's columns
    const int r = q * 32 + lane;                  // row of the tile = TMEM lane
    const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16);
    uint32_t tiles = 0, nfull0 = 0, nfull1 = 0;
    // Conversions read the row-major state with eight rows x four 16-byte pieces per warp instruction (64 contiguous
    // bytes per row) instead of one row per lane: a quarter of the memory wavefronts, and conflict-free stores.
    const int nw = warp - 4, c_r8 = lane >> 2, c_kq = lane & 3;
    // BF16 rows of a tile -> X (layer-1 A operand)
    auto convert_x = [&](int tile) {
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        const int rr = nw * 16 + g * 8 + c_r8;
        const long long row = (long long)tile * PA_M + rr;
        const float* xr = p.x + (size_t)(row < p.n ? row : 0) * D;
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = row < p.n ? __ldg(reinterpret_cast<const float4*>(xr + (c_kq + 4 * i) * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        uint8_t* dx = xbuf + ((size_t)(rr >> 3) * (D / 8)) * 128 + (rr & 7) * 16;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int k4 = c_kq + 4 * i;
          *reinterpret_cast<uint2*>(dx + (size_t)(k4 >> 1) * 128 + (k4 & 1) * 8) =
              make_uint2(pack_bf16x2(v[i].x, v[i].y), pack_bf16x2(v[i].z, v[i].w));
        }
      }
      fence_async_smem();
      mbar_arrive_warp(&ctl->x_ready);
    };
    if ((int)blockIdx.x < n_tiles) convert_x(blockIdx.x);
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tiles) {
      const int next_tile = tile + (int)gridDim.x;
      {
        // pull the rows of the tile after the next towards L2
        const long long prow = (long long)(next_tile + (int)gridDim.x) * PA_M + r;
        if (prow < p.n) {
          const float* xn = p.x + (size_t)prow * D + hsel * 64;
          prefetch_l2(xn);
          prefetch_l2(xn + 32);
        }
      }
      for (int u = 0; u <= 2 * n_hb; ++u) {
        const int buf = u & 1;
        if (!tc_wait_elect(buf ? &ctl->acc_full[1] : &ctl->acc_full[0], (buf ? nfull1++ : nfull0++) & 1, abort_flag)) goto done;
        tc_fence_after();
        const uint32_t t_acc = t_lane + (buf ? PA_COL_ACC1 : PA_COL_ACC0) + (uint32_t)(hsel * 64);
        if (u == n_hb) {
          // z: this thread's 64 components go to the block's scratch tile, where the env warps pick them up
          uint32_t v[64];
#pragma unroll
          for (int g = 0; g < 4; ++g) tmem_ld16(t_acc + (uint32_t)(g * 16), v + 16 * g);
          tmem_ld_wait();
          tc_fence_before();
          {
            // scratch tile [k/4][row][4]: a warp's 32 rows are contiguous, for this store and for the env warps' loads
            float* zs = ev.z_scratch + ((size_t)blockIdx.x * 2 + (tiles & 1)) * (PA_M * D);
#pragma unroll
            for (int i = 0; i < 16; ++i)
              *reinterpret_cast<uint4*>(zs + ((size_t)(hsel * 16 + i) * PA_M + r) * 4) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          }
          mbar_arrive_warp(&ctl->acc_empty[buf]);
          mbar_arrive_warp(&ctl->z_stored);
          // layer 1 of this tile is complete, so X is free: the next tile's rows go in while layer 2 runs
          if (next_tile < n_tiles) convert_x(next_tile);
          continue;
        }
        const int layer = u < n_hb ? 0 : 1;
        const int b = ((layer == 0 ? u : u - n_hb - 1) + rot) % n_hb;   // neuron block of this use
        const float* bias = layer == 0 ? p.b1 : p.b2;
        const int c0 = b * PA_NB + hsel * 64;          // first of this thread's 64 columns
        uint32_t v[64];
#pragma unroll
        for (int g = 0; g < 4; ++g) tmem_ld16(t_acc + (uint32_t)(g * 16), v + 16 * g);
        tmem_ld_wait();
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t o[16];
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) {
            float f0 = __uint_as_float(v[hh * 32 + 4 * j4 + 0]), f1 = __uint_as_float(v[hh * 32 + 4 * j4 + 1]);
            float f2 = __uint_as_float(v[hh * 32 + 4 * j4 + 2]), f3 = __uint_as_float(v[hh * 32 + 4 * j4 + 3]);
            const float4 bb = __ldg(reinterpret_cast<const float4*>(bias + c0 + hh * 32 + 4 * j4));
            f0 += bb.x; f1 += bb.y; f2 += bb.z; f3 += bb.w;
            o[2 * j4] = pack_bf16x2_relu(f0, f1);
            o[2 * j4 + 1] = pack_bf16x2_relu(f2, f3);
          }
          if (layer == 0) {
            tmem_st16(t_lane + PA_COL_HB + (uint32_t)((c0 + hh * 32) / 2), o);
          } else {
            uint8_t* dst = ubuf + ((size_t)(r >> 3) * (H / 8)) * 128 + (r & 7) * 16 + (size_t)((c0 + hh * 32) / 8) * 128;
#pragma unroll
            for (int g = 0; g < 4; ++g)
              *reinterpret_cast<uint4*>(dst + (size_t)g * 128) = make_uint4(o[4 * g], o[4 * g + 1], o[4 * g + 2], o[4 * g + 3]);
          }
        }
        if (layer == 0) tmem_st_wait();
        else fence_async_smem();
        tc_fence_before();
        mbar_arrive_warp(&ctl->acc_empty[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------------ env warps
    asm volatile("setmaxnreg.inc.sync.aligned.u32 112;");
    const int ew = warp - 12;                      // 0..7; the first four also read the head outputs (one TMEM quarter each)
    const int e_r8 = lane >> 2, e_kq = lane & 3;   // env step: eight rows x four 16-byte pieces per warp instruction
    uint32_t tiles = 0;
    // FP16 high / low parts of a tile's scaled rows -> U (A operand of z = A s); the FP32 row is the record's observation
    auto convert_u = [&](int tile) {
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        const int rr = ew * 16 + g * 8 + e_r8;
        const long long row = (long long)tile * PA_M + rr;
        const bool live = row < p.n;
        const float* xr = p.x + (size_t)(live ? row : 0) * D;
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = live ? __ldg(reinterpret_cast<const float4*>(xr + (e_kq + 4 * i) * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        uint8_t* dhi = ubuf + ((size_t)(rr >> 3) * (D / 8)) * 128 + (rr & 7) * 16;
        uint8_t* dlo = dhi + PA_X_BYTES;
        float* rec = ev.ring + (ev.slot0 + (unsigned long long)(live ? row : 0)) * ev.rec_words;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int k4 = e_kq + 4 * i;
          const float4 sv = v[i];
          // high part: the scaled value cut to 11 significant bits (exact in FP16); low part: the exact remainder, rounded
          float4 s4, hi, lo;
          s4.x = sv.x * PA_S_SCALE; s4.y = sv.y * PA_S_SCALE; s4.z = sv.z * PA_S_SCALE; s4.w = sv.w * PA_S_SCALE;
          hi.x = __uint_as_float(__float_as_uint(s4.x) & 0xFFFFE000u); lo.x = s4.x - hi.x;
          hi.y = __uint_as_float(__float_as_uint(s4.y) & 0xFFFFE000u); lo.y = s4.y - hi.y;
          hi.z = __uint_as_float(__float_as_uint(s4.z) & 0xFFFFE000u); lo.z = s4.z - hi.z;
          hi.w = __uint_as_float(__float_as_uint(s4.w) & 0xFFFFE000u); lo.w = s4.w - hi.w;
          const size_t off = (size_t)(k4 >> 1) * 128 + (k4 & 1) * 8;
          *reinterpret_cast<uint2*>(dhi + off) = make_uint2(pack_f16x2(hi.x, hi.y), pack_f16x2(hi.z, hi.w));
          *reinterpret_cast<uint2*>(dlo + off) = make_uint2(pack_f16x2(lo.x, lo.y), pack_f16x2(lo.z, lo.w));
          if (live) __stcs(reinterpret_cast<float4*>(rec + k4 * 4), sv);
        }
      }
      fence_async_smem();
      mbar_arrive_warp(&ctl->u_ready);
    };
    if ((int)blockIdx.x < n_tiles) convert_u(blockIdx.x);
    unsigned long long n_episodes = 0;
    double ret_sum = 0.0;
    const float zc = ev.z_to_t;                    // accumulator -> 2 log2(e) * z
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tiles) {
      if (ew < 4) {
        const int r = ew * 32 + lane;              // row of the tile = TMEM lane
        const long long row = (long long)tile * PA_M + r;
        if (!tc_wait_elect(&ctl->head_full, tiles & 1, abort_flag)) goto done;
        tc_fence_after();
        uint32_t qraw[16];
        tmem_ld16(tmem + ((uint32_t)(ew * 32) << 16) + PA_COL_ACC1, qraw);
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive_warp(&ctl->env_taken);
        // epsilon-greedy on this row: explore iff x0 < threshold, else the first maximum
        float qv[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) qv[j] = __uint_as_float(qraw[j]) + (j < p.Aout ? __ldg(p.b3 + j) : 0.f);
        if (row < p.n && p.out) {
          float* o = p.out + (size_t)row * p.Aout;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j < p.Aout) o[j] = qv[j];
        }
        const uint4 w = stream_words(ev.seed, STREAM_ACTION, 0, (uint32_t)row, ev.t);
        int best = 0;
        float qb = qv[0];
#pragma unroll
        for (int j = 1; j < 16; ++j)
          if (j < ev.A && qv[j] > qb) { qb = qv[j]; best = j; }
        ctl->act[tiles & 1][r] = ((unsigned long long)w.x < ev.explore_thr) ? (int)__umulhi(w.y, (uint32_t)ev.A) : best;
        mbar_arrive_warp(&ctl->act_ready);
      } else {
        mbar_arrive_warp(&ctl->env_taken);         // this warp has finished the previous tile
        if (!tc_wait_elect(&ctl->head_full, tiles & 1, abort_flag)) goto done;
      }
      // the head of this tile is complete, so U is free: the next tile's FP16 parts go in before this tile's env step
      if (tile + (int)gridDim.x < n_tiles) convert_u(tile + (int)gridDim.x);
      if (!tc_wait_elect(&ctl->act_ready, tiles & 1, abort_flag)) goto done;
      // z was stored long before the head finished; the wait orders the loads below after those stores
      if (!tc_wait_elect(&ctl->z_stored, tiles & 1, abort_flag)) goto done;
      const float* zs = ev.z_scratch + ((size_t)blockIdx.x * 2 + (tiles & 1)) * (PA_M * D);
#pragma unroll 1
      for (int g = 0; g < 2; ++g) {
        const int rr = ew * 16 + g * 8 + e_r8;
        const long long row = (long long)tile * PA_M + rr;
        const bool live = row < p.n;
        const int action = ctl->act[tiles & 1][rr];
        float* rec = ev.ring + (ev.slot0 + (unsigned long long)(live ? row : 0)) * ev.rec_words;
        const int ep0 = live ? ev.ep_step[row] : 0;
        const float ret0 = live ? ev.ep_return[row] : 0.f;
        const float* Ba = ev.lgB_t + (size_t)action * D;     // B[a] times 2 log2(e)
        // s' = tanh(z + B[a]) + noise; piece k4 = components 4 k4 .. 4 k4 + 3 = one Philox block
        float4 zz[8], sn[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) zz[i] = __ldcg(reinterpret_cast<const float4*>(zs + ((size_t)(e_kq + 4 * i) * PA_M + rr) * 4));
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int k4 = e_kq + 4 * i;
          const uint4 w = stream_words(ev.seed, STREAM_NOISE, (uint32_t)k4, (uint32_t)row, ev.t);
          const float2 n01 = box_muller_scaled(w.x, w.y, ev.noise_std), n23 = box_muller_scaled(w.z, w.w, ev.noise_std);
          const float4 bb = __ldg(reinterpret_cast<const float4*>(Ba + 4 * k4));
          float4 o;
          o.x = tanh_from_t(fmaf(zz[i].x, zc, bb.x)) + n01.x;
          o.y = tanh_from_t(fmaf(zz[i].y, zc, bb.y)) + n01.y;
          o.z = tanh_from_t(fmaf(zz[i].z, zc, bb.z)) + n23.x;
          o.w = tanh_from_t(fmaf(zz[i].w, zc, bb.w)) + n23.y;
          sq = fmaf(o.x, o.x, sq); sq = fmaf(o.y, o.y, sq); sq = fmaf(o.z, o.z, sq); sq = fmaf(o.w, o.w, sq);
          sn[i] = o;
          if (live) __stcs(reinterpret_cast<float4*>(rec + D + 4 * k4), o);
        }
        // the four lanes of a row add their partial squared norms (same order in every lane)
        sq += __shfl_xor_sync(0xffffffffu, sq, 1);
        sq += __shfl_xor_sync(0xffffffffu, sq, 2);
        if (live) {
          const float rew = -sq / (float)D;
          int ep = ep0 + 1;
          float ep_ret = ret0 + rew;
          const int done = (sqrtf(sq) > ev.done_norm || ep >= ev.max_ep) ? 1 : 0;
          float* st = ev.state + (size_t)row * D;
          if (done) {
            ep_ret = 0.f;
            ep = 0;
#pragma unroll 4
            for (int i = 0; i < 8; ++i) {
              const int k4 = e_kq + 4 * i;
              const uint4 w = stream_words(ev.seed, STREAM_RESET, (uint32_t)k4, (uint32_t)row, ev.t);
              *reinterpret_cast<float4*>(st + 4 * k4) = make_float4(uniform_range(w.x, -0.1f, 0.2f), uniform_range(w.y, -0.1f, 0.2f),
                                                                    uniform_range(w.z, -0.1f, 0.2f), uniform_range(w.w, -0.1f, 0.2f));
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) *reinterpret_cast<float4*>(st + 4 * (e_kq + 4 * i)) = sn[i];
          }
          if (e_kq == 0) {
            *reinterpret_cast<float4*>(rec + 2 * D) =
                make_float4(__int_as_float(action), rew, __int_as_float(done), __int_as_float(ev.version));
            if (done) {
              n_episodes += 1;
              ret_sum += (double)(ret0 + rew);
            }
            ev.ep_step[row] = ep;
            ev.ep_return[row] = ep_ret;
          }
        }
      }
    }
    // episode statistics: one atomic pair per warp
    {
      unsigned long long n = n_episodes;
      double rs = ret_sum;
      for (int o = 16; o > 0; o >>= 1) {
        n += __shfl_down_sync(0xffffffffu, n, o);
        rs += __shfl_down_sync(0xffffffffu, rs, o);
      }
      if (lane == 0 && n) {
        atomicAdd(&ev.stats->episodes, n);
        atomicAdd(&ev.stats->return_sum, rs);
      }
      if (blockIdx.x == 0 && tid == 12 * 32) ev.block_ver[ev.slot0 / (unsigned long long)p.n] = ev.version;
    }
  }
done:
  __syncthreads();
  if (tid == 0 && ctl->abort_flag) atomicExch(p.error, 2ull);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// FP32 blob -> BF16 chunks in the order the pipelined actor streams them.  Hidden layers: per 128-neuron block, chunks of
// 128 rows x 128 columns; element (r, k) of a chunk sits at ((r/8) * 16 + k/8) * 64 + (r%8) * 8 + k%8.  Head: one chunk of
// 16 rows x H columns, element (r, k) at ((r/8) * (H/8) + k/8) * 64 + (r%8) * 8 + k%8.
__global__ void pack_pipelined_weights_kernel(const float* __restrict__ blob, uint16_t* __restrict__ dst, int D, int H, int A) {
  const size_t n1 = (size_t)H * D, n2 = (size_t)H * H, n3 = (size_t)PA_N3 * H;
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n1 + n2 + n3) return;
  const float* W1 = blob;
  const float* W2 = W1 + n1 + H;
  const float* W3 = W2 + n2 + H;
  float v = 0.f;
  if (i < n1 + n2) {
    const bool first = i < n1;
    const size_t j = first ? i : i - n1;
    const int K = first ? D : H;
    const int chunks_per_block = K / PA_KC;
    const size_t chunk = j / (PA_NB * PA_KC), within = j % (PA_NB * PA_KC);
    const int b = (int)(chunk / chunks_per_block), c = (int)(chunk % chunks_per_block);
    const int core = (int)(within / 64), in_core = (int)(within % 64);
    const int rg = core / (PA_KC / 8), kg = core % (PA_KC / 8);
    const int n = b * PA_NB + rg * 8 + in_core / 8, k = c * PA_KC + kg * 8 + in_core % 8;
    v = (first ? W1 : W2)[(size_t)n * K + k];
  } else {
    const size_t j = i - n1 - n2;
    const int core = (int)(j / 64), in_core = (int)(j % 64);
    const int rg = core / (H / 8), kg = core % (H / 8);
    const int n = rg * 8 + in_core / 8, k = kg * 8 + in_core % 8;
    if (n < A) v = W3[(size_t)n * H + k];
  }
  uint32_t u = __float_as_uint(v);
  u += 0x7FFFu + ((u >> 16) & 1u);
  dst[i] = (uint16_t)(u >> 16);
}

// The env matrix A [128][128] scaled by `scale` (a power of two) as two FP16 chunks, high parts then low parts, each in the
// layout of a weight chunk (row = component of z, column = component of s); B [n_actions][128] times 2 log2(e).
__global__ void pack_env_f16_kernel(const float* __restrict__ A, const float* __restrict__ B, float scale, int n_b,
                                    uint16_t* __restrict__ dst, float* __restrict__ b_t) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < PA_D * PA_D) {
    const int core = i / 64, in_core = i % 64;
    const int rg = core / (PA_D / 8), kg = core % (PA_D / 8);
    const int n = rg * 8 + in_core / 8, k = kg * 8 + in_core % 8;
    const float v = A[(size_t)n * PA_D + k] * scale;
    const __half hi = __float2half_rn(v);
    const __half lo = __float2half_rn(v - __half2float(hi));
    dst[i] = __half_as_ushort(hi);
    dst[PA_D * PA_D + i] = __half_as_ushort(lo);
  }
  if (i < n_b) b_t[i] = B[i] * 2.88539008177792681472f;
}

}  // namespace

bool tc_pipelined_supported(int D, int H, int A) {
  return D == PA_D && H >= PA_NB && H <= 512 && H % PA_NB == 0 && A >= 1 && A <= PA_N3;
}

size_t tc_pipelined_scratch_floats() { return (size_t)PA_MAX_GRID * 2 * PA_M * PA_D; }
size_t tc_pipelined_env_halfs() { return (size_t)2 * PA_D * PA_D; }
float tc_pipelined_state_scale() { return PA_S_SCALE; }

cudaError_t launch_pack_pipelined_weights(const float* blob, uint16_t* dst, int D, int H, int A, cudaStream_t s) {
  const size_t n = tc_weight_elems(D, H);
  pack_pipelined_weights_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(blob, dst, D, H, A);
  return cudaGetLastError();
}

cudaError_t launch_pack_pipelined_env(const float* A, const float* B, float scale, int n_actions, uint16_t* dst, float* b_t,
                                      cudaStream_t s) {
  const int n = PA_D * PA_D > n_actions * PA_D ? PA_D * PA_D : n_actions * PA_D;
  pack_env_f16_kernel<<<(n + 255) / 256, 256, 0, s>>>(A, B, scale, n_actions * PA_D, dst, b_t);
  return cudaGetLastError();
}

cudaError_t launch_actor_tc_pipelined(const TcMlpParams& p, int sm_count, cudaStream_t s) {
  if (p.n <= 0) return cudaSuccess;
  if (!tc_pipelined_supported(p.D, p.H, p.Aout) || !p.env.fused) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)PA_X_BYTES + PA_U_BYTES + (size_t)PA_STAGES * PA_STAGE_BYTES + sizeof(PaSmem) + 64;
  cudaError_t e = cudaFuncSetAttribute(actor_tc_pipelined_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int n_tiles = (p.n + PA_M - 1) / PA_M;
  int grid = n_tiles < sm_count ? n_tiles : sm_count;
  if (grid > PA_MAX_GRID) grid = PA_MAX_GRID;
  if (!p.env.z_scratch || !p.env.lgA16 || !p.env.lgB_t) return cudaErrorInvalidValue;
  actor_tc_pipelined_kernel<<<grid, PA_THREADS, smem, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tj
