// Pipelined tensor-core actor step for the linear-Gaussian workload (obs_dim 128, hidden a multiple of 128 up to 512):
// network, action selection, z = A s, env epilogue, record and reset in one persistent kernel whose roles overlap.
//
// A thread block owns 128 rows (envs) per tile, one row per TMEM lane, and walks tiles persistently.  Roles:
//   warp 0, one lane    producer: streams 16 KB operand chunks (env matrix parts, then weights) from L2 into a 4-slot ring
//   warp 1, one lane    MMA issuer (tcgen05.mma, M = 128)
//   warps 4-11          network warps (two threads per row): state row -> BF16 (layer-1 operand) and TF32 high/low parts
//                       (operand of z = A s), record's observation; per 64-neuron block of a hidden layer: accumulator ->
//                       bias, ReLU, BF16 -> next layer's operand
//   warps 12-19         env warps (two threads per row): take the head outputs and z out of TMEM, select the action, finish
//                       the step (tanh, Philox noise, reward, done, record, reset or new state, episode counters)
// The env warps work on tile i while the network warps and the tensor pipe are already on tile i + 1.
//
// Tensor memory (512 columns): [0, H/2) h1 as packed BF16 pairs -- the A operand of layer 2 is read from tensor memory, so
// the hidden activations never touch shared memory; [256, 384) z; [384, 448) and [448, 512) two 64-column accumulators that
// alternate between the MMA of one 64-neuron block and the epilogue of the previous one (the head's 16 outputs reuse the first).
// Shared memory: X (BF16 state tile, 32 KB) | U (128 KB: TF32 high and low parts of the state tile early in the tile, h2 later,
// as the head's A operand) | ring (64 KB) | barriers.
// Every wait is bounded: on a timeout the block raises an abort flag, records an error, frees its TMEM and leaves.
#include "tj_internal.h"
#include "tj_tc.cuh"

namespace tj {

namespace {

constexpr int PA_M = 128;                  // rows per tile
constexpr int PA_D = 128;                  // observation / state width this kernel is built for
constexpr int PA_NB = 64;                  // neurons per accumulator block
constexpr int PA_KC = 128;                 // K elements per weight chunk (64 x 128 BF16 = 16 KB)
constexpr int PA_STAGES = 4;
constexpr int PA_STAGE_BYTES = 16384;
constexpr int PA_X_BYTES = PA_M * PA_D * 2;
constexpr int PA_U_BYTES = 131072;
constexpr int PA_THREADS = 640;            // warps 0-3: producer, MMA issuer, two idle; 4-11 network; 12-19 env
constexpr int PA_GROUP_WARPS = 8;          // warps of the network group and of the env group (one barrier arrival each)
constexpr uint32_t PA_COL_HB = 0, PA_COL_Z = 256, PA_COL_ACC0 = 384, PA_COL_ACC1 = 448;
constexpr int PA_N3 = 16;                  // head width on the tensor cores

struct PaSmem {
  uint64_t full[PA_STAGES], empty[PA_STAGES];
  uint64_t x_ready;        // network -> MMA: operands of the tile are in X and U
  uint64_t acc_full[2];    // MMA -> network: a 64-column accumulator is complete
  uint64_t acc_empty[2];   // network -> MMA: it has been drained (and its activations stored)
  uint64_t head_full;      // MMA -> env and network: head outputs and z complete; X and U may be rewritten
  uint64_t env_taken;      // env -> MMA: head outputs and z are in registers
  uint64_t pair_sync;      // env: the two threads of a row exchange partial norms
  float sq[2][PA_M];
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
  const int n_hb = H / PA_NB;            // 64-neuron blocks per hidden layer
  const int n_kc = H / PA_KC;            // 128-wide K chunks of layer 2

  if (tid == 0) {
    for (int s = 0; s < PA_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    mbar_init(&ctl->x_ready, PA_GROUP_WARPS);
    mbar_init(&ctl->acc_full[0], 1);
    mbar_init(&ctl->acc_full[1], 1);
    mbar_init(&ctl->acc_empty[0], PA_GROUP_WARPS);
    mbar_init(&ctl->acc_empty[1], PA_GROUP_WARPS);
    mbar_init(&ctl->head_full, 1);
    mbar_init(&ctl->env_taken, PA_GROUP_WARPS);
    mbar_init(&ctl->pair_sync, PA_GROUP_WARPS);
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
    // registers: 640 threads x 96 at launch = 61,440; 128 x 40 + 256 x 96 + 256 x 120 = 60,416 after the two changes
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- producer
      uint32_t it = 0;
      const uint32_t head_bytes = (uint32_t)PA_N3 * H * 2;
      const int n_w = n_hb * (1 + n_kc);                       // 16 KB weight chunks of the two hidden layers
      for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x) {
        for (int c = 0; c < 8 + n_w + 1; ++c, ++it) {
          const uint8_t* src;
          uint32_t bytes = PA_STAGE_BYTES;
          if (c < 8) src = reinterpret_cast<const uint8_t*>(c < 4 ? ev.lgA_hi : ev.lgA_lo) + (size_t)(c & 3) * PA_STAGE_BYTES;
          else if (c < 8 + n_w) src = reinterpret_cast<const uint8_t*>(p.wtc) + (size_t)(c - 8) * PA_STAGE_BYTES;
          else { src = reinterpret_cast<const uint8_t*>(p.wtc) + (size_t)n_w * PA_STAGE_BYTES; bytes = head_bytes; }
          const int s = it % PA_STAGES;
          if (!tc_wait(&ctl->empty[s], ((it / PA_STAGES) & 1) ^ 1, abort_flag)) goto done;
          mbar_expect_tx(&ctl->full[s], bytes);
          bulk_copy_g2s(ring + (size_t)s * PA_STAGE_BYTES, src, bytes, &ctl->full[s]);
        }
      }
    } else if (warp == 1 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      uint32_t it = 0, tiles = 0, use[2] = {0, 0};
      const uint32_t idesc64 = make_idesc(PA_NB), idesc16 = make_idesc(PA_N3), idesc_z = make_idesc_tf32(D);
      const uint32_t x_addr = smem_addr(xbuf), u_addr = smem_addr(ubuf);
      const uint32_t acc_col[2] = {PA_COL_ACC0, PA_COL_ACC1};
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tiles) {
        if (!tc_wait(&ctl->x_ready, tiles & 1, abort_flag)) goto done;
        if (tiles > 0 && !tc_wait(&ctl->env_taken, (tiles - 1) & 1, abort_flag)) goto done;
        tc_fence_after();
        // z = A s as three TF32 products: (s_hi, A_hi), (s_lo, A_hi), (s_hi, A_lo); K = 8 per instruction
        {
          const uint32_t a_sbo = (uint32_t)(D / 4) * 128u, b_sbo = (uint32_t)(32 / 4) * 128u, lo_off = (uint32_t)PA_M * D * 4;
          for (int half = 0; half < 2; ++half) {
            for (int kc = 0; kc < 4; ++kc, ++it) {
              const int s = it % PA_STAGES;
              if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
              const uint32_t b_base = smem_addr(ring + (size_t)s * PA_STAGE_BYTES);
              const uint32_t a_base = u_addr + (uint32_t)(kc * 8) * 128u;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                umma_tf32(tmem + PA_COL_Z, make_desc(a_base + j * 256u, 128u, a_sbo), make_desc(b_base + j * 256u, 128u, b_sbo),
                          idesc_z, (half | kc | j) != 0);
                if (half == 0)
                  umma_tf32(tmem + PA_COL_Z, make_desc(a_base + lo_off + j * 256u, 128u, a_sbo),
                            make_desc(b_base + j * 256u, 128u, b_sbo), idesc_z, true);
              }
              umma_commit(&ctl->empty[s]);
            }
          }
        }
        // layer 1: per 64-neuron block one chunk (64 x 128); A operand = X in shared memory
        for (int b = 0; b < n_hb; ++b, ++it) {
          const int buf = b & 1;
          if (!tc_wait(&ctl->acc_empty[buf], (use[buf] & 1) ^ 1, abort_flag)) goto done;
          tc_fence_after();
          const int s = it % PA_STAGES;
          if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
          const uint32_t b_base = smem_addr(ring + (size_t)s * PA_STAGE_BYTES);
#pragma unroll
          for (int j = 0; j < PA_KC / 16; ++j)
            umma_bf16(tmem + acc_col[buf], make_desc(x_addr + j * 256u, 128u, 2048u), make_desc(b_base + j * 256u, 128u, 2048u),
                      idesc64, j != 0);
          umma_commit(&ctl->empty[s]);
          umma_commit(&ctl->acc_full[buf]);
          ++use[buf];
        }
        // layer 2: per block H/128 chunks; A operand = h1 in tensor memory (8 columns per K = 16)
        for (int b = 0; b < n_hb; ++b) {
          const int buf = b & 1;
          if (!tc_wait(&ctl->acc_empty[buf], (use[buf] & 1) ^ 1, abort_flag)) goto done;
          tc_fence_after();
          for (int c = 0; c < n_kc; ++c, ++it) {
            if (b == 0 && c == n_kc - 1) {
              // the last columns of h1 come from the last layer-1 block, drained through the other accumulator
              if (!tc_wait(&ctl->acc_empty[1], (use[1] & 1) ^ 1, abort_flag)) goto done;
              tc_fence_after();
            }
            const int s = it % PA_STAGES;
            if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
            const uint32_t b_base = smem_addr(ring + (size_t)s * PA_STAGE_BYTES);
            const uint32_t a_col = tmem + PA_COL_HB + (uint32_t)(c * (PA_KC / 2));
#pragma unroll
            for (int j = 0; j < PA_KC / 16; ++j)
              umma_bf16_ts(tmem + acc_col[buf], a_col + (uint32_t)(j * 8), make_desc(b_base + j * 256u, 128u, 2048u), idesc64,
                           (c | j) != 0);
            umma_commit(&ctl->empty[s]);
          }
          umma_commit(&ctl->acc_full[buf]);
          ++use[buf];
        }
        // head: 16 outputs, K = H, A operand = h2 in shared memory; into the first accumulator
        {
          if (!tc_wait(&ctl->acc_empty[0], (use[0] & 1) ^ 1, abort_flag)) goto done;
          if (!tc_wait(&ctl->acc_empty[1], (use[1] & 1) ^ 1, abort_flag)) goto done;
          tc_fence_after();
          const int s = it % PA_STAGES;
          if (!tc_wait(&ctl->full[s], (it / PA_STAGES) & 1, abort_flag)) goto done;
          const uint32_t b_base = smem_addr(ring + (size_t)s * PA_STAGE_BYTES);
          const uint32_t sbo = (uint32_t)(H / 8) * 128u;
          for (int j = 0; j < H / 16; ++j)
            umma_bf16(tmem + PA_COL_ACC0, make_desc(u_addr + j * 256u, 128u, sbo), make_desc(b_base + j * 256u, 128u, sbo), idesc16,
                      j != 0);
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
    uint32_t tiles = 0, use[2] = {0, 0};
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tiles) {
      const long long row = (long long)tile * PA_M + r;
      const bool live = row < p.n;
      // this thread's half of the FP32 state row
      float4 keep[16];
      {
        const float* xr = p.x + (size_t)(live ? row : 0) * D + hsel * 64;
#pragma unroll
        for (int i = 0; i < 16; ++i) keep[i] = live ? __ldg(reinterpret_cast<const float4*>(xr + i * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      // X and U are read by the previous tile's MMAs until its head is complete
      if (tiles > 0 && !tc_wait_elect(&ctl->head_full, (tiles - 1) & 1, abort_flag)) goto done;
      {
        uint8_t* dx = xbuf + ((size_t)(r >> 3) * (D / 8)) * 128 + (r & 7) * 16;
        uint8_t* dhi = ubuf + ((size_t)(r >> 3) * (D / 4)) * 128 + (r & 7) * 16;
        uint8_t* dlo = dhi + (size_t)PA_M * D * 4;
#pragma unroll
        for (int gi = 0; gi < 8; ++gi) {
          const float4 a = keep[2 * gi], b = keep[2 * gi + 1];
          uint4 v;
          v.x = pack_bf16x2(a.x, a.y); v.y = pack_bf16x2(a.z, a.w);
          v.z = pack_bf16x2(b.x, b.y); v.w = pack_bf16x2(b.z, b.w);
          *reinterpret_cast<uint4*>(dx + (size_t)(hsel * 8 + gi) * 128) = v;
        }
#pragma unroll
        for (int gi = 0; gi < 16; ++gi) {
          const float4 sv = keep[gi];
          float4 hi, lo;
          hi.x = __uint_as_float(__float_as_uint(sv.x) & 0xFFFFE000u); lo.x = sv.x - hi.x;
          hi.y = __uint_as_float(__float_as_uint(sv.y) & 0xFFFFE000u); lo.y = sv.y - hi.y;
          hi.z = __uint_as_float(__float_as_uint(sv.z) & 0xFFFFE000u); lo.z = sv.z - hi.z;
          hi.w = __uint_as_float(__float_as_uint(sv.w) & 0xFFFFE000u); lo.w = sv.w - hi.w;
          *reinterpret_cast<float4*>(dhi + (size_t)(hsel * 16 + gi) * 128) = hi;
          *reinterpret_cast<float4*>(dlo + (size_t)(hsel * 16 + gi) * 128) = lo;
        }
      }
      fence_async_smem();
      mbar_arrive_warp(&ctl->x_ready);
      if (live) {
        // the record's observation
        const unsigned long long slot = (ev.cursor + (unsigned long long)row) % (unsigned long long)ev.C;
        float* rec = ev.ring + slot * ev.rec_words + hsel * 64;
#pragma unroll
        for (int i = 0; i < 16; ++i) *reinterpret_cast<float4*>(rec + i * 4) = keep[i];
      }
      {
        // pull the next tile's state rows towards L2 while this tile computes
        const long long nrow = (long long)(tile + (int)gridDim.x) * PA_M + r;
        if (nrow < p.n) {
          const float* xn = p.x + (size_t)nrow * D + hsel * 64;
          prefetch_l2(xn);
          prefetch_l2(xn + 32);
        }
      }
      for (int layer = 0; layer < 2; ++layer) {
        const float* bias = layer == 0 ? p.b1 : p.b2;
        for (int b = 0; b < n_hb; ++b) {
          const int buf = b & 1;
          if (!tc_wait_elect(&ctl->acc_full[buf], use[buf] & 1, abort_flag)) goto done;
          ++use[buf];
          tc_fence_after();
          const int c0 = b * PA_NB + hsel * 32;          // first of this thread's 32 columns
          uint32_t v[32];
          tmem_ld16(t_lane + (buf ? PA_COL_ACC1 : PA_COL_ACC0) + (uint32_t)(hsel * 32), v);
          tmem_ld16(t_lane + (buf ? PA_COL_ACC1 : PA_COL_ACC0) + (uint32_t)(hsel * 32 + 16), v + 16);
          tmem_ld_wait();
          uint32_t o[16];
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) {
            const float4 bb = __ldg(reinterpret_cast<const float4*>(bias + c0 + 4 * j4));
            const float f0 = fmaxf(__uint_as_float(v[4 * j4 + 0]) + bb.x, 0.f);
            const float f1 = fmaxf(__uint_as_float(v[4 * j4 + 1]) + bb.y, 0.f);
            const float f2 = fmaxf(__uint_as_float(v[4 * j4 + 2]) + bb.z, 0.f);
            const float f3 = fmaxf(__uint_as_float(v[4 * j4 + 3]) + bb.w, 0.f);
            o[2 * j4] = pack_bf16x2(f0, f1);
            o[2 * j4 + 1] = pack_bf16x2(f2, f3);
          }
          if (layer == 0) {
            tmem_st16(t_lane + PA_COL_HB + (uint32_t)(c0 / 2), o);
            tmem_st_wait();
          } else {
            uint8_t* dst = ubuf + ((size_t)(r >> 3) * (H / 8)) * 128 + (r & 7) * 16 + (size_t)(c0 / 8) * 128;
#pragma unroll
            for (int g = 0; g < 4; ++g)
              *reinterpret_cast<uint4*>(dst + (size_t)g * 128) = make_uint4(o[4 * g], o[4 * g + 1], o[4 * g + 2], o[4 * g + 3]);
            fence_async_smem();
          }
          tc_fence_before();
          mbar_arrive_warp(&ctl->acc_empty[buf]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ env warps
    asm volatile("setmaxnreg.inc.sync.aligned.u32 120;");
    const int q = warp & 3;
    const int hsel = (warp - 12) >> 2;
    const int r = q * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16);
    uint32_t tiles = 0;
    unsigned long long n_episodes = 0;
    double ret_sum = 0.0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tiles) {
      const long long row = (long long)tile * PA_M + r;
      const bool live = row < p.n;
      if (!tc_wait_elect(&ctl->head_full, tiles & 1, abort_flag)) goto done;
      tc_fence_after();
      uint32_t qraw[16], zv[64];
      tmem_ld16(t_lane + PA_COL_ACC0, qraw);
#pragma unroll
      for (int g = 0; g < 4; ++g) tmem_ld16(t_lane + PA_COL_Z + (uint32_t)(hsel * 64 + g * 16), zv + 16 * g);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive_warp(&ctl->env_taken);
      // epsilon-greedy on this row: explore iff x0 < threshold, else the first maximum
      int action;
      {
        float qv[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) qv[j] = __uint_as_float(qraw[j]) + (j < p.Aout ? __ldg(p.b3 + j) : 0.f);
        if (live && p.out && hsel == 0) {
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
        action = ((unsigned long long)w.x < ev.explore_thr) ? (int)__umulhi(w.y, (uint32_t)ev.A) : best;
      }
      const unsigned long long slot = (ev.cursor + (unsigned long long)(live ? row : 0)) % (unsigned long long)ev.C;
      float* rec = ev.ring + slot * ev.rec_words;
      // both threads of a row read the episode counters early; only one writes them at the end
      const int ep0 = live ? ev.ep_step[row] : 0;
      const float ret0 = live ? ev.ep_return[row] : 0.f;
      // s' = tanh(z + B[a]) + noise, kept in the registers that held z
      const float* Ba = ev.lgB + (size_t)action * D + hsel * 64;
      float sq = 0.f;
#pragma unroll
      for (int b4 = 0; b4 < 16; ++b4) {
        const uint4 w = stream_words(ev.seed, STREAM_NOISE, (uint32_t)(hsel * 16 + b4), (uint32_t)row, ev.t);
        const float2 z01 = box_muller_fast(w.x, w.y), z23 = box_muller_fast(w.z, w.w);
        const float4 bb = __ldg(reinterpret_cast<const float4*>(Ba + 4 * b4));
        float4 o;
        o.x = tanh_fast(__uint_as_float(zv[4 * b4 + 0]) + bb.x) + ev.noise_std * z01.x;
        o.y = tanh_fast(__uint_as_float(zv[4 * b4 + 1]) + bb.y) + ev.noise_std * z01.y;
        o.z = tanh_fast(__uint_as_float(zv[4 * b4 + 2]) + bb.z) + ev.noise_std * z23.x;
        o.w = tanh_fast(__uint_as_float(zv[4 * b4 + 3]) + bb.w) + ev.noise_std * z23.y;
        sq = fmaf(o.x, o.x, sq); sq = fmaf(o.y, o.y, sq); sq = fmaf(o.z, o.z, sq); sq = fmaf(o.w, o.w, sq);
        zv[4 * b4 + 0] = __float_as_uint(o.x); zv[4 * b4 + 1] = __float_as_uint(o.y);
        zv[4 * b4 + 2] = __float_as_uint(o.z); zv[4 * b4 + 3] = __float_as_uint(o.w);
        if (live) *reinterpret_cast<float4*>(rec + D + hsel * 64 + 4 * b4) = o;
      }
      // the two halves of a row exchange their partial squared norms (low half first in the sum)
      ctl->sq[hsel][r] = sq;
      mbar_arrive_warp(&ctl->pair_sync);
      if (!tc_wait_elect(&ctl->pair_sync, tiles & 1, abort_flag)) goto done;
      sq = ctl->sq[0][r] + ctl->sq[1][r];
      if (live) {
        const float rew = -sq / (float)D;
        int ep = ep0 + 1;
        float ep_ret = ret0 + rew;
        const int done = (sqrtf(sq) > ev.done_norm || ep >= ev.max_ep) ? 1 : 0;
        float* st = ev.state + (size_t)row * D + hsel * 64;
        if (done) {
          ep_ret = 0.f;
          ep = 0;
#pragma unroll 4
          for (int b4 = 0; b4 < 16; ++b4) {
            const uint4 w = stream_words(ev.seed, STREAM_RESET, (uint32_t)(hsel * 16 + b4), (uint32_t)row, ev.t);
            *reinterpret_cast<float4*>(st + 4 * b4) = make_float4(uniform_range(w.x, -0.1f, 0.2f), uniform_range(w.y, -0.1f, 0.2f),
                                                                  uniform_range(w.z, -0.1f, 0.2f), uniform_range(w.w, -0.1f, 0.2f));
          }
        } else {
#pragma unroll
          for (int b4 = 0; b4 < 16; ++b4)
            *reinterpret_cast<float4*>(st + 4 * b4) = make_float4(__uint_as_float(zv[4 * b4]), __uint_as_float(zv[4 * b4 + 1]),
                                                                  __uint_as_float(zv[4 * b4 + 2]), __uint_as_float(zv[4 * b4 + 3]));
        }
        if (hsel == 0) {
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
      if (blockIdx.x == 0 && tid == 12 * 32)
        ev.block_ver[(ev.cursor % (unsigned long long)ev.C) / (unsigned long long)p.n] = ev.version;
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

// FP32 blob -> BF16 chunks in the order the pipelined actor streams them.  Hidden layers: per 64-neuron block, chunks of
// 64 rows x 128 columns; element (r, k) of a chunk sits at ((r/8) * 16 + k/8) * 64 + (r%8) * 8 + k%8.  Head: one chunk of
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

}  // namespace

bool tc_pipelined_supported(int D, int H, int A) {
  return D == PA_D && H >= PA_KC && H <= 512 && H % PA_KC == 0 && A >= 1 && A <= PA_N3;
}

cudaError_t launch_pack_pipelined_weights(const float* blob, uint16_t* dst, int D, int H, int A, cudaStream_t s) {
  const size_t n = tc_weight_elems(D, H);
  pack_pipelined_weights_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(blob, dst, D, H, A);
  return cudaGetLastError();
}

cudaError_t launch_actor_tc_pipelined(const TcMlpParams& p, int sm_count, cudaStream_t s) {
  if (p.n <= 0) return cudaSuccess;
  if (!tc_pipelined_supported(p.D, p.H, p.Aout) || !p.env.fused) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)PA_X_BYTES + PA_U_BYTES + (size_t)PA_STAGES * PA_STAGE_BYTES + sizeof(PaSmem) + 64;
  cudaError_t e = cudaFuncSetAttribute(actor_tc_pipelined_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int n_tiles = (p.n + PA_M - 1) / PA_M;
  const int grid = n_tiles < sm_count ? n_tiles : sm_count;
  actor_tc_pipelined_kernel<<<grid, PA_THREADS, smem, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tj
