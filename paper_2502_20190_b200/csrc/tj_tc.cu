// BF16 tensor-core policy MLP (tcgen05.mma with TMEM accumulators) for wide networks.
//
//   out[n][A] = W3 relu(W2 relu(W1 x + b1) + b2) + b3     x: [n][D] FP32 rows,  weights BF16, accumulation FP32
//
// One thread block owns a tile of 128 rows (one row per TMEM lane) and walks tiles persistently.  Roles:
//   warp 0, one lane   producer: streams pre-tiled BF16 weight chunks from global/L2 into a shared-memory ring with
//                      bulk async copies (mbarrier complete_tx)
//   warp 1, one lane   issues tcgen05.mma (M = 128, N <= 256, K = 16) over the ring; tcgen05.commit frees ring
//                      slots and signals "accumulator full"
//   warps 2-9          (256 threads, TC_SPLIT = 2 per row, each owning half of the columns) convert the FP32 input rows to BF16 into the A-operand buffer;
//                      after each layer read the accumulator from TMEM (tcgen05.ld), add the bias, apply ReLU,
//                      round to BF16 and write the next layer's A operand; after the last layer write the outputs
// Operands use the no-swizzle K-major core-matrix layout: 8 rows x 16 bytes are contiguous (128 B), cores adjacent
// in K are 128 B apart (leading byte offset), groups of 8 rows are (K/8)*128 B apart (stride byte offset).
// Fused actor mode (linear-Gaussian env): after the head layer the same block selects the action (epsilon-greedy on the
// accumulator row), re-reads the FP32 state row, writes it as the record's observation and splits it into TF32
// high and low parts; A s then runs on the tensor cores as three TF32 products (hi*hi + lo*hi + hi*lo, FP32
// accumulation, error ~2^-21 relative per term), and the epilogue threads finish the step: + B[a], tanh, Philox
// noise, reward, done, record, reset, new state.
// Every wait is bounded: on a timeout the block raises an abort flag, records an error, frees its TMEM and leaves.
#include "tj_internal.h"
#include "tj_tc.cuh"

namespace tj {

namespace {

constexpr int TC_M = 128;        // rows per tile
constexpr int TC_KC = 32;        // K elements per weight chunk
constexpr int TC_STAGES = 5;     // ring slots
constexpr int TC_STAGE_BYTES = 256 * TC_KC * 2;   // largest chunk: 256 output rows
constexpr int TC_SPLIT = 2;         // epilogue threads per row (each owns 1/TC_SPLIT of the columns); 4 measured no faster
constexpr int TC_EPI_THREADS = 128 * TC_SPLIT;
constexpr int TC_THREADS = 64 + TC_EPI_THREADS;   // producer warp, MMA warp, 4 * TC_SPLIT epilogue warps
constexpr int TC_KEEP = 32 / TC_SPLIT;            // float4 registers holding a thread's share of a 128-wide state row
constexpr int TC_N3 = 16;        // head width on the tensor cores (outputs padded to 16)

// bytes of the A-operand buffer: the widest BF16 operand; in fused mode also the TF32 high+low state tile and
// the FP32 staging rows of the stepped state
__host__ __device__ inline size_t tc_abuf_bytes(int D, int H, bool fused) {
  size_t n = (size_t)TC_M * (D > H ? D : H) * 2;
  if (fused) {
    const size_t hl = (size_t)2 * TC_M * D * 4, st = (size_t)TC_M * (D + 4) * 4;
    if (hl > n) n = hl;
    if (st > n) n = st;
  }
  return (n + 1023) & ~(size_t)1023;
}

struct TcSmem {
  uint64_t full[TC_STAGES], empty[TC_STAGES], a_ready, acc_full, rows_done, pair_sync;
  float sq[TC_SPLIT][TC_M];
  uint32_t tmem_base;
  int abort_flag;
};

template <bool FUSED>
__global__ void __launch_bounds__(TC_THREADS, 1) mlp_bf16_tc_kernel(const TcMlpParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int D = p.D, H = p.H;
  uint8_t* abuf = smem_raw;                                          // [128][Kmax] bf16, core-matrix layout
  uint8_t* ring = abuf + tc_abuf_bytes(D, H, FUSED);                 // TC_STAGES x TC_STAGE_BYTES
  float* bias = reinterpret_cast<float*>(ring + TC_STAGES * TC_STAGE_BYTES);   // b1 [H], b2 [H], b3 [16]
  TcSmem* ctl = reinterpret_cast<TcSmem*>(bias + 2 * H + TC_N3);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_tiles = (p.n + TC_M - 1) / TC_M;
  const int n_blocks = H > 256 ? 2 : 1, NB = H / n_blocks;           // output-neuron blocks per hidden layer

  if (tid == 0) {
    for (int s = 0; s < TC_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    mbar_init(&ctl->a_ready, TC_EPI_THREADS);
    mbar_init(&ctl->acc_full, 1);
    mbar_init(&ctl->rows_done, TC_EPI_THREADS);
    mbar_init(&ctl->pair_sync, TC_EPI_THREADS);
    ctl->abort_flag = 0;
  }
  for (int i = tid; i < 2 * H + TC_N3; i += TC_THREADS) {
    float v;
    if (i < H) v = p.b1[i];
    else if (i < 2 * H) v = p.b2[i - H];
    else v = (i - 2 * H) < p.Aout ? p.b3[i - 2 * H] : 0.f;
    bias[i] = v;
  }
  __syncthreads();
  if (warp == 1) {   // one warp allocates all 512 TMEM columns (one block per SM) and publishes the base address
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&ctl->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  // chunk schedule of one tile, the same for producer and MMA issuer:
  //   layer 1: n_blocks x (D/KC) chunks of NB rows; layer 2: n_blocks x (H/KC) chunks of NB rows;
  //   layer 3: one chunk of 16 rows x H columns
  const int c1 = n_blocks * (D / TC_KC), c2 = n_blocks * (H / TC_KC), c3 = 1;
  const int ce = D / TC_KC;   // fused mode: chunks of the env matrix per TF32 pass (three passes)

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ producer
    uint32_t it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x) {
      const uint8_t* src = reinterpret_cast<const uint8_t*>(p.wtc);
      for (int c = 0; c < c1 + c2 + c3; ++c, ++it) {
        const uint32_t bytes = c < c1 + c2 ? (uint32_t)NB * TC_KC * 2 : (uint32_t)TC_N3 * H * 2;
        const int s = it % TC_STAGES;
        if (!tc_wait(&ctl->empty[s], ((it / TC_STAGES) & 1) ^ 1, abort_flag)) goto done;
        mbar_expect_tx(&ctl->full[s], bytes);
        bulk_copy_g2s(ring + (size_t)s * TC_STAGE_BYTES, src, bytes, &ctl->full[s]);
        src += bytes;
      }
      if (FUSED) {
        const uint32_t bytes = (uint32_t)D * TC_KC * 4;
        for (int c = 0; c < 2 * ce; ++c, ++it) {
          const uint8_t* esrc = reinterpret_cast<const uint8_t*>(c < ce ? p.env.lgA_hi : p.env.lgA_lo) + (size_t)(c % ce) * bytes;
          const int s = it % TC_STAGES;
          if (!tc_wait(&ctl->empty[s], ((it / TC_STAGES) & 1) ^ 1, abort_flag)) goto done;
          mbar_expect_tx(&ctl->full[s], bytes);
          bulk_copy_g2s(ring + (size_t)s * TC_STAGE_BYTES, esrc, bytes, &ctl->full[s]);
        }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    uint32_t it = 0, layer_count = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      for (int layer = 0; layer < 3; ++layer, ++layer_count) {
        const int K = layer == 0 ? D : H;
        const int nb_count = layer == 2 ? 1 : n_blocks;
        const int rows = layer == 2 ? TC_N3 : NB;
        const uint32_t idesc = make_idesc(rows);
        const uint32_t a_sbo = (uint32_t)(K / 8) * 128u, b_sbo = (uint32_t)(TC_KC / 8) * 128u;
        if (!tc_wait(&ctl->a_ready, layer_count & 1, abort_flag)) goto done;
        tc_fence_after();
        if (layer == 2) {
          // the head's weights arrive as one chunk: 16 rows x H columns
          const int s = it % TC_STAGES;
          if (!tc_wait(&ctl->full[s], (it / TC_STAGES) & 1, abort_flag)) goto done;
          const uint32_t b_base = smem_addr(ring + (size_t)s * TC_STAGE_BYTES);
          for (int j = 0; j < H / 16; ++j)
            umma_bf16(tmem, make_desc(smem_addr(abuf) + j * 256u, 128u, a_sbo), make_desc(b_base + j * 256u, 128u, a_sbo), idesc,
                      j != 0);
          umma_commit(&ctl->empty[s]);
          ++it;
        } else {
          for (int nb = 0; nb < nb_count; ++nb) {
            for (int kc = 0; kc < K / TC_KC; ++kc, ++it) {
              const int s = it % TC_STAGES;
              if (!tc_wait(&ctl->full[s], (it / TC_STAGES) & 1, abort_flag)) goto done;
              const uint32_t b_base = smem_addr(ring + (size_t)s * TC_STAGE_BYTES);
              const uint32_t a_base = smem_addr(abuf) + (uint32_t)(kc * (TC_KC / 8)) * 128u;
#pragma unroll
              for (int j = 0; j < TC_KC / 16; ++j) {
                umma_bf16(tmem + (uint32_t)(nb * NB), make_desc(a_base + j * 256u, 128u, a_sbo),
                          make_desc(b_base + j * 256u, 128u, b_sbo), idesc, (kc | j) != 0);
              }
              umma_commit(&ctl->empty[s]);    // the slot is free once these MMAs have read it
            }
          }
        }
        umma_commit(&ctl->acc_full);        // accumulator of this layer complete
      }
      if (FUSED) {
        // z = A s as three TF32 products: (s_hi, A_hi), (s_lo, A_hi), (s_hi, A_lo)
        const uint32_t idesc = make_idesc_tf32(D);
        const uint32_t a_sbo = (uint32_t)(D / 4) * 128u, b_sbo = (uint32_t)(TC_KC / 4) * 128u;
        const uint32_t lo_off = (uint32_t)TC_M * D * 4;
        if (!tc_wait(&ctl->a_ready, layer_count & 1, abort_flag)) goto done;
        tc_fence_after();
        for (int half = 0; half < 2; ++half) {       // chunks of A_hi (used with s_hi and s_lo), then of A_lo (with s_hi)
          for (int kc = 0; kc < ce; ++kc, ++it) {
            const int s = it % TC_STAGES;
            if (!tc_wait(&ctl->full[s], (it / TC_STAGES) & 1, abort_flag)) goto done;
            const uint32_t b_base = smem_addr(ring + (size_t)s * TC_STAGE_BYTES);
            const uint32_t a_base = smem_addr(abuf) + (uint32_t)(kc * (TC_KC / 4)) * 128u;
#pragma unroll
            for (int j = 0; j < TC_KC / 8; ++j) {
              umma_tf32(tmem, make_desc(a_base + j * 256u, 128u, a_sbo), make_desc(b_base + j * 256u, 128u, b_sbo), idesc,
                        (half | kc | j) != 0);
              if (half == 0)
                umma_tf32(tmem, make_desc(a_base + lo_off + j * 256u, 128u, a_sbo), make_desc(b_base + j * 256u, 128u, b_sbo),
                          idesc, true);
            }
            umma_commit(&ctl->empty[s]);
          }
        }
        umma_commit(&ctl->acc_full);
        ++layer_count;
      }
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ operand conversion and epilogues
    // 4 * TC_SPLIT warps: TC_SPLIT per TMEM lane quarter.  A row (TMEM lane) is shared by TC_SPLIT threads, each
    // owning one share of the columns / components (hsel).
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int hsel = (warp - 2) >> 2;             // which half of the columns this thread handles
    const int r = q * 32 + lane;                  // row of the tile = TMEM lane
    const uint32_t t_lane = tmem + ((uint32_t)(q * 32) << 16);
    uint32_t layer_count = 0;
    int action = 0;
    uint32_t tiles_done = 0, pair_count = 0;
    unsigned long long n_episodes = 0;
    double ret_sum = 0.0;
    float4 keep[FUSED ? TC_KEEP : 1];   // this thread's half row of the FP32 state (fused mode)
    bool have_row = false;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      const long long row = (long long)tile * TC_M + r;
      const bool live = row < p.n;
      // layer-1 A operand: this row of x, FP32 -> BF16, 8 elements (16 bytes) at a time.  In fused mode
      // (D <= 128) the thread keeps its half row in registers: it is the record's observation and the TF32
      // operand later in the tile, so the state is read from memory once.
      {
        const float* xr = p.x + (size_t)(live ? row : 0) * D;
        uint8_t* dst = abuf + ((size_t)(r >> 3) * (D / 8)) * 128 + (r & 7) * 16;
        const int g0 = hsel * (D / (8 * TC_SPLIT)), g1 = g0 + D / (8 * TC_SPLIT);
        if (FUSED && !have_row) {      // first tile of this block; later tiles were fetched during the previous env epilogue
#pragma unroll
          for (int i = 0; i < TC_KEEP; ++i) {
            keep[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (live && i < D / (4 * TC_SPLIT)) keep[i] = __ldg(reinterpret_cast<const float4*>(xr + g0 * 8 + i * 4));
          }
        }
#pragma unroll
        for (int gi = 0; gi < (FUSED ? TC_KEEP / 2 : 16 / TC_SPLIT); ++gi) {
          const int kg = g0 + gi;
          if (kg >= g1) break;
          float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
          if (FUSED) {
            lo = keep[2 * gi];
            hi = keep[2 * gi + 1];
          } else if (live) {
            lo = __ldg(reinterpret_cast<const float4*>(xr + kg * 8));
            hi = __ldg(reinterpret_cast<const float4*>(xr + kg * 8 + 4));
          }
          uint4 v;
          v.x = pack_bf16x2(lo.x, lo.y); v.y = pack_bf16x2(lo.z, lo.w);
          v.z = pack_bf16x2(hi.x, hi.y); v.w = pack_bf16x2(hi.z, hi.w);
          *reinterpret_cast<uint4*>(dst + (size_t)kg * 128) = v;
        }
      }
      fence_async_smem();
      mbar_arrive(&ctl->a_ready);
      for (int layer = 0; layer < 3; ++layer, ++layer_count) {
        if (!tc_wait_warp(&ctl->acc_full, layer_count & 1, abort_flag)) goto done;
        tc_fence_after();
        if (layer < 2) {
          // h = relu(acc + b) -> BF16 -> A operand of the next layer (K = H); 32 columns per TMEM round trip
          const float* b = bias + layer * H;
          uint8_t* dst = abuf + ((size_t)(r >> 3) * (H / 8)) * 128 + (r & 7) * 16;
          const int c_begin = hsel * (H / TC_SPLIT), c_end = c_begin + H / TC_SPLIT;
          for (int c0 = c_begin; c0 < c_end; c0 += 32) {
            uint32_t v[32];
            const bool two = c0 + 32 <= c_end;
            tmem_ld16(t_lane + (uint32_t)c0, v);
            if (two) tmem_ld16(t_lane + (uint32_t)(c0 + 16), v + 16);
            tmem_ld_wait();
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              if (hh == 1 && !two) break;
              const int cc = c0 + 16 * hh;
              uint32_t o[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float f0 = __uint_as_float(v[16 * hh + 2 * j]) + b[cc + 2 * j];
                const float f1 = __uint_as_float(v[16 * hh + 2 * j + 1]) + b[cc + 2 * j + 1];
                o[j] = pack_bf16x2_relu(f0, f1);
              }
              *reinterpret_cast<uint4*>(dst + (size_t)(cc / 8) * 128) = make_uint4(o[0], o[1], o[2], o[3]);
              *reinterpret_cast<uint4*>(dst + (size_t)(cc / 8 + 1) * 128) = make_uint4(o[4], o[5], o[6], o[7]);
            }
          }
          tc_fence_before();
          fence_async_smem();
          mbar_arrive(&ctl->a_ready);
        } else {
          uint32_t v[16];
          tmem_ld16(t_lane, v);
          tmem_ld_wait();
          tc_fence_before();
          float qv[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) qv[j] = __uint_as_float(v[j]) + bias[2 * H + j];
          if (live && p.out && hsel == 0) {
            float* o = p.out + (size_t)row * p.Aout;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (j < p.Aout) o[j] = qv[j];
          }
          if (FUSED) {
            // epsilon-greedy on this row: explore iff x0 < threshold, else the first maximum
            const uint4 w = stream_words(p.env.seed, STREAM_ACTION, 0, (uint32_t)row, p.env.t);
            int best = 0;
            float qb = qv[0];
#pragma unroll
            for (int j = 1; j < 16; ++j)
              if (j < p.env.A && qv[j] > qb) { qb = qv[j]; best = j; }
            action = ((unsigned long long)w.x < p.env.explore_thr) ? (int)__umulhi(w.y, (uint32_t)p.env.A) : best;
          }
        }
      }
      if (FUSED) {
        const TcEnvParams& ev = p.env;
        const unsigned long long slot = (ev.cursor + (unsigned long long)(live ? row : 0)) % (unsigned long long)ev.C;
        float* rec = ev.ring + slot * ev.rec_words;
        // the FP32 state row once more: record's observation, and TF32 high / low parts as the A operand
        {
          uint8_t* dst_hi = abuf + ((size_t)(r >> 3) * (D / 4)) * 128 + (r & 7) * 16;
          uint8_t* dst_lo = dst_hi + (size_t)TC_M * D * 4;
          const int g0 = hsel * (D / (4 * TC_SPLIT));
#pragma unroll
          for (int gi = 0; gi < TC_KEEP; ++gi) {
            if (gi >= D / (4 * TC_SPLIT)) break;
            const int kg = g0 + gi;
            const float4 sv = keep[gi];
            float4 hi, lo;
            hi.x = __uint_as_float(__float_as_uint(sv.x) & 0xFFFFE000u); lo.x = sv.x - hi.x;
            hi.y = __uint_as_float(__float_as_uint(sv.y) & 0xFFFFE000u); lo.y = sv.y - hi.y;
            hi.z = __uint_as_float(__float_as_uint(sv.z) & 0xFFFFE000u); lo.z = sv.z - hi.z;
            hi.w = __uint_as_float(__float_as_uint(sv.w) & 0xFFFFE000u); lo.w = sv.w - hi.w;
            *reinterpret_cast<float4*>(dst_hi + (size_t)kg * 128) = hi;
            *reinterpret_cast<float4*>(dst_lo + (size_t)kg * 128) = lo;
          }
        }
        fence_async_smem();
        mbar_arrive(&ctl->a_ready);
        // while the TF32 products run: the record's observation, then the next tile's row of the state
        if (live) {
#pragma unroll
          for (int gi = 0; gi < TC_KEEP; ++gi)
            if (gi < D / (4 * TC_SPLIT)) *reinterpret_cast<float4*>(rec + (hsel * (D / (4 * TC_SPLIT)) + gi) * 4) = keep[gi];
        }
        {
          const long long nrow = (long long)(tile + (int)gridDim.x) * TC_M + r;
          have_row = true;
#pragma unroll
          for (int i = 0; i < TC_KEEP; ++i) {
            keep[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (nrow < p.n && i < D / (4 * TC_SPLIT))
              keep[i] = __ldg(reinterpret_cast<const float4*>(p.x + (size_t)nrow * D + hsel * (D / TC_SPLIT) + i * 4));
          }
        }
        if (!tc_wait_warp(&ctl->acc_full, layer_count & 1, abort_flag)) goto done;
        ++layer_count;
        tc_fence_after();
        // s' = tanh(z + B[a]) + noise, 16 components at a time; kept in shared memory until `done` is known
        float* sb = reinterpret_cast<float*>(abuf) + (size_t)r * (D + 4);
        const float* Ba = ev.lgB + (size_t)action * D;
        float sq = 0.f;
        const int c_begin = hsel * (D / TC_SPLIT), c_end = c_begin + D / TC_SPLIT;
        for (int c0 = c_begin; c0 < c_end; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(t_lane + (uint32_t)c0, v);
          tmem_ld_wait();
          float sn[16];
#pragma unroll
          for (int b4 = 0; b4 < 4; ++b4) {
            const uint4 w = stream_words(ev.seed, STREAM_NOISE, (uint32_t)(c0 / 4 + b4), (uint32_t)row, ev.t);
            const float2 z01 = box_muller_fast(w.x, w.y), z23 = box_muller_fast(w.z, w.w);
            const float4 bb = __ldg(reinterpret_cast<const float4*>(Ba + c0 + 4 * b4));
            sn[4 * b4 + 0] = tanh_fast(__uint_as_float(v[4 * b4 + 0]) + bb.x) + ev.noise_std * z01.x;
            sn[4 * b4 + 1] = tanh_fast(__uint_as_float(v[4 * b4 + 1]) + bb.y) + ev.noise_std * z01.y;
            sn[4 * b4 + 2] = tanh_fast(__uint_as_float(v[4 * b4 + 2]) + bb.z) + ev.noise_std * z23.x;
            sn[4 * b4 + 3] = tanh_fast(__uint_as_float(v[4 * b4 + 3]) + bb.w) + ev.noise_std * z23.y;
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) sq = fmaf(sn[j], sn[j], sq);
#pragma unroll
          for (int b4 = 0; b4 < 4; ++b4) {
            const float4 o = make_float4(sn[4 * b4], sn[4 * b4 + 1], sn[4 * b4 + 2], sn[4 * b4 + 3]);
            *reinterpret_cast<float4*>(sb + c0 + 4 * b4) = o;
            if (live) *reinterpret_cast<float4*>(rec + D + c0 + 4 * b4) = o;
          }
        }
        tc_fence_before();
        // the two halves of a row exchange their partial squared norms (low half first in the sum)
        ctl->sq[hsel][r] = sq;
        // both threads of a row read the episode counters before the barrier; only one writes them after it
        const int ep0 = live ? ev.ep_step[row] : 0;
        const float ret0 = live ? ev.ep_return[row] : 0.f;
        mbar_arrive(&ctl->pair_sync);
        if (!tc_wait_warp(&ctl->pair_sync, pair_count & 1, abort_flag)) goto done;
        ++pair_count;
        sq = ctl->sq[0][r];
#pragma unroll
        for (int h2 = 1; h2 < TC_SPLIT; ++h2) sq += ctl->sq[h2][r];
        if (live) {
          const float rew = -sq / (float)D;
          int ep = ep0 + 1;
          float ep_ret = ret0 + rew;
          const int done = (sqrtf(sq) > ev.done_norm || ep >= ev.max_ep) ? 1 : 0;
          float* st = ev.state + (size_t)row * D;
          const int b_begin = hsel * (D / (4 * TC_SPLIT)), b_end = b_begin + D / (4 * TC_SPLIT);
          if (done) {
            ep_ret = 0.f;
            ep = 0;
            for (int b4 = b_begin; b4 < b_end; ++b4) {
              const uint4 w = stream_words(ev.seed, STREAM_RESET, (uint32_t)b4, (uint32_t)row, ev.t);
              *reinterpret_cast<float4*>(st + 4 * b4) = make_float4(uniform_range(w.x, -0.1f, 0.2f), uniform_range(w.y, -0.1f, 0.2f),
                                                                    uniform_range(w.z, -0.1f, 0.2f), uniform_range(w.w, -0.1f, 0.2f));
            }
          } else {
            for (int b4 = b_begin; b4 < b_end; ++b4)
              *reinterpret_cast<float4*>(st + 4 * b4) = *reinterpret_cast<const float4*>(sb + 4 * b4);
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
        // the staging rows alias the next tile's operand buffer: every row must be consumed before it is rewritten
        mbar_arrive(&ctl->rows_done);
        if (!tc_wait_warp(&ctl->rows_done, tiles_done & 1, abort_flag)) goto done;
        ++tiles_done;
      }
    }
    if (FUSED) {
      // episode statistics: one atomic pair per warp
      unsigned long long n = n_episodes;
      double rs = ret_sum;
      for (int o = 16; o > 0; o >>= 1) {
        n += __shfl_down_sync(0xffffffffu, n, o);
        rs += __shfl_down_sync(0xffffffffu, rs, o);
      }
      if (lane == 0 && n) {
        atomicAdd(&p.env.stats->episodes, n);
        atomicAdd(&p.env.stats->return_sum, rs);
      }
      if (blockIdx.x == 0 && tid == 64)
        p.env.block_ver[(p.env.cursor % (unsigned long long)p.env.C) / (unsigned long long)p.n] = p.env.version;
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

// FP32 blob -> BF16 chunks in the order the producer streams them; within a chunk of R rows x KC columns
// element (r, k) sits at ((r/8) * (KC/8) + k/8) * 64 + (r%8) * 8 + k%8.  Hidden layers: R = NB, KC = 32;
// head: one chunk with R = 16, KC = H.
__global__ void pack_tc_weights_kernel(const float* __restrict__ blob, uint16_t* __restrict__ dst, int D, int H, int A,
                                       int value_head) {
  const int n_blocks = H > 256 ? 2 : 1, NB = H / n_blocks;
  const size_t n1 = (size_t)H * D, n2 = (size_t)H * H, n3 = (size_t)TC_N3 * H;
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n1 + n2 + n3) return;
  const float* W1 = blob;
  const float* W2 = W1 + n1 + H;
  const float* W3 = W2 + n2 + H;
  const float* Wv = W3 + (size_t)A * H + A;
  size_t j = i;
  const float* W;
  int K, R, rows_total, n_off;
  if (j < n1) { W = W1; K = D; R = NB; rows_total = H; }
  else if (j < n1 + n2) { j -= n1; W = W2; K = H; R = NB; rows_total = H; }
  else { j -= n1 + n2; W = W3; K = H; R = TC_N3; rows_total = A; }
  const int KCc = W == W3 ? H : TC_KC;               // columns per chunk (the head is one chunk)
  const size_t chunk_elems = (size_t)R * KCc;
  const size_t chunk = j / chunk_elems, within = j % chunk_elems;
  const int chunks_per_block = K / KCc;
  const int nb = (int)(chunk / chunks_per_block), kc = (int)(chunk % chunks_per_block);
  n_off = nb * R;
  const int core = (int)(within / 64), in_core = (int)(within % 64);
  const int rg = core / (KCc / 8), kg = core % (KCc / 8);
  const int r = rg * 8 + in_core / 8, k = kc * KCc + kg * 8 + in_core % 8;
  const int n = n_off + r;
  float v = 0.f;
  if (n < rows_total) v = W[(size_t)n * K + k];
  else if (W == W3 && value_head && n == A) v = Wv[k];
  uint32_t u = __float_as_uint(v);
  u += 0x7FFFu + ((u >> 16) & 1u);
  dst[i] = (uint16_t)(u >> 16);
}

// TD error from precomputed Q rows: q = Qo[j][act], q' = max_a Qt[j][a]; per-block partial sums of the Huber loss
__global__ void td_from_q_kernel(const float* __restrict__ q_online, const float* __restrict__ q_target, int n, int A,
                                 const int* __restrict__ act, const float* __restrict__ rew,
                                 const int* __restrict__ done, float gamma, float kappa, float* __restrict__ td_out,
                                 float* __restrict__ huber_out, float* __restrict__ partial) {
  __shared__ float hub[16];
  const int j = blockIdx.x * 16 + threadIdx.x;
  float h = 0.f;
  if (threadIdx.x < 16 && j < n) {
    int a = act[j];
    a = a < 0 ? 0 : (a >= A ? A - 1 : a);
    const float q = q_online[(size_t)j * A + a];
    float qmax = q_target[(size_t)j * A];
    for (int i = 1; i < A; ++i) qmax = fmaxf(qmax, q_target[(size_t)j * A + i]);
    const float y = rew[j] + gamma * (done[j] ? 0.f : 1.f) * qmax;
    const float delta = y - q, ad = fabsf(delta);
    h = ad <= kappa ? 0.5f * delta * delta : kappa * (ad - 0.5f * kappa);
    if (td_out) td_out[j] = delta;
    if (huber_out) huber_out[j] = h;
  }
  if (threadIdx.x < 16) hub[threadIdx.x] = h;
  __syncthreads();
  if (threadIdx.x == 0) {
    float sum = 0.f;
    for (int i = 0; i < 16; ++i) sum += hub[i];
    partial[blockIdx.x] = sum;
  }
}

}  // namespace

bool tc_mlp_supported(int D, int H, int Aout) {
  if (D % TC_KC || H % TC_KC || D < TC_KC || H < TC_KC || H > 512 || D > 128 || Aout > TC_N3) return false;
  if (H % (16 * TC_SPLIT) || D % (8 * TC_SPLIT)) return false;   // every epilogue thread owns whole 16-column groups
  const int n_blocks = H > 256 ? 2 : 1;
  return (H / n_blocks) % 16 == 0;
}

size_t tc_weight_elems(int D, int H) { return (size_t)H * D + (size_t)H * H + (size_t)TC_N3 * H; }

cudaError_t launch_pack_tc_weights(const float* blob, uint16_t* dst, int D, int H, int A, int value_head, cudaStream_t s) {
  const size_t n = tc_weight_elems(D, H);
  pack_tc_weights_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(blob, dst, D, H, A, value_head);
  return cudaGetLastError();
}

cudaError_t launch_tc_mlp(const TcMlpParams& p, int sm_count, cudaStream_t s) {
  if (p.n <= 0) return cudaSuccess;
  const bool fused = p.env.fused != 0;
  const size_t smem = tc_abuf_bytes(p.D, p.H, fused) + (size_t)TC_STAGES * TC_STAGE_BYTES + (size_t)(2 * p.H + TC_N3) * 4 +
                      sizeof(TcSmem) + 64;
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  auto kernel = fused ? mlp_bf16_tc_kernel<true> : mlp_bf16_tc_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int n_tiles = (p.n + TC_M - 1) / TC_M;
  const int grid = n_tiles < sm_count ? n_tiles : sm_count;
  kernel<<<grid, TC_THREADS, smem, s>>>(p);
  return cudaGetLastError();
}

// the env matrix A [D][D] as TF32 high and low parts, tiled in chunks of D rows x KC columns:
// element (r, k) of chunk kc sits at ((r/8) * (KC/4) + (k%KC)/4) * 32 + (r%8) * 4 + k%4
__global__ void pack_env_matrix_kernel(const float* __restrict__ A, uint32_t* __restrict__ hi, uint32_t* __restrict__ lo, int D) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= D * D) return;
  const int chunk_elems = D * TC_KC;
  const int kc = i / chunk_elems, within = i % chunk_elems;
  const int core = within / 32, in_core = within % 32;
  const int rg = core / (TC_KC / 4), kg = core % (TC_KC / 4);
  const int r = rg * 8 + in_core / 4, k = kc * TC_KC + kg * 4 + in_core % 4;
  const float v = A[(size_t)r * D + k];
  const float h = __uint_as_float(__float_as_uint(v) & 0xFFFFE000u);
  hi[i] = __float_as_uint(h);
  lo[i] = __float_as_uint(v - h);
}

cudaError_t launch_pack_env_matrix(const float* A, uint32_t* hi, uint32_t* lo, int D, cudaStream_t s) {
  pack_env_matrix_kernel<<<(D * D + 255) / 256, 256, 0, s>>>(A, hi, lo, D);
  return cudaGetLastError();
}

bool tc_fused_supported(int D, int H, int A) {
  return tc_mlp_supported(D, H, A) && D <= 128 && D % (16 * TC_SPLIT) == 0 && A <= TC_N3 &&
         tc_abuf_bytes(D, H, true) + (size_t)TC_STAGES * TC_STAGE_BYTES + (size_t)(2 * H + TC_N3) * 4 + 256 <= 227 * 1024;
}

cudaError_t launch_td_from_q(const float* q_online, const float* q_target, int n, int A, const int* act, const float* rew,
                             const int* done, float gamma, float kappa, float* td_out, float* huber_out, float* partial,
                             cudaStream_t s) {
  td_from_q_kernel<<<(n + 15) / 16, 32, 0, s>>>(q_online, q_target, n, A, act, rew, done, gamma, kappa, td_out, huber_out,
                                                partial);
  return cudaGetLastError();
}

}  // namespace tj
