// Host-side context and the launch interface between the C ABI shell and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/tj.h"

namespace tj {

// Policy parameters as the kernels read them: every matrix transposed to [in][out_padded] so that a thread
// fetches four consecutive output neurons with one 128-bit load; the value head (if any) is column A of the
// last matrix.  All sizes in floats.
struct WeightLayout {
  int D, H, A, Aout, Hp, Ap;
  size_t off_W1t, off_b1, off_W2t, off_b2, off_W3t, off_b3, total;
};

inline int round_up4(int x) { return (x + 3) & ~3; }

inline WeightLayout make_weight_layout(int D, int H, int A, int value_head) {
  WeightLayout L;
  L.D = D; L.H = H; L.A = A; L.Aout = A + (value_head ? 1 : 0);
  L.Hp = round_up4(H);
  L.Ap = round_up4(L.Aout);
  size_t o = 0;
  auto take = [&](size_t n) { size_t r = o; o += (n + 63) & ~(size_t)63; return r; };  // 256-byte aligned parts
  L.off_W1t = take((size_t)D * L.Hp);
  L.off_b1 = take(L.Hp);
  L.off_W2t = take((size_t)H * L.Hp);
  L.off_b2 = take(L.Hp);
  L.off_W3t = take((size_t)H * L.Ap);
  L.off_b3 = take(L.Ap);
  L.total = o;
  return L;
}

struct DevStats {
  unsigned long long episodes;
  double return_sum;
  unsigned long long hist[33];
  unsigned long long max_stale;
  unsigned long long error;
};

struct ActorParams {
  int N, D, H, A, Aout, Hp, Ap, S_d, rec_words, max_ep, policy_kind;
  const float* W;  // packed weights, WeightLayout offsets below
  size_t off_W1t, off_b1, off_W2t, off_b2, off_W3t, off_b3, w_total;
  float* state;
  int* ep_step;
  float* ep_return;
  uint2 seed;
  unsigned long long explore_thr;
  long long t0;
  int n_steps;
  float* ring;
  long long C;
  unsigned long long cursor0;
  int* block_ver;
  int version;
  int T, G;
  float* seg_obs;
  int* seg_act;
  float* seg_rew;
  uint8_t* seg_done;
  float* seg_logp;
  float* seg_val;
  const float* lgAt;  // [D][Dp], transposed
  const float* lgB;   // [A][Dp]
  float lg_noise_std, lg_done_norm;
  float* dbg_logits;
  const float* logits_in;  // when set, network outputs [N][A] computed by another kernel (tensor-core path)
  DevStats* stats;
};

struct TdParams {
  int n, D, H, A, Hp, Ap;
  const float* Wonline;
  const float* Wtarget;
  size_t off_W1t, off_b1, off_W2t, off_b2, off_W3t, off_b3, w_total;
  const float* obs;
  const int* act;
  const float* rew;
  const float* next_obs;
  const int* done;
  float gamma, kappa;
  float* td_out;
  float* huber_out;
  float* loss_out;
  float* partial;  // scratch: one float per thread block
  unsigned long long* error;  // device error word of the context (a bounded wait that ran out)
};

struct SgdParams {
  int n, D, H, A;
  float* theta;                // online parameters, publish layout, updated in place
  const float* theta_target;   // target parameters, same layout
  const float* obs;
  const int* act;
  const float* rew;
  const float* next_obs;
  const int* done;
  float gamma, kappa;
  float *h1, *h2, *dh1, *dh2;  // scratch [n][H] each
  float* g;                    // scratch [n][A]: dL/dq, non-zero at the selected action only
  float* partial;              // scratch: one Huber partial sum per 16 rows
  float* grad_partial;         // scratch: per row range one partial gradient laid out like the parameter blob
  float* w2t;                  // scratch [H][H]: W2 transposed, the backward pass's operand on the older tensor-core path
  int sm_count;                // SMs of the device (sizes the row ranges of the tensor-core gradient products)
  float* wpack;                // scratch: split copies of W1, W2 (both networks) and W2^T for the tensor-core products
  int ldg;                     // row stride of g (A for the Q head, A + 1 with the value head's entry in column A)
  int value_head;              // 1: policy + value heads (PPO), theta carries Wv, bv after b3
  // PPO only
  const float* logp_old;
  const float* adv;
  const float* ret;
  float clip_eps, c_v, c_e;
  float* stat_partial;         // scratch: five partial sums per 16 rows (loss, policy, value, entropy, clipped rows)
  unsigned long long* error;   // device error word of the context (a bounded wait that ran out)
};

struct AdamParams {
  float *m, *v;               // moment blobs, same layout as theta
  float beta1, beta2, eps, c1, c2;
};

struct SampleParams {
  int B, D, N, rec_words;
  uint2 seed;
  long long k;
  long long v_learner;
  const float* ring;
  const int* elig_list;
  const int* elig_count;
  int* idx_out;
  float* obs;
  int* act;
  float* rew;
  float* next_obs;
  int* done;
  int* ver;
  DevStats* stats;
};

struct MinibatchParams {
  int n, D, hb;
  long long R, first;
  uint2 seed;
  unsigned long long shuffle_id;
  const float* seg_obs;
  const int* seg_act;
  const float* seg_logp;
  const float* adv_in;
  const float* ret_in;
  float* obs;
  int* act;
  float* logp;
  float* adv;
  float* ret;
  int* row;
};

struct TcEnvParams {
  int fused;                 // 0: network only
  int A, max_ep, rec_words, version;
  float* state;
  int* ep_step;
  float* ep_return;
  uint2 seed;
  unsigned long long explore_thr, t;
  float* ring;
  long long C;
  unsigned long long cursor;
  int* block_ver;
  const uint32_t *lgA_hi, *lgA_lo;   // env matrix, TF32 high / low parts, tiled
  const float* lgB;                  // [A][D]
  float noise_std, done_norm;
  DevStats* stats;
  float* z_scratch;                  // pipelined actor: per thread block two tiles of z, [2][32][128][4] floats
  unsigned long long slot0;          // pipelined actor: cursor mod C, the ring slot of env 0 in this step
  const uint16_t* lgA16;             // pipelined actor: scaled env matrix as FP16 high / low chunks
  const float* lgB_t;                // pipelined actor: B [A][D] times 2 log2(e)
  float z_to_t;                      // pipelined actor: accumulator of the scaled product -> 2 log2(e) * z
};

struct TcMlpParams {
  const float* x;          // [n][D] FP32 rows
  int n, D, H, Aout;
  const uint16_t* wtc;     // BF16 weight chunks in streaming order
  const float *b1, *b2, *b3;
  float* out;              // [n][Aout] (nullable in fused mode)
  unsigned long long* error;
  TcEnvParams env;
};

bool tc_mlp_supported(int D, int H, int Aout);
size_t tc_weight_elems(int D, int H);
cudaError_t launch_pack_tc_weights(const float* blob, uint16_t* dst, int D, int H, int A, int value_head, cudaStream_t s);
cudaError_t launch_tc_mlp(const TcMlpParams& p, int sm_count, cudaStream_t s);
cudaError_t launch_pack_env_matrix(const float* A, uint32_t* hi, uint32_t* lo, int D, cudaStream_t s);
bool tc_fused_supported(int D, int H, int A);
// pipelined fused actor (obs_dim 128, hidden a multiple of 128): its own weight chunk order
bool tc_pipelined_supported(int D, int H, int A);
cudaError_t launch_pack_pipelined_weights(const float* blob, uint16_t* dst, int D, int H, int A, cudaStream_t s);
cudaError_t launch_actor_tc_pipelined(const TcMlpParams& p, int sm_count, cudaStream_t s);
size_t tc_pipelined_scratch_floats();   // z scratch for the largest grid the launcher uses
size_t tc_pipelined_env_halfs();        // FP16 high / low chunks of the env matrix
float tc_pipelined_state_scale();       // power of two the state is multiplied by before its FP16 split
cudaError_t launch_pack_pipelined_env(const float* A, const float* B, float scale, int n_actions, uint16_t* dst, float* b_t,
                                      cudaStream_t s);
cudaError_t launch_td_from_q(const float* q_online, const float* q_target, int n, int A, const int* act, const float* rew,
                             const int* done, float gamma, float kappa, float* td_out, float* huber_out, float* partial,
                             cudaStream_t s);
cudaError_t launch_td_finish(const float* partial, int n_partial, int n, float* loss_out, cudaStream_t s);

// launchers (each returns the cudaGetLastError() of its launches)
cudaError_t launch_init_env(int env_kind, int N, int S_d, uint2 seed, float* state, int* ep_step, float* ep_return,
                            cudaStream_t s);
cudaError_t launch_pack_weights(const float* blob, float* dst, const WeightLayout& L, int value_head, int bf16,
                                cudaStream_t s);
cudaError_t launch_actor(int env_kind, const ActorParams& p, cudaStream_t s);
cudaError_t launch_eligible(const int* block_ver, int n_blocks, long long v_learner, long long bound, int* elig_list,
                            int* elig_count, cudaStream_t s);
cudaError_t launch_sample_gather(const SampleParams& p, cudaStream_t s);
cudaError_t launch_td(const TdParams& p, cudaStream_t s);
int td_grid(int n);
constexpr int SG_SPLITS = 32;     // at most this many row ranges per gradient product (partial sums go through scratch)
// tensor-core products of the update (csrc/tj_sgd_tc.cu): C = epilogue(A B^T), B split and laid out once per update
enum { GM_BIAS_RELU = 0, GM_BIAS = 1, GM_MASK = 2 };   // relu(acc + bias[n]) | acc + bias[n] | acc where mask[m][n] > 0, else 0
struct TcGemm {
  const float* A; int lda;      // M x K row-major, 16-byte rows
  const float* Bpack;           // B (N x K) as launch_pack_tf32_operands wrote it
  float* C; int ldc;            // M x N
  int M, N, K;
  const float* bias;            // GM_BIAS_RELU
  const float* mask; int ldm;   // GM_MASK
};
struct TcGemmBatch { TcGemm g[2]; int n; };
struct TcPackJob { const float* W; int ld; int transpose; int N, K; float* dst; };
struct TcPackJobs { TcPackJob j[6]; int n; };
// dW = Am^T Bm for Am [rows][M], Bm [rows][N]; bias_off >= 0: the column sums of Am (the bias gradient) go to that offset
struct TcWgrad { const float* Am; int lda; const float* Bm; int ldb; int M, N; int off; int bias_off; int tile_begin; };
struct TcWgradBatch { TcWgrad g[4]; int n; int n_tiles; };
bool tc_wgrad_ok(int N, int rows);
int tc_wgrad_tiles(int M, int N);
cudaError_t launch_wgrad_tc(const TcWgradBatch& batch, float* P, int count, int n_rows, int rows_per_range, int n_ranges,
                            unsigned long long* error, cudaStream_t s);
bool tc_gemm2_ok(const float* A, int lda, int M, int N, int K);
size_t tc_pack_floats(int N, int K);
cudaError_t launch_pack_tf32_operands(const TcPackJobs& jobs, cudaStream_t s);
cudaError_t launch_gemm_tc2(const TcGemmBatch& batch, int epi, unsigned long long* error, cudaStream_t s);
size_t sgd_scratch_floats(int max_rows, int D, int H);   // activations, deltas and 32 partial gradients of the blob
int sgd_partial_count(int n);
bool sgd_supported(int D, int H, int A);
cudaError_t launch_sgd_step(const SgdParams& p, float lr, const AdamParams* adam /* nullable: plain SGD */, cudaStream_t s);
int sgd_step_launches(const SgdParams& p);   // kernels one launch_sgd_step call launches (the path depends on the shape)
int ppo_step_launches(const SgdParams& p, bool with_stats);
cudaError_t launch_ppo_step(const SgdParams& p, float lr, const AdamParams* adam, float* stats_out /* device [5], nullable */,
                            cudaStream_t s);
int td_static_max_rows();
cudaError_t launch_td_static(const TdParams& p, int device, cudaStream_t s, bool* too_large);
cudaError_t launch_gae(const float* rew, const float* val, const uint8_t* done, int T, int N, float gamma, float lambda,
                       float* adv, float* ret, cudaStream_t s);
int shuffle_half_bits(long long R);
size_t normalize_scratch_doubles();
cudaError_t launch_normalize(const float* x, long long n, double eps, float* out, double* scratch, cudaStream_t s);
cudaError_t launch_segment_minibatch(const MinibatchParams& p, cudaStream_t s);
// FP32-accuracy tensor-core actor for the small envs (hidden x hidden layer as three FP16 products of split operands)
bool split_actor_supported(int env_kind, int D, int H, int Aout);
size_t split_weight_halfs(int H);
cudaError_t launch_pack_split_weights(const float* blob, int D, int H, uint16_t* dst, float* scale, cudaStream_t s);
cudaError_t launch_actor_split(int env_kind, const ActorParams& p, const uint16_t* w2parts, const float* w2scale, int sm_count,
                               cudaStream_t s);
int td_split_grid(int n);   // loss partials (one per 128 rows) of launch_td_split
cudaError_t launch_td_split(const TdParams& p, const uint16_t* parts_online, const float* scale_online, const uint16_t* parts_target,
                            const float* scale_target, cudaStream_t s);
size_t fma_rate_sink_floats(int sm_count);
double launch_fma_rate(float* sink, int sm_count, int outer, cudaStream_t s, cudaError_t* err);
cudaError_t launch_transpose_pad(const float* src, float* dst, int rows, int cols, int ld_dst, cudaStream_t s);

}  // namespace tj

struct SegSlot {
  int64_t index = -1;   // which segment number sits in the slot
  int64_t version = 0;
  int state = 0;        // 0 empty, 1 filling, 2 complete, 3 consumed or dropped
  int64_t acquired_index = -1;   // segment number handed out by the last tj_segment_acquire of this slot
};

struct tj_ctx {
  tj_config cfg;
  cudaStream_t stream;        // actor stream (and everything else while no learner stream is set)
  cudaStream_t lstream;       // learner stream: sample, gather, TD error, updates, GAE, publish
  bool two_stream;            // lstream differs from stream: the hand-overs below order the two
  // hand-overs between the streams (Sec. 3.1: dependencies I and III as asynchronous exchanges): each event is recorded
  // on one stream after the launches of a call and awaited by the other stream before the launches that depend on them
  cudaEvent_t ev_actor, ev_sample, ev_publish, ev_learner;
  bool has_actor, has_sample, has_publish, has_learner;
  int N, D, H, A, S_d, value_head, rec_words, max_ep;
  size_t n_blob;
  tj::WeightLayout wl;
  // device memory (all inside the caller's workspace)
  float* state;
  int* ep_step;
  float* ep_return;
  float* wbuf[2];       // online parameters, double buffered
  float* wtarget;
  float* blob_stage;    // staging for host blobs
  float* ring;
  int* block_ver;
  int* elig_list;
  int* elig_count;
  float* td_partial;
  double* norm_scratch;  // per-block partial sums of tj_normalize
  float* sgd_scratch;   // learner update: activations and their gradients for one minibatch (FP32 replay contexts)
  int sgd_rows;         // rows the scratch holds
  tj::DevStats* dstats;
  float* lgAt;
  float* lgB;
  float* lg_stage;
  // FP32-accuracy tensor-core actor (TJ_W_FP32_TC): W2's FP16 parts and their scales, double buffered like wbuf
  bool use_split;
  uint16_t* wsplit[2];
  float* wsplit_scale[2];
  uint16_t* wsplit_target;     // the target network's split matrix (refreshed with the target parameters)
  float* wsplit_scale_target;
  // tensor-core path (BF16 weights, supported shapes only)
  bool use_tc;
  int sm_count;
  uint16_t* wtc[2];
  uint16_t* wtc_target;
  float* logits_buf;   // [N][A]
  bool use_tc_fused;
  bool use_tc_pipelined;
  uint16_t* wtc_pipe[2];   // weight chunks in the pipelined actor's order, double buffered like wtc
  float* z_scratch;
  uint16_t* lgA16;      // pipelined actor: env matrix, FP16 high / low chunks, scaled by lg_scale
  float* lgB_t;         // pipelined actor: B times 2 log2(e)
  float z_to_t;
  uint32_t *lgA_hi, *lgA_lo;
  float* tdq[2];       // [kMaxTcTdRows][A] online / target outputs
  float *seg_obs, *seg_rew, *seg_logp, *seg_val;
  int* seg_act;
  uint8_t* seg_done;
  // host bookkeeping
  int active;           // which wbuf is the newest published
  int64_t version, k_last_sync;
  bool has_target;
  int64_t t, k;
  uint64_t cursor;
  std::vector<int32_t> h_block_ver;
  std::vector<SegSlot> seg;
  int64_t next_consume;
  tj_stats_t hs;        // host-side counters
  bool profiling;
  std::vector<cudaEvent_t> ev_pool;                  // free events
  struct Span { cudaEvent_t a, b; int cls; };
  std::vector<Span> spans;                            // recorded, not yet read
  std::string err;
};
