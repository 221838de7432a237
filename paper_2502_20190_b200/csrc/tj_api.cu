// C ABI shell: configuration checks, workspace carving, host-side bookkeeping (versions, cursor, segment
// slots, counters) and the kernel launches behind each entry point.
#include <algorithm>
#include <chrono>
#include <thread>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "tj_internal.h"

using namespace tj;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxTdRows = 1 << 20;
constexpr int kMaxTcTdRows = 1 << 16;   // rows of Q outputs the tensor-core TD path keeps in the workspace

struct Carver {
  char* base;
  size_t off = 0;
  explicit Carver(void* b) : base(static_cast<char*>(b)) {}
  template <typename T>
  T* take(size_t count) {
    off = (off + kAlign - 1) & ~(kAlign - 1);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

int env_state_dim(const tj_config& c) { return c.env_kind == TJ_ENV_LINGAUSS ? c.obs_dim : 4; }

const char* validate(const tj_config* c) {
  if (!c) return "null config";
  if (c->struct_size != sizeof(tj_config)) return "struct_size does not match this library's tj_config";
  if (c->n_envs < 1) return "n_envs must be positive";
  if (c->hidden < 1 || c->hidden > 768) return "hidden out of range (1..768: two activation tiles must fit in shared memory)";
  if (c->n_actions < 1 || c->n_actions > 64) return "n_actions out of range";
  switch (c->env_kind) {
    case TJ_ENV_CARTPOLE:
      if (c->obs_dim != 4 || c->n_actions != 2) return "CartPole needs obs_dim 4 and 2 actions";
      break;
    case TJ_ENV_ACROBOT:
      if (c->obs_dim != 6 || c->n_actions != 3) return "Acrobot needs obs_dim 6 and 3 actions";
      break;
    case TJ_ENV_LINGAUSS:
      if (c->obs_dim < 4 || c->obs_dim > 128 || c->obs_dim % 4) return "LinGauss needs obs_dim a multiple of 4, at most 128";
      if (!c->host_lg_A || !c->host_lg_B) return "LinGauss needs host_lg_A and host_lg_B";
      break;
    default:
      return "unknown env_kind";
  }
  if (c->policy_kind != TJ_POLICY_EPS_GREEDY && c->policy_kind != TJ_POLICY_CATEGORICAL) return "unknown policy_kind";
  if (c->weight_dtype != TJ_W_FP32 && c->weight_dtype != TJ_W_BF16 && c->weight_dtype != TJ_W_FP32_TC) return "unknown weight_dtype";
  if (c->weight_dtype == TJ_W_FP32_TC &&
      !split_actor_supported(c->env_kind, c->obs_dim, c->hidden, c->n_actions + (c->policy_kind == TJ_POLICY_CATEGORICAL ? 1 : 0)))
    return "TJ_W_FP32_TC needs CartPole or Acrobot and a hidden width of 64, 128, 192 or 256";
  if (!(c->epsilon >= 0.f && c->epsilon <= 1.f)) return "epsilon must lie in [0,1]";
  if (c->max_episode_steps < 0) return "max_episode_steps must not be negative";
  if (c->replay_capacity < 0) return "replay_capacity must not be negative";
  if (c->replay_capacity > 0) {
    if (c->replay_capacity % c->n_envs) return "replay_capacity must be a multiple of n_envs";
    if (c->replay_capacity > (int64_t)1 << 31) return "replay_capacity too large";
    if (c->minibatch < 1 || c->minibatch > kMaxTdRows) return "minibatch out of range";
    if (c->staleness_bound < 0 || c->warmup < 0) return "staleness_bound and warmup must not be negative";
    if (c->policy_kind != TJ_POLICY_EPS_GREEDY) return "the replay ring is used with the eps-greedy Q head";
  } else {
    if (c->rollout_len < 1 || c->n_segments < 1) return "segment mode needs rollout_len and n_segments";
    if (c->env_kind == TJ_ENV_LINGAUSS) return "segment mode is implemented for CartPole and Acrobot";
    if (c->policy_kind != TJ_POLICY_CATEGORICAL) return "segment mode is used with the categorical policy";
    if (c->staleness_bound < 0) return "staleness_bound must not be negative";
  }
  if (c->target_sync_interval < 0) return "target_sync_interval must not be negative";
  return nullptr;
}

size_t blob_floats(int D, int H, int A, int vh) {
  return (size_t)H * D + H + (size_t)H * H + H + (size_t)A * H + A + (vh ? (size_t)H + 1 : 0);
}

// one pass decides every address; base == nullptr only measures
size_t carve(tj_ctx* x, void* base) {
  const tj_config& c = x->cfg;
  Carver cv(base);
  const int N = c.n_envs, D = c.obs_dim, S_d = env_state_dim(c);
  const int vh = c.policy_kind == TJ_POLICY_CATEGORICAL;
  const WeightLayout wl = make_weight_layout(D, c.hidden, c.n_actions, vh);
  x->state = cv.take<float>((size_t)N * S_d);
  x->ep_step = cv.take<int>(N);
  x->ep_return = cv.take<float>(N);
  x->wbuf[0] = cv.take<float>(wl.total);
  x->wbuf[1] = cv.take<float>(wl.total);
  x->wtarget = cv.take<float>(wl.total);
  x->blob_stage = cv.take<float>(blob_floats(D, c.hidden, c.n_actions, vh));
  x->dstats = cv.take<DevStats>(1);
  x->td_partial = cv.take<float>((size_t)td_grid(kMaxTdRows));
  x->norm_scratch = cv.take<double>(normalize_scratch_doubles());
  if (c.replay_capacity > 0) {
    const size_t nb = (size_t)(c.replay_capacity / N);
    x->ring = cv.take<float>((size_t)c.replay_capacity * (2 * D + 4));
    x->block_ver = cv.take<int>(nb);
    x->elig_list = cv.take<int>(nb);
    x->elig_count = cv.take<int>(1);
    x->sgd_rows = 0;
    x->sgd_scratch = nullptr;
    if (c.policy_kind == TJ_POLICY_EPS_GREEDY && sgd_supported(D, c.hidden, c.n_actions)) {
      x->sgd_rows = c.minibatch;
      x->sgd_scratch = cv.take<float>(sgd_scratch_floats(c.minibatch, D, c.hidden));
    }
  } else {
    const size_t TN = (size_t)c.rollout_len * N, G = c.n_segments;
    x->seg_obs = cv.take<float>(G * TN * D);
    x->seg_act = cv.take<int>(G * TN);
    x->seg_rew = cv.take<float>(G * TN);
    x->seg_logp = cv.take<float>(G * TN);
    x->seg_val = cv.take<float>(G * ((size_t)c.rollout_len + 1) * N);
    x->seg_done = cv.take<uint8_t>(G * TN);
    x->sgd_rows = 0;
    x->sgd_scratch = nullptr;
    if (c.policy_kind == TJ_POLICY_CATEGORICAL && sgd_supported(D, c.hidden, c.n_actions + 1)) {
      x->sgd_rows = c.minibatch > 0 ? c.minibatch : 4096;
      x->sgd_scratch = cv.take<float>(sgd_scratch_floats(x->sgd_rows, D, c.hidden));
    }
  }
  if (c.env_kind == TJ_ENV_LINGAUSS) {
    x->lgAt = cv.take<float>((size_t)D * round_up4(D));
    x->lgB = cv.take<float>((size_t)c.n_actions * round_up4(D));
    x->lg_stage = cv.take<float>((size_t)D * D + (size_t)c.n_actions * D);
  }
  x->use_split = c.weight_dtype == TJ_W_FP32_TC;
  if (x->use_split) {
    for (int i = 0; i < 2; ++i) {
      x->wsplit[i] = cv.take<uint16_t>(split_weight_halfs(c.hidden));
      x->wsplit_scale[i] = cv.take<float>(2);
    }
    x->wsplit_target = cv.take<uint16_t>(split_weight_halfs(c.hidden));
    x->wsplit_scale_target = cv.take<float>(2);
  }
  x->use_tc = c.weight_dtype == TJ_W_BF16 && tc_mlp_supported(D, c.hidden, c.n_actions + vh);
  if (x->use_tc) {
    const size_t ne = tc_weight_elems(D, c.hidden);
    x->wtc[0] = cv.take<uint16_t>(ne);
    x->wtc[1] = cv.take<uint16_t>(ne);
    x->wtc_target = cv.take<uint16_t>(ne);
    x->logits_buf = cv.take<float>((size_t)N * c.n_actions);
    x->tdq[0] = cv.take<float>((size_t)kMaxTcTdRows * c.n_actions);
    x->tdq[1] = cv.take<float>((size_t)kMaxTcTdRows * c.n_actions);
  }
  x->use_tc_fused = x->use_tc && c.env_kind == TJ_ENV_LINGAUSS && c.replay_capacity > 0 && tc_fused_supported(D, c.hidden, c.n_actions);
  if (x->use_tc_fused) {
    x->lgA_hi = cv.take<uint32_t>((size_t)D * D);
    x->lgA_lo = cv.take<uint32_t>((size_t)D * D);
  }
  x->use_tc_pipelined = x->use_tc_fused && tc_pipelined_supported(D, c.hidden, c.n_actions);
  if (x->use_tc_pipelined) {
    x->wtc_pipe[0] = cv.take<uint16_t>(tc_weight_elems(D, c.hidden));
    x->wtc_pipe[1] = cv.take<uint16_t>(tc_weight_elems(D, c.hidden));
    x->z_scratch = cv.take<float>(tc_pipelined_scratch_floats());
    x->lgA16 = cv.take<uint16_t>(tc_pipelined_env_halfs());
    x->lgB_t = cv.take<float>((size_t)c.n_actions * D);
  }
  return (cv.off + kAlign - 1) & ~(kAlign - 1);
}

int fail(tj_ctx* x, int code, const char* msg) {
  if (x) x->err = msg;
  return code;
}
int cuda_fail(tj_ctx* x, cudaError_t e, const char* where) {
  if (x) x->err = std::string(where) + ": " + cudaGetErrorString(e);
  return TJ_ERR_CUDA;
}

thread_local std::string g_err;  // for failures before a context exists

// Counts the launches made inside its scope and, while profiling is on, brackets them with two events.
struct LaunchScope {
  tj_ctx* x;
  cudaEvent_t a = nullptr, b = nullptr;
  int cls;
  cudaStream_t st;
  // may_create = false: time the launches only if two pooled events are free (an entry point that must not create
  // anything skips the timing rather than make events).  on_learner: the launches go to the learner stream.
  LaunchScope(tj_ctx* ctx, int kernel_class, int n_launches, bool may_create = true, bool on_learner = false)
      : x(ctx), cls(kernel_class), st(on_learner ? ctx->lstream : ctx->stream) {
    x->hs.kernel_launches += n_launches;
    if (!x->profiling) return;
    if (!may_create && x->ev_pool.size() < 2) return;
    a = take(); b = take();
    if (a && b) cudaEventRecord(a, st);
  }
  ~LaunchScope() {
    if (!a || !b) return;
    cudaEventRecord(b, st);
    x->spans.push_back({a, b, cls});
  }
  cudaEvent_t take() {
    if (!x->ev_pool.empty()) { cudaEvent_t e = x->ev_pool.back(); x->ev_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    return cudaEventCreate(&e) == cudaSuccess ? e : nullptr;
  }
};

// reads every finished span into the per-class totals; the stream must have been synchronised
void drain_spans(tj_ctx* x) {
  for (auto& sp : x->spans) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, sp.a, sp.b) == cudaSuccess) {
      x->hs.kernel_ms[sp.cls] += ms;
      x->hs.kernel_count[sp.cls] += 1;
    }
    x->ev_pool.push_back(sp.a);
    x->ev_pool.push_back(sp.b);
  }
  x->spans.clear();
}

// ---- ordering between the actor stream and the learner stream (no-ops while they are the same stream)
void learner_waits_for_actor(tj_ctx* x) {      // the learner is about to read what actor launches wrote (ring, segments)
  if (x->two_stream && x->has_actor) cudaStreamWaitEvent(x->lstream, x->ev_actor, 0);
}
void actor_launched(tj_ctx* x) {
  if (x->two_stream) { cudaEventRecord(x->ev_actor, x->stream); x->has_actor = true; }
}
void learner_launched(tj_ctx* x) {
  if (x->two_stream) { cudaEventRecord(x->ev_learner, x->lstream); x->has_learner = true; }
}

uint64_t explore_threshold(float eps) {
  const double e = (double)eps;
  if (!(e > 0.0)) return 0;
  if (e >= 1.0) return 4294967296ull;
  return (uint64_t)std::floor(e * 4294967296.0);
}

}  // namespace

extern "C" {

int tj_query_workspace(const tj_config* cfg, size_t* bytes, size_t* align) {
  const char* why = validate(cfg);
  if (why) { g_err = why; return TJ_ERR_CONFIG; }
  if (!bytes) { g_err = "bytes is null"; return TJ_ERR_INVALID_ARG; }
  tj_ctx tmp{};
  tmp.cfg = *cfg;
  *bytes = carve(&tmp, nullptr);
  if (align) *align = kAlign;
  return TJ_OK;
}

int tj_create(const tj_config* cfg, void* workspace, size_t bytes, void* cuda_stream, tj_ctx** out) {
  if (!out) { g_err = "out is null"; return TJ_ERR_INVALID_ARG; }
  *out = nullptr;
  const char* why = validate(cfg);
  if (why) { g_err = why; return TJ_ERR_CONFIG; }
  if (!workspace) { g_err = "workspace is null"; return TJ_ERR_INVALID_ARG; }
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) { g_err = "workspace is not 256-byte aligned"; return TJ_ERR_WORKSPACE; }
  tj_ctx* x = new (std::nothrow) tj_ctx{};
  if (!x) { g_err = "out of host memory"; return TJ_ERR_INVALID_ARG; }
  x->cfg = *cfg;
  x->cfg.host_lg_A = x->cfg.host_lg_B = nullptr;
  const size_t need = carve(x, workspace);
  if (bytes < need) { delete x; g_err = "workspace smaller than tj_query_workspace reports"; return TJ_ERR_WORKSPACE; }
  x->stream = static_cast<cudaStream_t>(cuda_stream);
  x->lstream = x->stream; x->two_stream = false;
  x->ev_actor = x->ev_sample = x->ev_publish = x->ev_learner = nullptr;
  x->has_actor = x->has_sample = x->has_publish = x->has_learner = false;
  x->N = cfg->n_envs; x->D = cfg->obs_dim; x->H = cfg->hidden; x->A = cfg->n_actions;
  x->S_d = env_state_dim(*cfg);
  x->value_head = cfg->policy_kind == TJ_POLICY_CATEGORICAL;
  x->rec_words = 2 * x->D + 4;
  x->max_ep = cfg->max_episode_steps > 0 ? cfg->max_episode_steps : (cfg->env_kind == TJ_ENV_LINGAUSS ? 200 : 500);
  x->n_blob = blob_floats(x->D, x->H, x->A, x->value_head);
  x->wl = make_weight_layout(x->D, x->H, x->A, x->value_head);
  x->active = 0; x->version = 0; x->k_last_sync = 0; x->has_target = false;
  x->t = 0; x->k = 0; x->cursor = 0; x->next_consume = 0; x->profiling = false;
  std::memset(&x->hs, 0, sizeof(x->hs));
  if (cfg->replay_capacity > 0) x->h_block_ver.assign((size_t)(cfg->replay_capacity / cfg->n_envs), 0);
  else x->seg.assign((size_t)cfg->n_segments, SegSlot{});

  cudaError_t e = cudaSetDevice(cfg->device);
  if (e != cudaSuccess) { g_err = std::string("cudaSetDevice: ") + cudaGetErrorString(e); delete x; return TJ_ERR_CUDA; }
  x->sm_count = 148;
  cudaDeviceGetAttribute(&x->sm_count, cudaDevAttrMultiProcessorCount, cfg->device);
  auto bail = [&](cudaError_t err, const char* where) {
    g_err = std::string(where) + ": " + cudaGetErrorString(err);
    delete x;
    return (int)TJ_ERR_CUDA;
  };
  if ((e = cudaMemsetAsync(x->dstats, 0, sizeof(DevStats), x->stream)) != cudaSuccess) return bail(e, "memset stats");
  if (cfg->replay_capacity > 0) {
    if ((e = cudaMemsetAsync(x->block_ver, 0, sizeof(int) * x->h_block_ver.size(), x->stream)) != cudaSuccess)
      return bail(e, "memset block versions");
    if ((e = cudaMemsetAsync(x->elig_count, 0, sizeof(int), x->stream)) != cudaSuccess) return bail(e, "memset count");
  }
  if (cfg->env_kind == TJ_ENV_LINGAUSS) {
    // stage A and B as given, then transpose/pad A on the device
    const int D = x->D, Dp = round_up4(D), A = x->A;
    float* stage = x->lg_stage;
    if ((e = cudaMemcpyAsync(stage, cfg->host_lg_A, sizeof(float) * D * D, cudaMemcpyHostToDevice, x->stream)) != cudaSuccess)
      return bail(e, "copy A");
    if ((e = cudaMemcpyAsync(stage + (size_t)D * D, cfg->host_lg_B, sizeof(float) * A * D, cudaMemcpyHostToDevice, x->stream)) != cudaSuccess)
      return bail(e, "copy B");
    if ((e = launch_transpose_pad(stage, x->lgAt, D, D, Dp, x->stream)) != cudaSuccess) return bail(e, "transpose A");
    // B [A][D] is used as it is: D is a multiple of 4, so rows are already 16-byte aligned
    if ((e = cudaMemcpyAsync(x->lgB, stage + (size_t)D * D, sizeof(float) * A * D, cudaMemcpyDeviceToDevice, x->stream)) != cudaSuccess)
      return bail(e, "copy B to its place");
    if (x->use_tc_fused && (e = launch_pack_env_matrix(stage, x->lgA_hi, x->lgA_lo, D, x->stream)) != cudaSuccess)
      return bail(e, "tile env matrix");
    if (x->use_tc_pipelined) {
      // FP16 split of the matrix: a power-of-two scale puts its largest entry in [1024, 2048), well inside FP16's range,
      // so that the low parts of all but the tiniest entries are normal numbers
      float amax = 0.f;
      for (size_t i = 0; i < (size_t)D * D; ++i) amax = std::max(amax, std::fabs(cfg->host_lg_A[i]));
      int ea = 0;
      if (amax > 0.f && std::isfinite(amax)) ea = 10 - (int)std::floor(std::log2((double)amax));
      ea = std::min(std::max(ea, -24), 24);
      const float scale = std::ldexp(1.0f, ea);
      x->z_to_t = 2.88539008177792681472f / (tc_pipelined_state_scale() * scale);
      if ((e = launch_pack_pipelined_env(stage, stage + (size_t)D * D, scale, A, x->lgA16, x->lgB_t, x->stream)) != cudaSuccess)
        return bail(e, "split env matrix");
    }
    if ((e = cudaStreamSynchronize(x->stream)) != cudaSuccess) return bail(e, "sync after LinGauss set-up");
  }
  const uint2 seed = make_uint2((uint32_t)cfg->seed, (uint32_t)(cfg->seed >> 32));
  if ((e = launch_init_env(cfg->env_kind, x->N, x->S_d, seed, x->state, x->ep_step, x->ep_return, x->stream)) != cudaSuccess)
    return bail(e, "init envs");
  *out = x;
  return TJ_OK;
}

int tj_destroy(tj_ctx* ctx) {
  if (!ctx) return TJ_ERR_INVALID_ARG;
  cudaStreamSynchronize(ctx->stream);
  if (ctx->two_stream) cudaStreamSynchronize(ctx->lstream);
  drain_spans(ctx);
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : {ctx->ev_actor, ctx->ev_sample, ctx->ev_publish, ctx->ev_learner})
    if (e) cudaEventDestroy(e);
  delete ctx;
  return TJ_OK;
}

int tj_set_learner_stream(tj_ctx* x, void* cuda_stream) {
  if (!x) return TJ_ERR_INVALID_ARG;
  cudaStream_t ls = static_cast<cudaStream_t>(cuda_stream);
  // everything enqueued so far is ordered before the switch
  cudaError_t e = cudaStreamSynchronize(x->stream);
  if (e == cudaSuccess && x->two_stream) e = cudaStreamSynchronize(x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "set learner stream: synchronise");
  if (ls == x->stream || !cuda_stream) {
    x->lstream = x->stream; x->two_stream = false;
    x->has_actor = x->has_sample = x->has_publish = x->has_learner = false;
    return TJ_OK;
  }
  for (cudaEvent_t* ev : {&x->ev_actor, &x->ev_sample, &x->ev_publish, &x->ev_learner})
    if (!*ev && (e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(x, e, "set learner stream: events");
  x->lstream = ls; x->two_stream = true;
  x->has_actor = x->has_sample = x->has_publish = x->has_learner = false;
  return TJ_OK;
}

int tj_wait(tj_ctx* x, int32_t which, int32_t timeout_ms) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (which < 0 || which > 1 || timeout_ms < 0) return fail(x, TJ_ERR_INVALID_ARG, "which must be 0 (actor stream) or 1 (learner stream), timeout_ms >= 0");
  cudaStream_t st = which == 0 ? x->stream : x->lstream;
  const auto t0 = std::chrono::steady_clock::now();
  for (;;) {
    const cudaError_t q = cudaStreamQuery(st);
    if (q == cudaSuccess) return TJ_OK;
    if (q != cudaErrorNotReady) return cuda_fail(x, q, "wait");
    const auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
    if (ms >= timeout_ms) return fail(x, TJ_ERR_TIMEOUT, which == 0 ? "the actor stream has not drained within the time limit" : "the learner stream has not drained within the time limit");
    std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
}

int tj_set_profiling(tj_ctx* x, int32_t on) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (on && !x->profiling) {
    cudaStreamSynchronize(x->stream);
    if (x->two_stream) cudaStreamSynchronize(x->lstream);
    drain_spans(x);
    for (int i = 0; i < TJ_KERNEL_CLASSES; ++i) { x->hs.kernel_ms[i] = 0.0; x->hs.kernel_count[i] = 0; }
  }
  x->profiling = on != 0;
  return TJ_OK;
}

int tj_publish_weights(tj_ctx* x, const void* blob, size_t nbytes, int32_t on_device, int64_t* version_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (!blob) return fail(x, TJ_ERR_INVALID_ARG, "blob is null");
  if (nbytes != x->n_blob * sizeof(float)) return fail(x, TJ_ERR_INVALID_ARG, "blob size does not match the configured network");
  cudaError_t e;
  // the buffer about to be rewritten may still be read by actor launches that are in flight
  learner_waits_for_actor(x);
  const float* src = static_cast<const float*>(blob);
  if (!on_device) {
    if ((e = cudaMemcpyAsync(x->blob_stage, blob, nbytes, cudaMemcpyHostToDevice, x->lstream)) != cudaSuccess)
      return cuda_fail(x, e, "publish: host to device copy");
    src = x->blob_stage;
  }
  LaunchScope scope(x, TJ_K_PUBLISH, x->use_tc_pipelined ? 3 : (x->use_tc ? 2 : (x->use_split ? 2 : 1)), true, true);
  const int next = x->active ^ 1;
  float* dst = x->version == 0 ? x->wbuf[x->active] : x->wbuf[next];
  if ((e = launch_pack_weights(src, dst, x->wl, x->value_head, x->cfg.weight_dtype == TJ_W_BF16, x->lstream)) != cudaSuccess)
    return cuda_fail(x, e, "publish: repack");
  if (x->use_split) {
    const int slot = x->version == 0 ? x->active : next;
    if ((e = launch_pack_split_weights(src, x->D, x->H, x->wsplit[slot], x->wsplit_scale[slot], x->lstream)) != cudaSuccess)
      return cuda_fail(x, e, "publish: split of the hidden x hidden matrix");
  }
  uint16_t* dst_tc = nullptr;
  if (x->use_tc) {
    dst_tc = x->version == 0 ? x->wtc[x->active] : x->wtc[next];
    if ((e = launch_pack_tc_weights(src, dst_tc, x->D, x->H, x->A, x->value_head, x->lstream)) != cudaSuccess)
      return cuda_fail(x, e, "publish: tensor-core repack");
    if (x->use_tc_pipelined &&
        (e = launch_pack_pipelined_weights(src, x->version == 0 ? x->wtc_pipe[x->active] : x->wtc_pipe[next], x->D, x->H, x->A,
                                           x->lstream)) != cudaSuccess)
      return cuda_fail(x, e, "publish: tensor-core repack (pipelined actor)");
  }
  if (x->version != 0) x->active = next;
  x->version += 1;
  if (!x->has_target || (x->cfg.target_sync_interval > 0 && x->k - x->k_last_sync >= x->cfg.target_sync_interval)) {
    if ((e = cudaMemcpyAsync(x->wtarget, dst, x->wl.total * sizeof(float), cudaMemcpyDeviceToDevice, x->lstream)) != cudaSuccess)
      return cuda_fail(x, e, "publish: target refresh");
    if (x->use_split) {
      const int slot = x->active;
      if ((e = cudaMemcpyAsync(x->wsplit_target, x->wsplit[slot], split_weight_halfs(x->H) * sizeof(uint16_t), cudaMemcpyDeviceToDevice,
                               x->lstream)) != cudaSuccess ||
          (e = cudaMemcpyAsync(x->wsplit_scale_target, x->wsplit_scale[slot], 2 * sizeof(float), cudaMemcpyDeviceToDevice, x->lstream)) !=
              cudaSuccess)
        return cuda_fail(x, e, "publish: target refresh (split matrix)");
    }
    if (x->use_tc && (e = cudaMemcpyAsync(x->wtc_target, dst_tc, tc_weight_elems(x->D, x->H) * sizeof(uint16_t),
                                          cudaMemcpyDeviceToDevice, x->lstream)) != cudaSuccess)
      return cuda_fail(x, e, "publish: target refresh (tensor-core weights)");
    x->has_target = true;
    x->k_last_sync = x->k;
  }
  if (x->two_stream) {   // the next actor call reads the new parameters: it waits for this
    cudaEventRecord(x->ev_publish, x->lstream);
    x->has_publish = true;
  }
  if (version_out) *version_out = x->version;
  return TJ_OK;
}

int tj_actor_step(tj_ctx* x, int32_t n_steps, float* dbg_logits) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (n_steps < 0) return fail(x, TJ_ERR_INVALID_ARG, "n_steps is negative");
  if (x->version == 0) return fail(x, TJ_ERR_NO_WEIGHTS, "actor called before the first publish");
  if (n_steps == 0) return TJ_OK;
  if (x->two_stream) {
    // newest published parameters; the sampler has finished with the ring blocks this call may overwrite; in segment
    // mode a slot is restarted only after the learner's calls on its last segment have been passed
    if (x->has_publish) cudaStreamWaitEvent(x->stream, x->ev_publish, 0);
    if (x->has_sample) cudaStreamWaitEvent(x->stream, x->ev_sample, 0);
    if (x->cfg.replay_capacity == 0 && x->has_learner) cudaStreamWaitEvent(x->stream, x->ev_learner, 0);
  }
  const tj_config& c = x->cfg;
  const bool on_policy = c.replay_capacity == 0;
  ActorParams p{};
  p.N = x->N; p.D = x->D; p.H = x->H; p.A = x->A; p.Aout = x->wl.Aout; p.Hp = x->wl.Hp; p.Ap = x->wl.Ap;
  p.S_d = x->S_d; p.rec_words = x->rec_words; p.max_ep = x->max_ep; p.policy_kind = c.policy_kind;
  p.W = x->wbuf[x->active];
  p.off_W1t = x->wl.off_W1t; p.off_b1 = x->wl.off_b1; p.off_W2t = x->wl.off_W2t; p.off_b2 = x->wl.off_b2;
  p.off_W3t = x->wl.off_W3t; p.off_b3 = x->wl.off_b3; p.w_total = x->wl.total;
  p.state = x->state; p.ep_step = x->ep_step; p.ep_return = x->ep_return;
  p.seed = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
  p.explore_thr = explore_threshold(c.epsilon);
  p.t0 = x->t; p.n_steps = n_steps;
  p.ring = x->ring; p.C = c.replay_capacity; p.cursor0 = x->cursor; p.block_ver = x->block_ver;
  p.version = (int)x->version;
  p.T = c.rollout_len; p.G = c.n_segments;
  p.seg_obs = x->seg_obs; p.seg_act = x->seg_act; p.seg_rew = x->seg_rew; p.seg_done = x->seg_done;
  p.seg_logp = x->seg_logp; p.seg_val = x->seg_val;
  p.lgAt = x->lgAt; p.lgB = x->lgB; p.lg_noise_std = c.lg_noise_std; p.lg_done_norm = c.lg_done_norm;
  p.dbg_logits = dbg_logits; p.stats = x->dstats;
  cudaError_t e = cudaSuccess;
  if (x->use_tc && c.env_kind == TJ_ENV_LINGAUSS) {
    // network on the tensor cores, then the env/selection/insert kernel reads its outputs; one pair per step
    const float* W = x->wbuf[x->active];
    for (int i = 0; i < n_steps && e == cudaSuccess; ++i) {
      TcMlpParams t{};
      t.x = x->state; t.n = x->N; t.D = x->D; t.H = x->H; t.Aout = x->A;
      t.wtc = x->wtc[x->active];
      t.b1 = W + x->wl.off_b1; t.b2 = W + x->wl.off_b2; t.b3 = W + x->wl.off_b3;
      t.out = x->logits_buf; t.error = &x->dstats->error;
      if (x->use_tc_fused) {
        // one kernel per step: network, selection, A s on the tensor cores, env epilogue, insert
        t.out = dbg_logits ? dbg_logits + (size_t)i * x->N * x->A : nullptr;
        TcEnvParams& ev = t.env;
        ev.fused = 1; ev.A = x->A; ev.max_ep = x->max_ep; ev.rec_words = x->rec_words; ev.version = (int)x->version;
        ev.state = x->state; ev.ep_step = x->ep_step; ev.ep_return = x->ep_return;
        ev.seed = p.seed; ev.explore_thr = p.explore_thr; ev.t = (unsigned long long)(x->t + i);
        ev.ring = x->ring; ev.C = c.replay_capacity; ev.cursor = x->cursor + (uint64_t)i * x->N; ev.block_ver = x->block_ver;
        ev.lgA_hi = x->lgA_hi; ev.lgA_lo = x->lgA_lo; ev.lgB = x->lgB;
        ev.noise_std = c.lg_noise_std; ev.done_norm = c.lg_done_norm; ev.stats = x->dstats;
        LaunchScope scope(x, TJ_K_ACTOR_FUSED, 1);
        if (x->use_tc_pipelined) {
          t.wtc = x->wtc_pipe[x->active];
          ev.z_scratch = x->z_scratch;
          ev.slot0 = ev.cursor % (unsigned long long)c.replay_capacity;
          ev.lgA16 = x->lgA16; ev.lgB_t = x->lgB_t; ev.z_to_t = x->z_to_t;
          e = launch_actor_tc_pipelined(t, x->sm_count, x->stream);
        } else {
          e = launch_tc_mlp(t, x->sm_count, x->stream);
        }
        continue;
      }
      {
        LaunchScope scope(x, TJ_K_MLP_TENSOR, 1);
        e = launch_tc_mlp(t, x->sm_count, x->stream);
      }
      if (e != cudaSuccess) break;
      ActorParams q = p;
      q.n_steps = 1; q.t0 = x->t + i; q.cursor0 = x->cursor + (uint64_t)i * x->N;
      q.logits_in = x->logits_buf;
      q.dbg_logits = dbg_logits ? dbg_logits + (size_t)i * x->N * x->A : nullptr;
      LaunchScope scope(x, TJ_K_ENV, 1);
      e = launch_actor(c.env_kind, q, x->stream);
    }
  } else if (x->use_split) {
    LaunchScope scope(x, TJ_K_ACTOR_FUSED, 1);
    e = launch_actor_split(c.env_kind, p, x->wsplit[x->active], x->wsplit_scale[x->active], x->sm_count, x->stream);
  } else {
    LaunchScope scope(x, TJ_K_ACTOR_FUSED, 1);
    e = launch_actor(c.env_kind, p, x->stream);
  }
  if (e != cudaSuccess) return cuda_fail(x, e, "actor step");
  actor_launched(x);
  // host mirror of what the kernel does to versions, cursor and segment slots
  for (int i = 0; i < n_steps; ++i) {
    if (on_policy) {
      const int64_t g = x->t / c.rollout_len;
      const int pos = (int)(x->t % c.rollout_len);
      SegSlot& sl = x->seg[(size_t)(g % c.n_segments)];
      if (pos == 0) {
        if (sl.state == 2) x->hs.dropped_overwritten += (int64_t)c.rollout_len * x->N;
        sl.state = 1; sl.index = g; sl.version = x->version;
      }
      if (pos == c.rollout_len - 1) sl.state = 2;
    } else {
      x->h_block_ver[(size_t)((x->cursor % (uint64_t)c.replay_capacity) / (uint64_t)x->N)] = (int32_t)x->version;
      x->cursor += (uint64_t)x->N;
    }
    x->t += 1;
  }
  x->hs.produced += (int64_t)n_steps * x->N;
  x->hs.actor_steps += n_steps;
  return TJ_OK;
}

int tj_replay_sample(tj_ctx* x, int32_t staleness_bound, int32_t* idx_out, const tj_batch* out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  const tj_config& c = x->cfg;
  if (c.replay_capacity == 0) return fail(x, TJ_ERR_INVALID_ARG, "no replay ring in segment mode");
  if (!out || !out->obs || !out->act || !out->rew || !out->next_obs || !out->done || !out->ver)
    return fail(x, TJ_ERR_INVALID_ARG, "batch arrays must not be null");
  if (out->n != c.minibatch) return fail(x, TJ_ERR_INVALID_ARG, "batch.n must equal the configured minibatch");
  if (x->version == 0) return fail(x, TJ_ERR_NO_WEIGHTS, "sample called before the first publish");
  const int64_t S = staleness_bound >= 0 ? staleness_bound : c.staleness_bound;
  const int64_t valid = (int64_t)std::min<uint64_t>(x->cursor, (uint64_t)c.replay_capacity);
  if (valid < c.warmup) return fail(x, TJ_ERR_WARMUP, "fewer resident records than warmup");
  const int n_blocks = (int)(valid / x->N);
  int64_t n_elig = 0;
  for (int b = 0; b < n_blocks; ++b)
    if (x->version - (int64_t)x->h_block_ver[(size_t)b] <= S) ++n_elig;
  if (n_elig == 0) {
    x->hs.starved_calls += 1;
    return fail(x, TJ_ERR_STARVED, "no resident record within the staleness bound");
  }
  if ((uint64_t)n_elig * (uint64_t)x->N > 0xFFFFFFFFull) return fail(x, TJ_ERR_UNSUPPORTED, "eligible set too large");
  learner_waits_for_actor(x);
  LaunchScope scope(x, TJ_K_SAMPLE, 2, true, true);
  cudaError_t e = launch_eligible(x->block_ver, n_blocks, x->version, S, x->elig_list, x->elig_count, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "eligible list");
  SampleParams p{};
  p.B = c.minibatch; p.D = x->D; p.N = x->N; p.rec_words = x->rec_words;
  p.seed = make_uint2((uint32_t)c.seed, (uint32_t)(c.seed >> 32));
  p.k = x->k; p.v_learner = x->version;
  p.ring = x->ring; p.elig_list = x->elig_list; p.elig_count = x->elig_count;
  p.idx_out = idx_out;
  p.obs = out->obs; p.act = out->act; p.rew = out->rew; p.next_obs = out->next_obs; p.done = out->done; p.ver = out->ver;
  p.stats = x->dstats;
  if ((e = launch_sample_gather(p, x->lstream)) != cudaSuccess) return cuda_fail(x, e, "sample and gather");
  if (x->two_stream) { cudaEventRecord(x->ev_sample, x->lstream); x->has_sample = true; }
  x->k += 1;
  x->hs.learner_steps += 1;
  x->hs.consumed += c.minibatch;
  x->hs.dropped_stale += valid - n_elig * x->N;
  return TJ_OK;
}

namespace {
// checks shared by the two TD-error entry points; 0 = fine
int td_check(tj_ctx* x, const tj_batch* b) {
  if (!b || !b->obs || !b->act || !b->rew || !b->next_obs || !b->done) return fail(x, TJ_ERR_INVALID_ARG, "batch arrays must not be null");
  if (b->n < 1) return fail(x, TJ_ERR_INVALID_ARG, "batch.n must be positive");
  if (x->cfg.policy_kind != TJ_POLICY_EPS_GREEDY) return fail(x, TJ_ERR_UNSUPPORTED, "TD error needs the Q head");
  if (x->version == 0 || !x->has_target) return fail(x, TJ_ERR_NO_WEIGHTS, "TD error called before the first publish");
  return TJ_OK;
}

TdParams td_params(const tj_ctx* x, const tj_batch* b, float* td_out, float* huber_out, float* loss_mean_out, float* partial) {
  TdParams p{};
  p.n = b->n; p.D = x->D; p.H = x->H; p.A = x->A; p.Hp = x->wl.Hp; p.Ap = x->wl.Ap;
  p.Wonline = x->wbuf[x->active]; p.Wtarget = x->wtarget;
  p.off_W1t = x->wl.off_W1t; p.off_b1 = x->wl.off_b1; p.off_W2t = x->wl.off_W2t; p.off_b2 = x->wl.off_b2;
  p.off_W3t = x->wl.off_W3t; p.off_b3 = x->wl.off_b3; p.w_total = x->wl.total;
  p.obs = b->obs; p.act = b->act; p.rew = b->rew; p.next_obs = b->next_obs; p.done = b->done;
  p.gamma = x->cfg.gamma; p.kappa = x->cfg.huber_delta;
  p.td_out = td_out; p.huber_out = huber_out; p.loss_out = loss_mean_out; p.partial = partial;
  p.error = &x->dstats->error;
  return p;
}
}  // namespace

int tj_td_error(tj_ctx* x, const tj_batch* b, float* td_out, float* huber_out, float* loss_mean_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (int st = td_check(x, b)) return st;
  if (b->n > kMaxTdRows) return fail(x, TJ_ERR_INVALID_ARG, "batch.n out of range");
  const TdParams p = td_params(x, b, td_out, huber_out, loss_mean_out, x->td_partial);
  cudaError_t e;
  if (x->use_tc) {
    // per chunk of at most kMaxTcTdRows rows (what the Q-value buffers hold): two tensor-core forwards (online on obs,
    // target on next_obs), then the elementwise TD/Huber pass.  The chunk length is a multiple of the 16 rows one
    // partial sum covers, so the partial sums lie exactly as they would for a single pass.
    for (int r0 = 0; r0 < b->n; r0 += kMaxTcTdRows) {
      const int rows = std::min(kMaxTcTdRows, b->n - r0);
      for (int which = 0; which < 2; ++which) {
        const float* W = which == 0 ? x->wbuf[x->active] : x->wtarget;
        TcMlpParams t{};
        t.x = (which == 0 ? b->obs : b->next_obs) + (size_t)r0 * x->D; t.n = rows; t.D = x->D; t.H = x->H; t.Aout = x->A;
        t.wtc = which == 0 ? x->wtc[x->active] : x->wtc_target;
        t.b1 = W + x->wl.off_b1; t.b2 = W + x->wl.off_b2; t.b3 = W + x->wl.off_b3;
        t.out = x->tdq[which]; t.error = &x->dstats->error;
        LaunchScope scope(x, TJ_K_MLP_TENSOR, 1, true, true);
        if ((e = launch_tc_mlp(t, x->sm_count, x->lstream)) != cudaSuccess) return cuda_fail(x, e, "TD error (tensor-core forward)");
      }
      LaunchScope scope(x, TJ_K_TD, 1, true, true);
      if ((e = launch_td_from_q(x->tdq[0], x->tdq[1], rows, x->A, b->act + r0, b->rew + r0, b->done + r0, p.gamma, p.kappa,
                                td_out ? td_out + r0 : nullptr, huber_out ? huber_out + r0 : nullptr,
                                x->td_partial + r0 / 16, x->lstream)) != cudaSuccess)
        return cuda_fail(x, e, "TD error (elementwise)");
    }
    if (loss_mean_out) {
      LaunchScope scope(x, TJ_K_TD, 1, true, true);
      if ((e = launch_td_finish(x->td_partial, td_grid(b->n), b->n, loss_mean_out, x->lstream)) != cudaSuccess)
        return cuda_fail(x, e, "TD error (loss reduction)");
    }
    learner_launched(x);
    return TJ_OK;
  }
  if (x->use_split && x->cfg.replay_capacity > 0 && x->A <= 4) {
    // weight mode TJ_W_FP32_TC: both forwards with the hidden x hidden layer on the tensor cores, like the actor's
    LaunchScope scope(x, TJ_K_TD, loss_mean_out ? 2 : 1, true, true);
    e = launch_td_split(p, x->wsplit[x->active], x->wsplit_scale[x->active], x->wsplit_target, x->wsplit_scale_target, x->lstream);
    if (e == cudaSuccess && loss_mean_out) e = launch_td_finish(x->td_partial, td_split_grid(b->n), b->n, loss_mean_out, x->lstream);
    if (e != cudaSuccess) return cuda_fail(x, e, "TD error (split-operand tensor-core forward)");
    learner_launched(x);
    return TJ_OK;
  }
  LaunchScope scope(x, TJ_K_TD, loss_mean_out ? 2 : 1, true, true);
  e = launch_td(p, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "TD error");
  learner_launched(x);
  return TJ_OK;
}

int tj_td_error_static(tj_ctx* x, const tj_batch* b, float* td_out, float* huber_out, float* loss_mean_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (int st = td_check(x, b)) return st;
  if (b->n > td_static_max_rows()) {
    char msg[160];
    std::snprintf(msg, sizeof(msg), "tj_td_error_static takes at most %d rows per call (got %d); use tj_td_error or split the batch",
                  td_static_max_rows(), b->n);
    return fail(x, TJ_ERR_INVALID_ARG, msg);
  }
  const TdParams p = td_params(x, b, td_out, huber_out, loss_mean_out, nullptr);
  bool too_large = false;
  LaunchScope scope(x, TJ_K_TD, loss_mean_out ? 2 : 1, /*may_create=*/false, true);
  cudaError_t e = launch_td_static(p, x->cfg.device, x->lstream, &too_large);
  if (too_large) return fail(x, TJ_ERR_INVALID_ARG, "tj_td_error_static: batch too large for the library's scratch");
  if (e == cudaErrorInvalidDevice) return fail(x, TJ_ERR_INVALID_ARG, "tj_td_error_static: the context's device must be the current device");
  if (e != cudaSuccess) return cuda_fail(x, e, "TD error (library scratch)");
  learner_launched(x);
  return TJ_OK;
}

namespace {
// h1, h2, dh1, dh2 [rows][H] | g [rows][17] | loss partials | PPO statistic partials | W2^T [H][H] | gradient partial sums
void lay_out_update_scratch(const tj_ctx* x, tj::SgdParams& p) {
  const size_t rows = ((size_t)x->sgd_rows + 15) / 16 * 16, RH = rows * (size_t)x->H;
  p.h1 = x->sgd_scratch; p.h2 = p.h1 + RH; p.dh1 = p.h2 + RH; p.dh2 = p.dh1 + RH;
  p.g = p.dh2 + RH;
  p.partial = p.g + rows * 17;
  p.stat_partial = p.partial + rows / 16 + 8;
  p.w2t = p.stat_partial + 5 * (rows / 16) + 8;
  p.w2t += (4 - ((reinterpret_cast<uintptr_t>(p.w2t) / sizeof(float)) & 3)) & 3;   // 16-byte rows for the vector loads
  p.grad_partial = p.w2t + (size_t)x->H * x->H;
  {
    // after the partial gradients: split weight copies for the tensor-core products, 128-byte aligned for the bulk copies
    const size_t blob = (size_t)x->H * x->D + x->H + (size_t)x->H * x->H + x->H + 17 * (size_t)x->H + 17;
    float* w = p.grad_partial + (size_t)tj::SG_SPLITS * blob;
    w += (32 - ((reinterpret_cast<uintptr_t>(w) / sizeof(float)) & 31)) & 31;
    p.wpack = w;
    p.sm_count = x->sm_count;
  }
}

int learner_update(tj_ctx* x, const tj_batch* b, float lr, float* theta, const float* theta_target, const tj::AdamParams* adam,
                   float* loss_mean_out) {
  if (!b || !b->obs || !b->act || !b->rew || !b->next_obs || !b->done) return fail(x, TJ_ERR_INVALID_ARG, "batch arrays must not be null");
  if (!theta || !theta_target) return fail(x, TJ_ERR_INVALID_ARG, "parameter blobs must not be null");
  if (theta == theta_target) return fail(x, TJ_ERR_INVALID_ARG, "theta and theta_target must be different buffers");
  if (!(lr >= 0.f)) return fail(x, TJ_ERR_INVALID_ARG, "lr must not be negative");
  if (!x->sgd_scratch || x->cfg.policy_kind != TJ_POLICY_EPS_GREEDY || x->cfg.replay_capacity <= 0)
    return fail(x, TJ_ERR_UNSUPPORTED, "the learner update is implemented for replay contexts with the Q head");
  if (b->n < 1 || b->n > x->sgd_rows) return fail(x, TJ_ERR_INVALID_ARG, "batch.n must be between 1 and the configured minibatch");
  SgdParams p{};
  p.n = b->n; p.D = x->D; p.H = x->H; p.A = x->A;
  p.theta = theta; p.theta_target = theta_target;
  p.obs = b->obs; p.act = b->act; p.rew = b->rew; p.next_obs = b->next_obs; p.done = b->done;
  p.gamma = x->cfg.gamma; p.kappa = x->cfg.huber_delta;
  lay_out_update_scratch(x, p);
  p.ldg = x->A; p.value_head = 0;
  p.error = &x->dstats->error;
  LaunchScope scope(x, TJ_K_SGD, tj::sgd_step_launches(p) + (loss_mean_out ? 1 : 0), true, true);
  cudaError_t e = launch_sgd_step(p, lr, adam, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "learner update");
  if (loss_mean_out && (e = launch_td_finish(p.partial, sgd_partial_count(b->n), b->n, loss_mean_out, x->lstream)) != cudaSuccess)
    return cuda_fail(x, e, "learner update (loss reduction)");
  learner_launched(x);
  return TJ_OK;
}
}  // namespace

int tj_sgd_step(tj_ctx* x, const tj_batch* b, float lr, float* theta, const float* theta_target, float* loss_mean_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  return learner_update(x, b, lr, theta, theta_target, nullptr, loss_mean_out);
}

int tj_adam_step(tj_ctx* x, const tj_batch* b, float lr, float beta1, float beta2, float eps, int64_t t, float* theta,
                 const float* theta_target, float* m, float* v, float* loss_mean_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (!m || !v) return fail(x, TJ_ERR_INVALID_ARG, "moment blobs must not be null");
  if (m == v || m == theta || v == theta) return fail(x, TJ_ERR_INVALID_ARG, "theta, m and v must be different buffers");
  if (t < 1) return fail(x, TJ_ERR_INVALID_ARG, "the Adam step counter starts at 1");
  if (!(beta1 >= 0.f && beta1 < 1.f && beta2 >= 0.f && beta2 < 1.f && eps > 0.f))
    return fail(x, TJ_ERR_INVALID_ARG, "Adam needs 0 <= beta1, beta2 < 1 and eps > 0");
  tj::AdamParams a{};
  a.m = m; a.v = v; a.beta1 = beta1; a.beta2 = beta2; a.eps = eps;
  a.c1 = (float)(1.0 - std::pow((double)beta1, (double)t));
  a.c2 = (float)(1.0 - std::pow((double)beta2, (double)t));
  return learner_update(x, b, lr, theta, theta_target, &a, loss_mean_out);
}

int tj_ppo_step(tj_ctx* x, const tj_ppo_batch* b, float lr, float beta1, float beta2, float eps, int64_t t, float clip_eps,
                float c_v, float c_e, float* theta, float* m, float* v, float* stats_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (!b || !b->obs || !b->act || !b->logp_old || !b->adv || !b->ret) return fail(x, TJ_ERR_INVALID_ARG, "batch arrays must not be null");
  if (!theta || !m || !v) return fail(x, TJ_ERR_INVALID_ARG, "parameter and moment blobs must not be null");
  if (m == v || m == theta || v == theta) return fail(x, TJ_ERR_INVALID_ARG, "theta, m and v must be different buffers");
  if (t < 1) return fail(x, TJ_ERR_INVALID_ARG, "the Adam step counter starts at 1");
  if (!(lr >= 0.f) || !(beta1 >= 0.f && beta1 < 1.f && beta2 >= 0.f && beta2 < 1.f && eps > 0.f))
    return fail(x, TJ_ERR_INVALID_ARG, "needs lr >= 0, 0 <= beta1, beta2 < 1 and eps > 0");
  if (!(clip_eps >= 0.f && clip_eps < 1.f)) return fail(x, TJ_ERR_INVALID_ARG, "clip_eps must lie in [0, 1)");
  if (x->cfg.policy_kind != TJ_POLICY_CATEGORICAL || !x->sgd_scratch)
    return fail(x, TJ_ERR_UNSUPPORTED, "the PPO update is implemented for segment contexts with the categorical policy and value head");
  if (b->n < 1 || b->n > x->sgd_rows) return fail(x, TJ_ERR_INVALID_ARG, "batch.n must be between 1 and the configured minibatch (4096 if none)");
  SgdParams p{};
  p.n = b->n; p.D = x->D; p.H = x->H; p.A = x->A;
  p.theta = theta; p.theta_target = nullptr;
  p.obs = b->obs; p.act = b->act; p.logp_old = b->logp_old; p.adv = b->adv; p.ret = b->ret;
  p.clip_eps = clip_eps; p.c_v = c_v; p.c_e = c_e;
  lay_out_update_scratch(x, p);
  p.ldg = x->A + 1; p.value_head = 1;
  p.error = &x->dstats->error;
  tj::AdamParams a{};
  a.m = m; a.v = v; a.beta1 = beta1; a.beta2 = beta2; a.eps = eps;
  a.c1 = (float)(1.0 - std::pow((double)beta1, (double)t));
  a.c2 = (float)(1.0 - std::pow((double)beta2, (double)t));
  LaunchScope scope(x, TJ_K_SGD, tj::ppo_step_launches(p, stats_out != nullptr), true, true);
  cudaError_t e = launch_ppo_step(p, lr, &a, stats_out, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "PPO update");
  learner_launched(x);
  return TJ_OK;
}

int tj_gae(tj_ctx* x, const float* rew, const float* val, const uint8_t* done, int32_t T, int32_t N, float gamma,
           float lambda, float* adv_out, float* ret_out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (!rew || !val || !done || !adv_out || !ret_out) return fail(x, TJ_ERR_INVALID_ARG, "GAE arrays must not be null");
  if (T < 0 || N < 0) return fail(x, TJ_ERR_INVALID_ARG, "T and N must not be negative");
  if (T == 0 || N == 0) return TJ_OK;
  LaunchScope scope(x, TJ_K_GAE, 1, true, true);
  cudaError_t e = launch_gae(rew, val, done, T, N, gamma, lambda, adv_out, ret_out, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "GAE");
  learner_launched(x);
  return TJ_OK;
}

int tj_segment_acquire(tj_ctx* x, tj_segment* out) {
  if (!x || !out) return TJ_ERR_INVALID_ARG;
  const tj_config& c = x->cfg;
  if (c.replay_capacity != 0) return fail(x, TJ_ERR_INVALID_ARG, "segments exist only in segment mode");
  const int T = c.rollout_len, N = x->N, G = c.n_segments;
  const int64_t begun = (x->t + T - 1) / T;
  if (x->next_consume < begun - G) x->next_consume = begun - G;
  for (; x->next_consume < begun; ++x->next_consume) {
    SegSlot& sl = x->seg[(size_t)(x->next_consume % G)];
    if (sl.index != x->next_consume) continue;  // overwritten by a later segment
    if (sl.state == 1) break;                   // still being produced
    if (sl.state != 2) continue;
    if (x->version - sl.version > c.staleness_bound) {
      sl.state = 3;
      x->hs.dropped_stale += (int64_t)T * N;
      continue;
    }
    const size_t slot = (size_t)(x->next_consume % G), TN = (size_t)T * N;
    out->T = T; out->N = N; out->version = sl.version;
    out->obs = x->seg_obs + slot * TN * x->D;
    out->act = x->seg_act + slot * TN;
    out->rew = x->seg_rew + slot * TN;
    out->done = x->seg_done + slot * TN;
    out->logp = x->seg_logp + slot * TN;
    out->val = x->seg_val + slot * ((size_t)T + 1) * N;
    sl.state = 3;
    sl.acquired_index = sl.index;
    learner_waits_for_actor(x);
    x->next_consume += 1;
    x->k += 1;
    x->hs.learner_steps += 1;
    x->hs.consumed += (int64_t)T * N;
    const int64_t stale = x->version - sl.version;
    x->hs.max_sampled_staleness = std::max(x->hs.max_sampled_staleness, stale);
    x->hs.staleness_hist[stale > 32 ? 32 : stale] += (int64_t)T * N;
    return TJ_OK;
  }
  x->hs.starved_calls += 1;
  return fail(x, TJ_ERR_STARVED, "no complete segment within the staleness bound");
}

int tj_normalize(tj_ctx* x, const float* in, int64_t n, float eps, float* out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (!in || !out) return fail(x, TJ_ERR_INVALID_ARG, "arrays must not be null");
  if (n < 0 || !(eps >= 0.f)) return fail(x, TJ_ERR_INVALID_ARG, "n and eps must not be negative");
  if (n == 0) return TJ_OK;
  LaunchScope scope(x, TJ_K_GAE, 3, true, true);
  cudaError_t e = launch_normalize(in, n, (double)eps, out, x->norm_scratch, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "normalisation");
  learner_launched(x);
  return TJ_OK;
}

int tj_segment_minibatch(tj_ctx* x, const tj_segment* segv, const float* adv, const float* ret, uint64_t shuffle_id, int64_t first,
                         const tj_ppo_minibatch* out) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (!segv || !adv || !ret || !out) return fail(x, TJ_ERR_INVALID_ARG, "arguments must not be null");
  if (!out->obs || !out->act || !out->logp_old || !out->adv || !out->ret) return fail(x, TJ_ERR_INVALID_ARG, "minibatch arrays must not be null");
  if (!segv->obs || !segv->act || !segv->logp || segv->T < 1 || segv->N < 1) return fail(x, TJ_ERR_INVALID_ARG, "not a segment");
  const int64_t R = (int64_t)segv->T * segv->N;
  if (out->n < 0 || first < 0 || first + out->n > R) return fail(x, TJ_ERR_INVALID_ARG, "positions first .. first + n must lie inside the segment's T * N rows");
  if (R > ((int64_t)1 << 31)) return fail(x, TJ_ERR_UNSUPPORTED, "segments of more than 2^31 rows");
  if (out->n == 0) return TJ_OK;
  MinibatchParams p{};
  p.n = out->n; p.D = x->D; p.hb = shuffle_half_bits(R); p.R = R; p.first = first;
  p.seed = make_uint2((uint32_t)x->cfg.seed, (uint32_t)(x->cfg.seed >> 32));
  p.shuffle_id = shuffle_id;
  p.seg_obs = segv->obs; p.seg_act = segv->act; p.seg_logp = segv->logp; p.adv_in = adv; p.ret_in = ret;
  p.obs = out->obs; p.act = out->act; p.logp = out->logp_old; p.adv = out->adv; p.ret = out->ret; p.row = out->row;
  LaunchScope scope(x, TJ_K_SAMPLE, 1, true, true);
  cudaError_t e = launch_segment_minibatch(p, x->lstream);
  if (e != cudaSuccess) return cuda_fail(x, e, "segment minibatch");
  learner_launched(x);
  return TJ_OK;
}

int tj_segment_check(tj_ctx* x, const tj_segment* segv) {
  if (!x || !segv) return TJ_ERR_INVALID_ARG;
  const tj_config& c = x->cfg;
  if (c.replay_capacity != 0) return fail(x, TJ_ERR_INVALID_ARG, "segments exist only in segment mode");
  const size_t TN = (size_t)c.rollout_len * x->N;
  if (!segv->rew || segv->rew < x->seg_rew || (size_t)(segv->rew - x->seg_rew) % TN) return fail(x, TJ_ERR_INVALID_ARG, "not a segment of this context");
  const size_t slot = (size_t)(segv->rew - x->seg_rew) / TN;
  if (slot >= (size_t)c.n_segments) return fail(x, TJ_ERR_INVALID_ARG, "not a segment of this context");
  const SegSlot& sl = x->seg[slot];
  // consumed (3) and still holding the segment it was acquired as: the producer has not come round to the slot
  if (sl.state == 3 && sl.version == segv->version && sl.index == sl.acquired_index) return TJ_OK;
  return fail(x, TJ_ERR_STALE_SEGMENT, "the producer has started to overwrite this segment's slot");
}

int tj_get_state(tj_ctx* x, tj_state_view* out) {
  if (!x || !out) return TJ_ERR_INVALID_ARG;
  out->state = x->state; out->ep_step = x->ep_step;
  out->cursor = x->cursor; out->t = x->t; out->k = x->k;
  out->actor_version = out->learner_version = x->version;
  return TJ_OK;
}

int tj_set_state(tj_ctx* x, const tj_state_view* in) {
  if (!x || !in) return TJ_ERR_INVALID_ARG;
  if (in->t < 0 || in->k < 0) return fail(x, TJ_ERR_INVALID_ARG, "counters must not be negative");
  // The ring's contents, its per-block versions and the segment slots are not part of the view, so the counters that index
  // them cannot move: another cursor (ring mode) or another step count (segment mode) would leave the sampler and the
  // segment bookkeeping describing records that are not the resident ones.
  if (x->cfg.replay_capacity > 0 && in->cursor != x->cursor)
    return fail(x, TJ_ERR_UNSUPPORTED, "the cursor cannot be moved: the ring and its block versions are not part of the state view");
  if (x->cfg.replay_capacity == 0 && in->t != x->t)
    return fail(x, TJ_ERR_UNSUPPORTED, "t cannot be moved in segment mode: the segment slots are not part of the state view");
  cudaError_t e;
  if (in->state && in->state != x->state &&
      (e = cudaMemcpyAsync(x->state, in->state, sizeof(float) * (size_t)x->N * x->S_d, cudaMemcpyDeviceToDevice, x->stream)) != cudaSuccess)
    return cuda_fail(x, e, "set state");
  if (in->ep_step && in->ep_step != x->ep_step &&
      (e = cudaMemcpyAsync(x->ep_step, in->ep_step, sizeof(int) * (size_t)x->N, cudaMemcpyDeviceToDevice, x->stream)) != cudaSuccess)
    return cuda_fail(x, e, "set episode steps");
  x->t = in->t; x->k = in->k;
  return TJ_OK;
}

int tj_stats(tj_ctx* x, tj_stats_t* o) {
  if (!x || !o) return TJ_ERR_INVALID_ARG;
  DevStats d;
  cudaError_t e = x->two_stream ? cudaStreamSynchronize(x->lstream) : cudaSuccess;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&d, x->dstats, sizeof(d), cudaMemcpyDeviceToHost, x->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(x->stream);
  if (e != cudaSuccess) return cuda_fail(x, e, "read counters");
  drain_spans(x);
  *o = x->hs;
  o->actor_version = o->learner_version = x->version;
  o->episodes_finished = (int64_t)d.episodes;
  o->return_sum = d.return_sum;
  o->device_error = (int64_t)d.error;
  if (x->cfg.replay_capacity > 0) {
    o->max_sampled_staleness = (int64_t)d.max_stale;
    for (int i = 0; i < 33; ++i) o->staleness_hist[i] = (int64_t)d.hist[i];
  }
  if (d.error) return fail(x, TJ_ERR_TIMEOUT, "a kernel's bounded wait ran out (device_error holds the code); its outputs are not valid");
  return TJ_OK;
}

int tj_ring_view(tj_ctx* x, const float** records, const int32_t** block_version, int32_t* record_words) {
  if (!x) return TJ_ERR_INVALID_ARG;
  if (records) *records = x->ring;
  if (block_version) *block_version = x->block_ver;
  if (record_words) *record_words = x->rec_words;
  return TJ_OK;
}

int tj_calibrate_fp32(tj_ctx* x, float* scratch, size_t scratch_bytes, double* tflops_out) {
  if (!x || !tflops_out) return TJ_ERR_INVALID_ARG;
  const size_t need = fma_rate_sink_floats(x->sm_count) * sizeof(float);
  if (!scratch || scratch_bytes < need) return fail(x, TJ_ERR_WORKSPACE, "calibration scratch too small (needs sm_count * 8 KiB)");
  cudaEvent_t a = nullptr, b = nullptr;
  if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return fail(x, TJ_ERR_CUDA, "calibration: event creation failed");
  cudaError_t e = cudaSuccess;
  double best = 0.0;
  launch_fma_rate(scratch, x->sm_count, 64, x->stream, &e);            // warm-up
  for (int rep = 0; rep < 5 && e == cudaSuccess; ++rep) {
    cudaEventRecord(a, x->stream);
    const double flops = launch_fma_rate(scratch, x->sm_count, 4096, x->stream, &e);
    cudaEventRecord(b, x->stream);
    if (e != cudaSuccess) break;
    if ((e = cudaEventSynchronize(b)) != cudaSuccess) break;
    float ms = 0.f;
    if ((e = cudaEventElapsedTime(&ms, a, b)) != cudaSuccess) break;
    if (ms > 0.f) best = std::max(best, flops / (ms * 1e-3) / 1e12);
  }
  cudaEventDestroy(a);
  cudaEventDestroy(b);
  if (e != cudaSuccess) return cuda_fail(x, e, "calibration");
  *tflops_out = best;
  return TJ_OK;
}

const char* tj_last_error(const tj_ctx* x) { return x ? x->err.c_str() : g_err.c_str(); }

}  // extern "C"
