"""ctypes binding of ``libtj.so`` (see ``include/tj.h``): argument marshalling only.

The module-level ``tj_*`` functions mirror the C ABI one to one.  ``Context`` is a
convenience wrapper that allocates the workspace and the output arrays with torch
(device memory and the stream are torch's; every computation runs in the library's
CUDA kernels).  There is no CPU fallback: without the compiled library or without a
CUDA device the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# TJ_LIB_PATH names another build of the library (same ABI), e.g. one compiled with different options
LIB_PATH = os.environ.get("TJ_LIB_PATH") or os.path.join(_HERE, "libtj.so")

TJ_OK, TJ_ERR_INVALID_ARG, TJ_ERR_CONFIG, TJ_ERR_WORKSPACE, TJ_ERR_CUDA = 0, -1, -2, -3, -4
TJ_ERR_NO_WEIGHTS, TJ_ERR_WARMUP, TJ_ERR_STARVED, TJ_ERR_STALE_SEGMENT, TJ_ERR_TIMEOUT, TJ_ERR_UNSUPPORTED = (
    -5, -6, -7, -8, -9, -10)
STATUS_NAMES = {0: "TJ_OK", -1: "TJ_ERR_INVALID_ARG", -2: "TJ_ERR_CONFIG", -3: "TJ_ERR_WORKSPACE", -4: "TJ_ERR_CUDA",
                -5: "TJ_ERR_NO_WEIGHTS", -6: "TJ_ERR_WARMUP", -7: "TJ_ERR_STARVED", -8: "TJ_ERR_STALE_SEGMENT",
                -9: "TJ_ERR_TIMEOUT", -10: "TJ_ERR_UNSUPPORTED"}

EXPORTS = ("tj_query_workspace", "tj_create", "tj_destroy", "tj_set_learner_stream", "tj_wait", "tj_publish_weights", "tj_actor_step", "tj_replay_sample",
           "tj_td_error", "tj_td_error_static", "tj_sgd_step", "tj_adam_step", "tj_ppo_step", "tj_gae", "tj_segment_acquire", "tj_segment_check", "tj_normalize", "tj_segment_minibatch", "tj_get_state", "tj_set_state", "tj_stats", "tj_set_profiling", "tj_ring_view", "tj_calibrate_fp32",
           "tj_last_error")


class TjConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("device", C.c_int32),
        ("env_kind", C.c_int32), ("n_envs", C.c_int32), ("obs_dim", C.c_int32), ("n_actions", C.c_int32),
        ("max_episode_steps", C.c_int32), ("lg_done_norm", C.c_float), ("lg_noise_std", C.c_float),
        ("host_lg_A", C.c_void_p), ("host_lg_B", C.c_void_p),
        ("hidden", C.c_int32), ("policy_kind", C.c_int32), ("weight_dtype", C.c_int32), ("epsilon", C.c_float),
        ("seed", C.c_uint64),
        ("replay_capacity", C.c_int64), ("minibatch", C.c_int32), ("staleness_bound", C.c_int32),
        ("warmup", C.c_int32), ("rollout_len", C.c_int32), ("n_segments", C.c_int32),
        ("target_sync_interval", C.c_int32), ("gamma", C.c_float), ("huber_delta", C.c_float),
        ("gae_lambda", C.c_float),
    ]


class TjBatch(C.Structure):
    _fields_ = [("n", C.c_int32), ("obs", C.c_void_p), ("act", C.c_void_p), ("rew", C.c_void_p),
                ("next_obs", C.c_void_p), ("done", C.c_void_p), ("ver", C.c_void_p)]


class TjSegment(C.Structure):
    _fields_ = [("T", C.c_int32), ("N", C.c_int32), ("version", C.c_int64), ("obs", C.c_void_p), ("act", C.c_void_p),
                ("rew", C.c_void_p), ("done", C.c_void_p), ("logp", C.c_void_p), ("val", C.c_void_p)]


class TjStateView(C.Structure):
    _fields_ = [("state", C.c_void_p), ("ep_step", C.c_void_p), ("cursor", C.c_uint64), ("t", C.c_int64),
                ("k", C.c_int64), ("actor_version", C.c_int64), ("learner_version", C.c_int64)]


class TjStats(C.Structure):
    _fields_ = [("produced", C.c_int64), ("consumed", C.c_int64), ("dropped_stale", C.c_int64),
                ("dropped_overwritten", C.c_int64), ("starved_calls", C.c_int64), ("actor_version", C.c_int64),
                ("learner_version", C.c_int64), ("actor_steps", C.c_int64), ("learner_steps", C.c_int64),
                ("max_sampled_staleness", C.c_int64), ("episodes_finished", C.c_int64), ("return_sum", C.c_double),
                ("staleness_hist", C.c_int64 * 33), ("device_error", C.c_int64), ("kernel_launches", C.c_int64),
                ("kernel_count", C.c_int64 * 8), ("kernel_ms", C.c_double * 8)]


_lib = None


def load_library():
    """Load libtj.so; raises (never falls back) when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libtj.so is missing: build it with `python -m paper_2502_20190_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    L.tj_query_workspace.argtypes = [vp, vp, vp]
    L.tj_create.argtypes = [vp, vp, C.c_size_t, vp, vp]
    L.tj_destroy.argtypes = [vp]
    L.tj_set_learner_stream.argtypes = [vp, vp]
    L.tj_wait.argtypes = [vp, i32, i32]
    L.tj_publish_weights.argtypes = [vp, vp, C.c_size_t, i32, vp]
    L.tj_actor_step.argtypes = [vp, i32, vp]
    L.tj_replay_sample.argtypes = [vp, i32, vp, vp]
    L.tj_td_error.argtypes = [vp, vp, vp, vp, vp]
    L.tj_td_error_static.argtypes = [vp, vp, vp, vp, vp]
    L.tj_gae.argtypes = [vp, vp, vp, vp, i32, i32, f32, f32, vp, vp]
    L.tj_sgd_step.argtypes = [vp, vp, f32, vp, vp, vp]
    L.tj_adam_step.argtypes = [vp, vp, f32, f32, f32, f32, i64, vp, vp, vp, vp, vp]
    L.tj_ppo_step.argtypes = [vp, vp, f32, f32, f32, f32, i64, f32, f32, f32, vp, vp, vp, vp]
    L.tj_segment_acquire.argtypes = [vp, vp]
    L.tj_segment_check.argtypes = [vp, vp]
    L.tj_normalize.argtypes = [vp, vp, i64, f32, vp]
    L.tj_segment_minibatch.argtypes = [vp, vp, vp, vp, C.c_uint64, i64, vp]
    L.tj_get_state.argtypes = [vp, vp]
    L.tj_set_state.argtypes = [vp, vp]
    L.tj_stats.argtypes = [vp, vp]
    L.tj_set_profiling.argtypes = [vp, i32]
    L.tj_ring_view.argtypes = [vp, vp, vp, vp]
    L.tj_calibrate_fp32.argtypes = [vp, vp, C.c_size_t, vp]
    L.tj_last_error.argtypes = [vp]
    L.tj_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name != "tj_last_error":
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


class TjError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, status), message))
        self.status = status


# ---------------------------------------------------------------- one-to-one wrappers
def tj_query_workspace(cfg: TjConfig):
    nbytes, align = C.c_size_t(), C.c_size_t()
    st = load_library().tj_query_workspace(C.byref(cfg), C.byref(nbytes), C.byref(align))
    return st, nbytes.value, align.value


def tj_create(cfg: TjConfig, workspace_ptr: int, nbytes: int, stream_ptr: int):
    h = C.c_void_p()
    st = load_library().tj_create(C.byref(cfg), workspace_ptr, nbytes, stream_ptr, C.byref(h))
    return st, h


def tj_destroy(h):
    return load_library().tj_destroy(h)


def tj_set_learner_stream(h, stream_ptr: int):
    return load_library().tj_set_learner_stream(h, stream_ptr or None)


def tj_wait(h, which: int, timeout_ms: int):
    return load_library().tj_wait(h, which, timeout_ms)


def tj_publish_weights(h, blob_ptr: int, nbytes: int, on_device: int):
    v = C.c_int64()
    st = load_library().tj_publish_weights(h, blob_ptr, nbytes, on_device, C.byref(v))
    return st, v.value


def tj_actor_step(h, n_steps: int, dbg_logits_ptr: int = 0):
    return load_library().tj_actor_step(h, n_steps, dbg_logits_ptr or None)


def tj_replay_sample(h, staleness_bound: int, idx_ptr: int, batch: TjBatch):
    return load_library().tj_replay_sample(h, staleness_bound, idx_ptr or None, C.byref(batch))


def tj_td_error(h, batch: TjBatch, td_ptr: int, huber_ptr: int, loss_ptr: int):
    return load_library().tj_td_error(h, C.byref(batch), td_ptr or None, huber_ptr or None, loss_ptr or None)


def tj_td_error_static(h, batch: TjBatch, td_ptr: int, huber_ptr: int, loss_ptr: int):
    """tj_td_error with the reduction scratch inside the library image (at most 65,536 rows; allocates nothing)."""
    return load_library().tj_td_error_static(h, C.byref(batch), td_ptr or None, huber_ptr or None, loss_ptr or None)


def tj_sgd_step(h, batch: TjBatch, lr: float, theta_ptr: int, theta_target_ptr: int, loss_ptr: int):
    """One learner update (Algorithm 1's update line as a minibatch semi-gradient step) on device blobs, in place."""
    return load_library().tj_sgd_step(h, C.byref(batch), lr, theta_ptr, theta_target_ptr, loss_ptr or None)


def tj_adam_step(h, batch: TjBatch, lr, beta1, beta2, eps, t, theta_ptr, theta_target_ptr, m_ptr, v_ptr, loss_ptr):
    """tj_sgd_step's gradient through Adam; m and v are device moment blobs updated in place."""
    return load_library().tj_adam_step(h, C.byref(batch), lr, beta1, beta2, eps, t, theta_ptr, theta_target_ptr, m_ptr, v_ptr,
                                       loss_ptr or None)


class TjPpoBatch(C.Structure):
    _fields_ = [("n", C.c_int32), ("obs", C.c_void_p), ("act", C.c_void_p), ("logp_old", C.c_void_p), ("adv", C.c_void_p),
                ("ret", C.c_void_p)]


def tj_ppo_step(h, batch: TjPpoBatch, lr, beta1, beta2, eps, t, clip_eps, c_v, c_e, theta_ptr, m_ptr, v_ptr, stats_ptr):
    """One PPO minibatch update (clipped surrogate + value loss - entropy bonus, Adam) on device blobs, in place."""
    return load_library().tj_ppo_step(h, C.byref(batch), lr, beta1, beta2, eps, t, clip_eps, c_v, c_e, theta_ptr, m_ptr, v_ptr,
                                      stats_ptr or None)


def tj_gae(h, rew_ptr, val_ptr, done_ptr, T, N, gamma, lam, adv_ptr, ret_ptr):
    return load_library().tj_gae(h, rew_ptr, val_ptr, done_ptr, T, N, gamma, lam, adv_ptr, ret_ptr)


def tj_segment_acquire(h):
    seg = TjSegment()
    st = load_library().tj_segment_acquire(h, C.byref(seg))
    return st, seg


class TjPpoMinibatch(C.Structure):
    _fields_ = [("n", C.c_int32), ("obs", C.c_void_p), ("act", C.c_void_p), ("logp_old", C.c_void_p), ("adv", C.c_void_p),
                ("ret", C.c_void_p), ("row", C.c_void_p)]


def tj_normalize(h, x_ptr: int, n: int, eps: float, out_ptr: int):
    return load_library().tj_normalize(h, x_ptr, n, eps, out_ptr)


def tj_segment_minibatch(h, seg: TjSegment, adv_ptr: int, ret_ptr: int, shuffle_id: int, first: int, out: TjPpoMinibatch):
    return load_library().tj_segment_minibatch(h, C.byref(seg), adv_ptr, ret_ptr, shuffle_id, first, C.byref(out))


def tj_segment_check(h, seg: TjSegment):
    return load_library().tj_segment_check(h, C.byref(seg))


def tj_get_state(h):
    v = TjStateView()
    st = load_library().tj_get_state(h, C.byref(v))
    return st, v


def tj_set_state(h, view: TjStateView):
    return load_library().tj_set_state(h, C.byref(view))


def tj_stats(h):
    s = TjStats()
    st = load_library().tj_stats(h, C.byref(s))
    return st, s


def tj_set_profiling(h, on: int):
    return load_library().tj_set_profiling(h, int(on))


def tj_ring_view(h):
    rec, bv, rw = C.c_void_p(), C.c_void_p(), C.c_int32()
    st = load_library().tj_ring_view(h, C.byref(rec), C.byref(bv), C.byref(rw))
    return st, rec.value, bv.value, rw.value


def tj_calibrate_fp32(h, scratch_ptr: int, scratch_bytes: int):
    out = C.c_double()
    st = load_library().tj_calibrate_fp32(h, scratch_ptr, scratch_bytes, C.byref(out))
    return st, out.value


def tj_last_error(h=None) -> str:
    return (load_library().tj_last_error(h) or b"").decode()


def make_config(*, env_kind, n_envs, obs_dim, n_actions, hidden, policy_kind=0, weight_dtype=0, epsilon=0.1, seed=0,
                replay_capacity=0, minibatch=1, staleness_bound=0, warmup=0, rollout_len=1, target_sync_interval=0,
                n_segments=1, gamma=0.99, huber_delta=1.0, gae_lambda=0.95, max_episode_steps=0, lg_done_norm=4.0,
                lg_noise_std=0.01, lg_A=None, lg_B=None, device=0, **_ignored):
    """Fill a tj_config; returns (cfg, keepalive) where keepalive holds the host arrays cfg points to."""
    keep = []
    pa = pb = None
    if lg_A is not None:
        a = np.ascontiguousarray(lg_A, np.float32)
        b = np.ascontiguousarray(lg_B, np.float32)
        keep += [a, b]
        pa, pb = a.ctypes.data, b.ctypes.data
    cfg = TjConfig(C.sizeof(TjConfig), device, env_kind, n_envs, obs_dim, n_actions, max_episode_steps, lg_done_norm,
                   lg_noise_std, pa, pb, hidden, policy_kind, weight_dtype, epsilon, int(seed) & (2**64 - 1),
                   replay_capacity, minibatch, staleness_bound, warmup, rollout_len, n_segments,
                   target_sync_interval, gamma, huber_delta, gae_lambda)
    return cfg, keep


# ---------------------------------------------------------------- torch-backed convenience wrapper
class Context:
    """A context whose workspace and outputs are torch CUDA tensors on torch's current stream."""

    def __init__(self, **fields):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.torch = torch
        self.cfg, self._keep = make_config(**fields)
        self.device = torch.device("cuda", self.cfg.device)
        st, nbytes, align = tj_query_workspace(self.cfg)
        if st != TJ_OK:
            raise TjError(st, tj_last_error())
        self.workspace_bytes = nbytes
        self.workspace = torch.empty(nbytes + align, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_off = (-base) % align
        self._ws_ptr = base + self._ws_off
        self.stream = torch.cuda.current_stream(self.device)
        st, self.h = tj_create(self.cfg, self._ws_ptr, nbytes, self.stream.cuda_stream)
        if st != TJ_OK:
            raise TjError(st, tj_last_error())
        c = self.cfg
        self.N, self.D, self.A, self.H, self.B = c.n_envs, c.obs_dim, c.n_actions, c.hidden, c.minibatch
        self.S_d = c.obs_dim if c.env_kind == 2 else 4
        self.value_head = c.policy_kind == 1
        self.rec_words = 2 * self.D + 4
        self._batch = None

    def use_learner_stream(self, on=True):
        """Learner-side calls on a second torch stream (concurrent with the actor), or back on the one stream."""
        if on:
            if getattr(self, "learner_stream", None) is None:
                self.learner_stream = self.torch.cuda.Stream(self.device)
            return self._check(tj_set_learner_stream(self.h, self.learner_stream.cuda_stream))
        return self._check(tj_set_learner_stream(self.h, 0))

    def wait(self, which, timeout_ms, allow=(TJ_OK, TJ_ERR_TIMEOUT)):
        return self._check(tj_wait(self.h, which, timeout_ms), allow)

    def close(self):
        if getattr(self, "h", None):
            tj_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, ok=(TJ_OK,)):
        if st not in ok:
            raise TjError(st, tj_last_error(self.h))
        return st

    def _view(self, ptr, shape, dtype):
        """torch view of a workspace address."""
        torch = self.torch
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        off = ptr - self.workspace.data_ptr()
        assert 0 <= off and off + n <= self.workspace.numel()
        return self.workspace[off:off + n].view(dtype).view(*shape)

    # ---- calls
    def publish_weights(self, blob):
        """blob: numpy float32 array (host) or torch CUDA float32 tensor (device)."""
        torch = self.torch
        if isinstance(blob, torch.Tensor):
            assert blob.is_cuda and blob.dtype == torch.float32 and blob.is_contiguous()
            st, v = tj_publish_weights(self.h, blob.data_ptr(), blob.numel() * 4, 1)
        else:
            blob = np.ascontiguousarray(blob, np.float32)
            st, v = tj_publish_weights(self.h, blob.ctypes.data, blob.size * 4, 0)
        self._check(st)
        return v

    def actor_step(self, n_steps=1, dbg_logits=None):
        ptr = 0
        if dbg_logits is not None:
            assert dbg_logits.is_cuda and dbg_logits.numel() >= n_steps * self.N * self.A
            ptr = dbg_logits.data_ptr()
        return self._check(tj_actor_step(self.h, n_steps, ptr))

    def alloc_batch(self, n=None):
        torch = self.torch
        n = n or self.B
        dev = self.device
        t = dict(obs=torch.empty((n, self.D), dtype=torch.float32, device=dev),
                 act=torch.empty(n, dtype=torch.int32, device=dev),
                 rew=torch.empty(n, dtype=torch.float32, device=dev),
                 next_obs=torch.empty((n, self.D), dtype=torch.float32, device=dev),
                 done=torch.empty(n, dtype=torch.int32, device=dev),
                 ver=torch.empty(n, dtype=torch.int32, device=dev),
                 idx=torch.empty(n, dtype=torch.int32, device=dev))
        t["c"] = TjBatch(n, t["obs"].data_ptr(), t["act"].data_ptr(), t["rew"].data_ptr(), t["next_obs"].data_ptr(),
                         t["done"].data_ptr(), t["ver"].data_ptr())
        return t

    def replay_sample(self, staleness_bound=-1, batch=None, allow=(TJ_OK,)):
        if batch is None:
            if self._batch is None:
                self._batch = self.alloc_batch()
            batch = self._batch
        st = tj_replay_sample(self.h, staleness_bound, batch["idx"].data_ptr(), batch["c"])
        self._check(st, allow)
        return st, batch

    def td_error(self, batch, out=None):
        torch = self.torch
        n = batch["c"].n
        if out is None:
            out = dict(td=torch.empty(n, dtype=torch.float32, device=self.device),
                       huber=torch.empty(n, dtype=torch.float32, device=self.device),
                       loss=torch.empty(1, dtype=torch.float32, device=self.device))
        self._check(tj_td_error(self.h, batch["c"], out["td"].data_ptr(), out["huber"].data_ptr(),
                                out["loss"].data_ptr()))
        return out

    def sgd_step(self, batch, lr, theta, theta_target):
        """theta (updated in place) and theta_target: float32 device tensors in the publish layout; returns the loss tensor"""
        torch = self.torch
        assert theta.dtype == torch.float32 and theta_target.dtype == torch.float32
        assert theta.is_contiguous() and theta_target.is_contiguous() and theta.numel() == theta_target.numel()
        loss = torch.empty(1, dtype=torch.float32, device=self.device)
        self._check(tj_sgd_step(self.h, batch["c"], float(lr), theta.data_ptr(), theta_target.data_ptr(), loss.data_ptr()))
        return loss

    def adam_step(self, batch, lr, theta, theta_target, m, v, t, beta1=0.9, beta2=0.999, eps=1e-8):
        torch = self.torch
        for x in (theta, theta_target, m, v):
            assert x.dtype == torch.float32 and x.is_contiguous() and x.numel() == theta.numel()
        loss = torch.empty(1, dtype=torch.float32, device=self.device)
        self._check(tj_adam_step(self.h, batch["c"], float(lr), float(beta1), float(beta2), float(eps), int(t), theta.data_ptr(),
                                 theta_target.data_ptr(), m.data_ptr(), v.data_ptr(), loss.data_ptr()))
        return loss

    def ppo_step(self, obs, act, logp_old, adv, ret, lr, theta, m, v, t, clip_eps=0.2, c_v=0.5, c_e=0.01, beta1=0.9,
                 beta2=0.999, eps=1e-8):
        """obs [n][D], act (int32), logp_old, adv, ret [n]: contiguous device tensors (views of a segment are fine);
        returns the 5 statistics tensor (loss, policy, value, entropy, clip fraction)"""
        torch = self.torch
        n = act.numel()
        for x_ in (obs, act, logp_old, adv, ret, theta, m, v):
            assert x_.is_contiguous()
        assert obs.numel() == n * self.D and act.dtype == torch.int32
        stats = torch.empty(5, dtype=torch.float32, device=self.device)
        b = TjPpoBatch(n, obs.data_ptr(), act.data_ptr(), logp_old.data_ptr(), adv.data_ptr(), ret.data_ptr())
        self._check(tj_ppo_step(self.h, b, float(lr), float(beta1), float(beta2), float(eps), int(t), float(clip_eps), float(c_v),
                                float(c_e), theta.data_ptr(), m.data_ptr(), v.data_ptr(), stats.data_ptr()))
        return stats

    def gae(self, rew, val, done, gamma, lam, adv=None, ret=None):
        torch = self.torch
        T, N = rew.shape
        assert val.shape == (T + 1, N) and done.shape == (T, N) and done.dtype == torch.uint8
        assert rew.is_contiguous() and val.is_contiguous() and done.is_contiguous()
        if adv is None:
            adv = torch.empty_like(rew)
        if ret is None:
            ret = torch.empty_like(rew)
        self._check(tj_gae(self.h, rew.data_ptr(), val.data_ptr(), done.data_ptr(), T, N, gamma, lam, adv.data_ptr(),
                           ret.data_ptr()))
        return adv, ret

    def segment_acquire(self, allow=(TJ_OK,)):
        torch = self.torch
        st, seg = tj_segment_acquire(self.h)
        self._check(st, allow)
        if st != TJ_OK:
            return st, None
        T, N, D = seg.T, seg.N, self.D
        return st, dict(T=T, N=N, version=seg.version, c=seg,
                        obs=self._view(seg.obs, (T, N, D), torch.float32), act=self._view(seg.act, (T, N), torch.int32),
                        rew=self._view(seg.rew, (T, N), torch.float32), done=self._view(seg.done, (T, N), torch.uint8),
                        logp=self._view(seg.logp, (T, N), torch.float32),
                        val=self._view(seg.val, (T + 1, N), torch.float32))

    def normalize(self, x, eps=1e-8, out=None):
        """(x - mean) / (std + eps) over all entries of a float32 device tensor, in the library's kernels."""
        assert x.is_cuda and x.dtype == self.torch.float32 and x.is_contiguous()
        if out is None:
            out = self.torch.empty_like(x)
        self._check(tj_normalize(self.h, x.data_ptr(), x.numel(), float(eps), out.data_ptr()))
        return out

    def alloc_minibatch(self, n):
        torch, dev = self.torch, self.device
        t = dict(obs=torch.empty((n, self.D), dtype=torch.float32, device=dev), act=torch.empty(n, dtype=torch.int32, device=dev),
                 logp_old=torch.empty(n, dtype=torch.float32, device=dev), adv=torch.empty(n, dtype=torch.float32, device=dev),
                 ret=torch.empty(n, dtype=torch.float32, device=dev), row=torch.empty(n, dtype=torch.int32, device=dev))
        t["c"] = TjPpoMinibatch(n, t["obs"].data_ptr(), t["act"].data_ptr(), t["logp_old"].data_ptr(), t["adv"].data_ptr(),
                                t["ret"].data_ptr(), t["row"].data_ptr())
        return t

    def segment_minibatch(self, seg, adv, ret, shuffle_id, first, mb):
        """Rows at positions first .. first + n - 1 of shuffle `shuffle_id` of the segment, copied into the minibatch arrays."""
        assert adv.is_contiguous() and ret.is_contiguous() and adv.numel() == seg["T"] * seg["N"] == ret.numel()
        self._check(tj_segment_minibatch(self.h, seg["c"], adv.data_ptr(), ret.data_ptr(), int(shuffle_id), int(first), mb["c"]))
        return mb

    def segment_check(self, seg, allow=(TJ_OK, TJ_ERR_STALE_SEGMENT)):
        return self._check(tj_segment_check(self.h, seg["c"]), allow)

    def get_state(self):
        torch = self.torch
        st, v = tj_get_state(self.h)
        self._check(st)
        return dict(state=self._view(v.state, (self.N, self.S_d), torch.float32),
                    ep_step=self._view(v.ep_step, (self.N,), torch.int32), cursor=v.cursor, t=v.t, k=v.k,
                    actor_version=v.actor_version, learner_version=v.learner_version)

    def set_state(self, state=None, ep_step=None, cursor=0, t=0, k=0):
        v = TjStateView(state.data_ptr() if state is not None else None,
                        ep_step.data_ptr() if ep_step is not None else None, cursor, t, k, 0, 0)
        return self._check(tj_set_state(self.h, v))

    def stats(self):
        st, s = tj_stats(self.h)
        self._check(st, (TJ_OK, TJ_ERR_TIMEOUT))   # on a latched device error the counters are filled all the same
        arrays = ("staleness_hist", "kernel_count", "kernel_ms")
        d = {k: getattr(s, k) for k, _ in TjStats._fields_ if k not in arrays}
        for k in arrays:
            d[k] = list(getattr(s, k))
        return d

    def calibrate_fp32(self):
        """Measured FP32 FMA rate of the device in TFLOP/s (a register-only FMA loop on every SM)."""
        scratch = self.torch.empty(256 * 8192, dtype=self.torch.uint8, device=self.device)
        st, v = tj_calibrate_fp32(self.h, scratch.data_ptr(), scratch.numel())
        self._check(st)
        return v

    def set_profiling(self, on):
        return self._check(tj_set_profiling(self.h, on))

    def ring_view(self):
        torch = self.torch
        st, rec, bv, rw = tj_ring_view(self.h)
        self._check(st)
        C_ = self.cfg.replay_capacity
        return (self._view(rec, (C_, rw), torch.float32), self._view(bv, (C_ // self.N,), torch.int32))
