"""ctypes front end of the plain CPU oracle (``tj_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline timing
may import this package; the CUDA library and its Python binding never do.  The
oracle is compiled with gcc on first use (``-ffp-contract=off``, no fast-math).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tj_oracle.c")
_HDR = os.path.join(_HERE, "tj_oracle.h")
_LIB = os.path.join(_HERE, "libtj_oracle.so")

OK, ERR_ARG, ERR_CONFIG, ERR_NO_WEIGHTS, ERR_WARMUP, ERR_STARVED = 0, -1, -2, -5, -6, -7
ENV_CARTPOLE, ENV_ACROBOT, ENV_LINGAUSS = 0, 1, 2
POLICY_EPS_GREEDY, POLICY_CATEGORICAL = 0, 1
W_FP32, W_BF16 = 0, 1
STREAM_ACTION, STREAM_RESET, STREAM_NOISE, STREAM_SAMPLE, STREAM_SHUFFLE = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source."""
    stale = (not os.path.exists(_LIB)) or any(
        os.path.getmtime(p) > os.path.getmtime(_LIB) for p in (_SRC, _HDR))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-Wall",
                               "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Config(C.Structure):
    _fields_ = [
        ("env_kind", C.c_int32), ("n_envs", C.c_int32), ("obs_dim", C.c_int32), ("n_actions", C.c_int32),
        ("hidden", C.c_int32), ("policy_kind", C.c_int32), ("weight_dtype", C.c_int32),
        ("epsilon", C.c_float), ("seed", C.c_uint64), ("replay_capacity", C.c_int64),
        ("minibatch", C.c_int32), ("staleness_bound", C.c_int32), ("warmup", C.c_int32),
        ("rollout_len", C.c_int32), ("target_sync_interval", C.c_int32), ("n_segments", C.c_int32),
        ("gamma", C.c_float), ("huber_delta", C.c_float), ("gae_lambda", C.c_float),
        ("max_episode_steps", C.c_int32), ("lg_done_norm", C.c_float), ("lg_noise_std", C.c_float),
        ("lg_A", C.c_void_p), ("lg_B", C.c_void_p),
    ]


class Stats(C.Structure):
    _fields_ = [
        ("produced", C.c_int64), ("consumed", C.c_int64), ("dropped_stale", C.c_int64),
        ("dropped_overwritten", C.c_int64), ("starved_calls", C.c_int64), ("actor_version", C.c_int64),
        ("learner_version", C.c_int64), ("actor_steps", C.c_int64), ("learner_steps", C.c_int64),
        ("max_sampled_staleness", C.c_int64), ("episodes_finished", C.c_int64), ("return_sum", C.c_double),
        ("staleness_hist", C.c_int64 * 33),
    ]


class Segment(C.Structure):
    _fields_ = [("T", C.c_int32), ("N", C.c_int32), ("version", C.c_int64), ("obs", C.c_void_p),
                ("act", C.c_void_p), ("rew", C.c_void_p), ("done", C.c_void_p), ("logp", C.c_void_p),
                ("val", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(build())
    vp, i32, u32, u64, i64, f32, f64 = (C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_int64, C.c_float,
                                        C.c_double)
    sig = {
        "orc_philox4x32_10": (None, [vp, vp, vp]),
        "orc_stream_words": (None, [u64, u32, u32, u32, u64, vp]),
        "orc_u01": (f32, [u32]),
        "orc_mulhi": (u32, [u32, u32]),
        "orc_normal4": (None, [vp, vp]),
        "orc_explore_threshold": (u64, [f32]),
        "orc_cartpole_step": (None, [vp, i32, vp, vp, vp, vp]),
        "orc_acrobot_deriv": (None, [vp, f64, vp]),
        "orc_acrobot_energy": (f64, [vp]),
        "orc_acrobot_rk4": (None, [vp, f64, f64, vp]),
        "orc_acrobot_step": (None, [vp, i32, vp, vp, vp, vp]),
        "orc_acrobot_obs": (None, [vp, vp]),
        "orc_lingauss_step": (None, [vp, i32, vp, vp, vp, i32, f64, f64, vp, vp, vp, vp]),
        "orc_blob_floats": (i64, [i32, i32, i32, i32]),
        "orc_mlp_forward_f32": (None, [vp, i32, i32, i32, i32, vp, vp, vp]),
        "orc_mlp_forward_f64": (None, [vp, i32, i32, i32, i32, vp, vp, vp]),
        "orc_bf16_round": (f32, [f32]),
        "orc_select_eps_greedy": (i32, [vp, i32, u32, u32, u64]),
        "orc_argmax_lowest": (i32, [vp, i32]),
        "orc_select_categorical": (i32, [vp, i32, f32, vp, vp]),
        "orc_td_one": (None, [f64, f64, f64, i32, f64, f64, vp, vp]),
        "orc_gae": (None, [vp, vp, vp, i32, i32, f64, f64, vp, vp]),
        "orc_shuffle_index": (i64, [u64, u64, i64, i64]),
        "orc_normalize": (None, [vp, i64, f64, vp]),
        "orc_create": (vp, [vp, vp]),
        "orc_destroy": (None, [vp]),
        "orc_publish": (i32, [vp, vp, i64]),
        "orc_actor_step": (i32, [vp, i32]),
        "orc_sample": (i32, [vp, i32, vp, vp]),
        "orc_td": (i32, [vp, vp, i32, vp, vp, vp, vp, vp]),
        "orc_segment_acquire": (i32, [vp, vp]),
        "orc_get_stats": (None, [vp, vp]),
        "orc_state_dim": (i32, [vp]),
        "orc_record_words": (i32, [vp]),
        "orc_state": (vp, [vp]),
        "orc_ep_step": (vp, [vp]),
        "orc_set_counters": (None, [vp, u64, i64, i64]),
        "orc_cursor": (u64, [vp]),
        "orc_ring": (vp, [vp]),
        "orc_block_version": (vp, [vp]),
    }
    for name in ("obs", "logits", "act", "rew", "done", "next_obs", "done_margin", "act_margin", "logp", "value"):
        sig["orc_last_" + name] = (vp, [vp])
    sig["orc_online_blob"] = (vp, [vp])
    sig["orc_target_blob"] = (vp, [vp])
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _view(ptr, shape, dtype):
    n = int(np.prod(shape))
    if n == 0 or not ptr:
        return np.zeros(shape, dtype)
    buf = (C.c_char * (n * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype).reshape(shape)


# --------------------------------------------------------------------------- building blocks
def philox4x32_10(ctr, key):
    c = np.asarray(ctr, np.uint32).copy()
    k = np.asarray(key, np.uint32).copy()
    o = np.zeros(4, np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(o))
    return o


def stream_words(seed, stream, block, c0, step):
    o = np.zeros(4, np.uint32)
    lib().orc_stream_words(int(seed) & (2**64 - 1), stream, block, c0, int(step) & (2**64 - 1), _p(o))
    return o


def u01(x):
    return float(lib().orc_u01(int(x)))


def mulhi(x, n):
    return int(lib().orc_mulhi(int(x), int(n)))


def normal4(words):
    w = np.asarray(words, np.uint32).copy()
    z = np.zeros(4, np.float64)
    lib().orc_normal4(_p(w), _p(z))
    return z


def explore_threshold(eps):
    return int(lib().orc_explore_threshold(float(eps)))


def _env_step(fn, s, a):
    s = np.asarray(s, np.float32).copy()
    sn = np.zeros(4, np.float32)
    r = C.c_float()
    term = C.c_int()
    m = C.c_double()
    fn(_p(s), int(a), _p(sn), C.byref(r), C.byref(term), C.byref(m))
    return sn, float(r.value), int(term.value), float(m.value)


def cartpole_step(s, a):
    return _env_step(lib().orc_cartpole_step, s, a)


def acrobot_step(s, a):
    return _env_step(lib().orc_acrobot_step, s, a)


def acrobot_deriv(y, torque):
    y = np.asarray(y, np.float64).copy()
    dy = np.zeros(4, np.float64)
    lib().orc_acrobot_deriv(_p(y), float(torque), _p(dy))
    return dy


def acrobot_energy(y):
    y = np.asarray(y, np.float64).copy()
    return float(lib().orc_acrobot_energy(_p(y)))


def acrobot_rk4(y, torque, dt):
    y = np.asarray(y, np.float64).copy()
    yn = np.zeros(4, np.float64)
    lib().orc_acrobot_rk4(_p(y), float(torque), float(dt), _p(yn))
    return yn


def acrobot_obs(s):
    s = np.asarray(s, np.float32).copy()
    o = np.zeros(6, np.float32)
    lib().orc_acrobot_obs(_p(s), _p(o))
    return o


def lingauss_step(s, a, A, Bm, noise, noise_std=0.01, done_norm=4.0):
    s = np.ascontiguousarray(s, np.float32)
    A = np.ascontiguousarray(A, np.float32)
    Bm = np.ascontiguousarray(Bm, np.float32)
    noise = np.ascontiguousarray(noise, np.float64)
    D = s.shape[0]
    sn = np.zeros(D, np.float32)
    r = C.c_float()
    term = C.c_int()
    m = C.c_double()
    lib().orc_lingauss_step(_p(s), int(a), _p(A), _p(Bm), _p(noise), D, float(noise_std), float(done_norm), _p(sn),
                            C.byref(r), C.byref(term), C.byref(m))
    return sn, float(r.value), int(term.value), float(m.value)


def blob_floats(D, H, A, value_head=False):
    return int(lib().orc_blob_floats(D, H, A, int(bool(value_head))))


def mlp_forward(blob, D, H, A, x, value_head=False, f64=False):
    blob = np.ascontiguousarray(blob, np.float32)
    x = np.ascontiguousarray(x, np.float32)
    assert blob.size == blob_floats(D, H, A, value_head) and x.size == D
    if f64:
        out = np.zeros(A, np.float64)
        v = C.c_double()
        lib().orc_mlp_forward_f64(_p(blob), D, H, A, int(value_head), _p(x), _p(out), C.byref(v))
    else:
        out = np.zeros(A, np.float32)
        v = C.c_float()
        lib().orc_mlp_forward_f32(_p(blob), D, H, A, int(value_head), _p(x), _p(out), C.byref(v))
    return (out, v.value) if value_head else out


def bf16_round(x):
    return float(lib().orc_bf16_round(float(x)))


def argmax_lowest(q):
    q = np.ascontiguousarray(q, np.float32)
    return int(lib().orc_argmax_lowest(_p(q), q.size))


def select_eps_greedy(q, x0, x1, threshold):
    q = np.ascontiguousarray(q, np.float32)
    return int(lib().orc_select_eps_greedy(_p(q), q.size, int(x0), int(x1), int(threshold)))


def select_categorical(logits, u):
    lg = np.ascontiguousarray(logits, np.float32)
    logp = C.c_double()
    m = C.c_double()
    a = lib().orc_select_categorical(_p(lg), lg.size, float(u), C.byref(logp), C.byref(m))
    return int(a), float(logp.value), float(m.value)


def td_one(q_sel, q_next_max, r, done, gamma, kappa):
    td = C.c_double()
    hub = C.c_double()
    lib().orc_td_one(float(q_sel), float(q_next_max), float(r), int(done), float(gamma), float(kappa), C.byref(td),
                     C.byref(hub))
    return float(td.value), float(hub.value)


def sgd_step(theta, theta_target, D, H, A, obs, act, rew, next_obs, done, gamma, kappa, lr):
    """One minibatch update of Algorithm 1's form (semi-gradient of the mean Huber loss); returns (theta_new, loss)."""
    theta = np.ascontiguousarray(theta, np.float32)
    theta_target = np.ascontiguousarray(theta_target, np.float32)
    obs = np.ascontiguousarray(obs, np.float32)
    next_obs = np.ascontiguousarray(next_obs, np.float32)
    act = np.ascontiguousarray(act, np.int32)
    done = np.ascontiguousarray(done, np.int32)
    rew = np.ascontiguousarray(rew, np.float32)
    n = act.size
    assert theta.size == blob_floats(D, H, A) == theta_target.size and obs.size == n * D == next_obs.size
    out = np.zeros_like(theta)
    loss = C.c_double()
    fn = lib().orc_sgd_step
    fn.restype = None
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                   C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_double, C.c_void_p, C.c_void_p]
    fn(_p(theta), _p(theta_target), D, H, A, _p(obs), _p(act), _p(rew), _p(next_obs), _p(done), n, float(gamma),
       float(kappa), float(lr), _p(out), C.byref(loss))
    return out, loss.value


def adam_step(theta, theta_target, D, H, A, obs, act, rew, next_obs, done, gamma, kappa, lr, beta1, beta2, eps, t, m, v):
    """The gradient of sgd_step through Adam; returns (theta_new, m_new, v_new, loss)."""
    arrs = [np.ascontiguousarray(a, np.float32) for a in (theta, theta_target, obs, rew, next_obs, m, v)]
    theta, theta_target, obs, rew, next_obs, m, v = arrs
    act = np.ascontiguousarray(act, np.int32)
    done = np.ascontiguousarray(done, np.int32)
    n = act.size
    assert theta.size == blob_floats(D, H, A) == theta_target.size == m.size == v.size and obs.size == n * D
    t_out, m_out, v_out = np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta)
    loss = C.c_double()
    fn = lib().orc_adam_step
    fn.restype = None
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                   C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, C.c_int64,
                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    fn(_p(theta), _p(theta_target), D, H, A, _p(obs), _p(act), _p(rew), _p(next_obs), _p(done), n, float(gamma),
       float(kappa), float(lr), float(beta1), float(beta2), float(eps), int(t), _p(m), _p(v), _p(t_out), _p(m_out),
       _p(v_out), C.byref(loss))
    return t_out, m_out, v_out, loss.value


def ppo_step(theta, D, H, A, obs, act, logp_old, adv, ret, clip_eps, c_v, c_e, lr, beta1, beta2, eps, t, m, v):
    """One PPO minibatch update (clipped surrogate + value loss - entropy bonus, Adam); returns
    (theta_new, m_new, v_new, loss, stats[4])."""
    arrs = [np.ascontiguousarray(a, np.float32) for a in (theta, obs, logp_old, adv, ret, m, v)]
    theta, obs, logp_old, adv, ret, m, v = arrs
    act = np.ascontiguousarray(act, np.int32)
    n = act.size
    assert theta.size == blob_floats(D, H, A, True) == m.size == v.size and obs.size == n * D
    t_out, m_out, v_out = np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta)
    loss = C.c_double()
    stats = np.zeros(4, np.float64)
    fn = lib().orc_ppo_step
    fn.restype = None
    fn.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                   C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, C.c_int64,
                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    fn(_p(theta), D, H, A, _p(obs), _p(act), _p(logp_old), _p(adv), _p(ret), n, float(clip_eps), float(c_v), float(c_e),
       float(lr), float(beta1), float(beta2), float(eps), int(t), _p(m), _p(v), _p(t_out), _p(m_out), _p(v_out),
       C.byref(loss), _p(stats))
    return t_out, m_out, v_out, loss.value, stats


def gae(rew, val, done, gamma, lam):
    rew = np.ascontiguousarray(rew, np.float32)
    val = np.ascontiguousarray(val, np.float32)
    done = np.ascontiguousarray(done, np.uint8)
    T, N = rew.shape
    assert val.shape == (T + 1, N) and done.shape == (T, N)
    adv = np.zeros((T, N), np.float64)
    ret = np.zeros((T, N), np.float64)
    lib().orc_gae(_p(rew), _p(val), _p(done), T, N, float(gamma), float(lam), _p(adv), _p(ret))
    return adv, ret


def shuffle_index(seed, shuffle_id, R, i):
    """Row that position i of shuffle `shuffle_id` takes, out of R rows."""
    return int(lib().orc_shuffle_index(int(seed) & (2**64 - 1), int(shuffle_id) & (2**64 - 1), int(R), int(i)))


def shuffle_order(seed, shuffle_id, R):
    return np.array([shuffle_index(seed, shuffle_id, R, i) for i in range(R)], np.int64)


def normalize(x, eps=1e-8):
    x = np.ascontiguousarray(x, np.float32).ravel()
    out = np.zeros(x.size, np.float64)
    lib().orc_normalize(_p(x), x.size, float(eps), _p(out))
    return out


# --------------------------------------------------------------------------- the whole path
class Oracle:
    """The path as a state machine with the library's call semantics (see tj_oracle.h)."""

    def __init__(self, *, env_kind, n_envs, obs_dim, n_actions, hidden, policy_kind=0, weight_dtype=0, epsilon=0.1,
                 seed=0, replay_capacity=0, minibatch=1, staleness_bound=0, warmup=0, rollout_len=1,
                 target_sync_interval=0, n_segments=1, gamma=0.99, huber_delta=1.0, gae_lambda=0.95,
                 max_episode_steps=0, lg_done_norm=4.0, lg_noise_std=0.01, lg_A=None, lg_B=None, **_ignored):
        self._A = None if lg_A is None else np.ascontiguousarray(lg_A, np.float32)
        self._B = None if lg_B is None else np.ascontiguousarray(lg_B, np.float32)
        cfg = Config(env_kind, n_envs, obs_dim, n_actions, hidden, policy_kind, weight_dtype, epsilon,
                     int(seed) & (2**64 - 1), replay_capacity, minibatch, staleness_bound, warmup, rollout_len,
                     target_sync_interval, n_segments, gamma, huber_delta, gae_lambda, max_episode_steps,
                     lg_done_norm, lg_noise_std,
                     None if self._A is None else self._A.ctypes.data,
                     None if self._B is None else self._B.ctypes.data)
        st = C.c_int()
        self.cfg = cfg
        self._h = lib().orc_create(C.byref(cfg), C.byref(st))
        if not self._h:
            raise ValueError("oracle rejected the configuration (status %d)" % st.value)
        self.N, self.D, self.A, self.H = n_envs, obs_dim, n_actions, hidden
        self.S_d = lib().orc_state_dim(self._h)
        self.rec_words = lib().orc_record_words(self._h)
        self.value_head = policy_kind == POLICY_CATEGORICAL
        self.C = replay_capacity
        self.n_blob = blob_floats(obs_dim, hidden, n_actions, self.value_head)

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # calls
    def publish(self, blob):
        blob = np.ascontiguousarray(blob, np.float32)
        return lib().orc_publish(self._h, _p(blob), blob.size)

    def actor_step(self, n_steps=1):
        return lib().orc_actor_step(self._h, n_steps)

    def sample(self, staleness_bound=-1):
        B = self.cfg.minibatch
        idx = np.zeros(B, np.int32)
        rec = np.zeros((B, self.rec_words), np.float32)
        st = lib().orc_sample(self._h, staleness_bound, _p(idx), _p(rec))
        return st, idx, rec

    def td(self, records):
        rec = np.ascontiguousarray(records, np.float32)
        n = rec.shape[0]
        td = np.zeros(n)
        hub = np.zeros(n)
        qs = np.zeros(n)
        qn = np.zeros(n)
        loss = C.c_double()
        st = lib().orc_td(self._h, _p(rec), n, _p(td), _p(hub), C.byref(loss), _p(qs), _p(qn))
        return st, td, hub, float(loss.value), qs, qn

    def segment_acquire(self):
        seg = Segment()
        st = lib().orc_segment_acquire(self._h, C.byref(seg))
        if st != OK:
            return st, None
        T, N, D = seg.T, seg.N, self.D
        out = dict(T=T, N=N, version=seg.version,
                   obs=_view(seg.obs, (T, N, D), np.float32).copy(), act=_view(seg.act, (T, N), np.int32).copy(),
                   rew=_view(seg.rew, (T, N), np.float32).copy(), done=_view(seg.done, (T, N), np.uint8).copy(),
                   logp=_view(seg.logp, (T, N), np.float32).copy(),
                   val=_view(seg.val, (T + 1, N), np.float32).copy())
        return st, out

    def stats(self):
        s = Stats()
        lib().orc_get_stats(self._h, C.byref(s))
        d = {k: getattr(s, k) for k, _ in Stats._fields_ if k != "staleness_hist"}
        d["staleness_hist"] = list(s.staleness_hist)
        return d

    # state
    @property
    def state(self):
        return _view(lib().orc_state(self._h), (self.N, self.S_d), np.float32)

    @property
    def ep_step(self):
        return _view(lib().orc_ep_step(self._h), (self.N,), np.int32)

    def set_counters(self, cursor, t, k):
        lib().orc_set_counters(self._h, int(cursor), int(t), int(k))

    @property
    def cursor(self):
        return int(lib().orc_cursor(self._h))

    @property
    def ring(self):
        return _view(lib().orc_ring(self._h), (self.C, self.rec_words), np.float32)

    @property
    def block_version(self):
        return _view(lib().orc_block_version(self._h), (self.C // self.N,), np.int32)

    def last(self, name):
        shapes = {"obs": ((self.N, self.D), np.float32), "logits": ((self.N, self.A), np.float32),
                  "act": ((self.N,), np.int32), "rew": ((self.N,), np.float32), "done": ((self.N,), np.int32),
                  "next_obs": ((self.N, self.D), np.float32), "done_margin": ((self.N,), np.float64),
                  "act_margin": ((self.N,), np.float64), "logp": ((self.N,), np.float32),
                  "value": ((self.N,), np.float32)}
        shape, dt = shapes[name]
        return _view(getattr(lib(), "orc_last_" + name)(self._h), shape, dt)

    @property
    def online_blob(self):
        return _view(lib().orc_online_blob(self._h), (self.n_blob,), np.float32)

    @property
    def target_blob(self):
        return _view(lib().orc_target_blob(self._h), (self.n_blob,), np.float32)


def split_records(rec, D):
    """[n][2D+4] record rows -> dict of obs, next_obs, act, rew, done, ver."""
    rec = np.ascontiguousarray(rec, np.float32)
    ints = rec.view(np.int32)
    return dict(obs=rec[:, :D].copy(), next_obs=rec[:, D:2 * D].copy(), act=ints[:, 2 * D].copy(),
                rew=rec[:, 2 * D + 1].copy(), done=ints[:, 2 * D + 2].copy(), ver=ints[:, 2 * D + 3].copy())
