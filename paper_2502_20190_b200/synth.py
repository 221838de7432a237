"""Seeded synthetic inputs and the five workload definitions.

This module holds none of the method's arithmetic: it only names the workload
shapes and draws the arrays (policy weights, the linear-Gaussian env's A and B)
that are handed, unchanged, to whichever implementation consumes them.
"""
from __future__ import annotations

import numpy as np

ENV_CARTPOLE, ENV_ACROBOT, ENV_LINGAUSS = 0, 1, 2
POLICY_EPS_GREEDY, POLICY_CATEGORICAL = 0, 1
W_FP32, W_BF16, W_FP32_TC = 0, 1, 2

SEED = 0x25022019

# The five workloads.  "actor_steps" and "cadence" describe how a driver loops
# over the calls; the rest are configuration fields.
WORKLOADS = {
    "cfg1": dict(env_kind=ENV_CARTPOLE, n_envs=64, obs_dim=4, n_actions=2, hidden=64, policy_kind=POLICY_EPS_GREEDY,
                 weight_dtype=W_FP32, epsilon=0.1, replay_capacity=65536, minibatch=256, staleness_bound=4,
                 warmup=256, target_sync_interval=1000, gamma=0.99, huber_delta=1.0,
                 actor_steps=1000, actor_per_learner=4, publish_every_actor_steps=50),
    "cfg2": dict(env_kind=ENV_CARTPOLE, n_envs=4096, obs_dim=4, n_actions=2, hidden=128,
                 policy_kind=POLICY_EPS_GREEDY, weight_dtype=W_FP32, epsilon=0.1, replay_capacity=1048576,
                 minibatch=1024, staleness_bound=8, warmup=1024, target_sync_interval=1000, gamma=0.99,
                 huber_delta=1.0, actor_steps=10000, actor_per_learner=4, publish_every_learner_steps=1),
    "cfg3": dict(env_kind=ENV_ACROBOT, n_envs=16384, obs_dim=6, n_actions=3, hidden=256,
                 policy_kind=POLICY_EPS_GREEDY, weight_dtype=W_FP32, epsilon=0.1, replay_capacity=1 << 22,
                 minibatch=4096, staleness_bound=4, warmup=4096, target_sync_interval=1000, gamma=0.99,
                 huber_delta=1.0, actor_steps=10000, actor_per_learner=4, publish_every_learner_steps=1,
                 staleness_sweep=(1, 4, 16)),
    "cfg4": dict(env_kind=ENV_CARTPOLE, n_envs=65536, obs_dim=4, n_actions=2, hidden=256,
                 policy_kind=POLICY_CATEGORICAL, weight_dtype=W_FP32, epsilon=0.0, replay_capacity=0,
                 rollout_len=128, n_segments=3, staleness_bound=2, gamma=0.99, gae_lambda=0.95,
                 actor_steps=128 * 8),
    "cfg5": dict(env_kind=ENV_LINGAUSS, n_envs=262144, obs_dim=128, n_actions=16, hidden=512,
                 policy_kind=POLICY_EPS_GREEDY, weight_dtype=W_BF16, epsilon=0.1, replay_capacity=1 << 24,
                 minibatch=8192, staleness_bound=16, warmup=8192, target_sync_interval=1000, gamma=0.99,
                 huber_delta=1.0, actor_steps=1000, actor_per_learner=4, publish_every_learner_steps=1,
                 staleness_sweep=(1, 2, 4, 8, 16)),
}

_CONFIG_KEYS = ("env_kind", "n_envs", "obs_dim", "n_actions", "hidden", "policy_kind", "weight_dtype", "epsilon",
                "seed", "replay_capacity", "minibatch", "staleness_bound", "warmup", "rollout_len",
                "target_sync_interval", "n_segments", "gamma", "huber_delta", "gae_lambda", "max_episode_steps",
                "lg_done_norm", "lg_noise_std", "lg_A", "lg_B")


def config_fields(workload: dict, **overrides) -> dict:
    """The configuration fields of a workload (driver-loop keys removed), with overrides applied."""
    w = dict(workload)
    w.update(overrides)
    w.setdefault("seed", SEED)
    if w["env_kind"] == ENV_LINGAUSS and w.get("lg_A") is None:
        A, B = lingauss_matrices(w["seed"], w["obs_dim"], w["n_actions"])
        w["lg_A"], w["lg_B"] = A, B
    return {k: w[k] for k in _CONFIG_KEYS if k in w}


def blob_floats(D: int, H: int, A: int, value_head: bool) -> int:
    return H * D + H + H * H + H + A * H + A + ((H + 1) if value_head else 0)


def bf16_representable(x: np.ndarray) -> np.ndarray:
    """Drop the low 16 bits of FP32 values so that they survive a bfloat16 store unchanged."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


def policy_blob(seed: int, version: int, D: int, H: int, A: int, value_head: bool = False,
                bf16_exact: bool = False) -> np.ndarray:
    """Policy parameters for one version: weights N(0, 1/fan_in), biases 0, laid out
    [W1 HxD, b1 H, W2 HxH, b2 H, W3 AxH, b3 A (, Wv H, bv 1)] row-major (out x in)."""
    rng = np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(version)]))
    parts = []
    for n_out, n_in in ((H, D), (H, H), (A, H)) + (((1, H),) if value_head else ()):
        W = (rng.standard_normal((n_out, n_in)) / np.sqrt(n_in)).astype(np.float32)
        if bf16_exact:
            W = bf16_representable(W)
        parts += [W.ravel(), np.zeros(n_out, np.float32)]
    blob = np.concatenate(parts).astype(np.float32)
    assert blob.size == blob_floats(D, H, A, value_head)
    return blob


def lingauss_matrices(seed: int, D: int, n_actions: int, bias_scale: float = 1.0):
    """A [D][D] with entries N(0, 1/D) and per-action bias B [n_actions][D] with entries N(0, bias_scale^2)."""
    rng = np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), 0xA0B0]))
    A = (rng.standard_normal((D, D)) / np.sqrt(D)).astype(np.float32)
    B = (bias_scale * rng.standard_normal((n_actions, D))).astype(np.float32)
    return A, B


def gae_inputs(seed: int, T: int, N: int, done_rate: float = 0.01):
    """Synthetic rollout arrays for GAE alone: rewards 1, values N(0,1)*10, dones Bernoulli(done_rate)."""
    rng = np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), 0x6AE]))
    rew = np.ones((T, N), np.float32)
    val = (10.0 * rng.standard_normal((T + 1, N))).astype(np.float32)
    done = (rng.random((T, N)) < done_rate).astype(np.uint8)
    return rew, val, done
