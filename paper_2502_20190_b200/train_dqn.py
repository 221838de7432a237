"""DQN on the vectorised CartPole env, driven entirely through the library's calls: tj_actor_step produces, tj_replay_sample
draws staleness-bounded minibatches, tj_adam_step learns, tj_publish_weights hands every new parameter version to the actor.

    python -m paper_2502_20190_b200.train_dqn [--staleness 1 8 64] [--iters 1500]

It is the paper's pipeline in miniature (Sec. 3.1: actor / buffer / learner; Sec. 3.3 and App. D.1: how stale the consumed
samples may be), used here to show that the pieces learn together and to compare staleness bounds on one GPU.  The mean
episode return is the episode length (reward 1 per step, cut at 500)."""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding, synth


def train(staleness_bound=8, iters=1500, n_envs=1024, hidden=64, minibatch=1024, updates_per_iter=4, lr=5e-4,
          target_every=200, epsilon=0.1, seed=1, report_every=100, device=0):
    """Runs `iters` iterations of (one env step of every env, `updates_per_iter` learner steps, each followed by a
    publish).  Returns a list of dicts: iteration, env steps, mean return of the episodes finished since the last report."""
    import torch
    torch.cuda.set_device(device)
    f = synth.config_fields({}, env_kind=synth.ENV_CARTPOLE, n_envs=n_envs, obs_dim=4, n_actions=2, hidden=hidden,
                            epsilon=epsilon, seed=seed, replay_capacity=n_envs * 128, minibatch=minibatch,
                            staleness_bound=staleness_bound, warmup=minibatch, target_sync_interval=target_every,
                            gamma=0.99, huber_delta=1.0, device=device)
    ctx = binding.Context(**f)
    theta = torch.from_numpy(synth.policy_blob(seed, 1, 4, hidden, 2)).cuda()
    theta_target = theta.clone()
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    batch = ctx.alloc_batch()
    ctx.publish_weights(theta)
    hist, t_adam, last_eps, last_ret, starved = [], 0, 0, 0.0, 0
    for it in range(1, iters + 1):
        ctx.actor_step(1)
        for _ in range(updates_per_iter):
            st, _ = ctx.replay_sample(batch=batch, allow=(0, binding.TJ_ERR_WARMUP, binding.TJ_ERR_STARVED))
            if st != 0:
                starved += 1
                continue
            t_adam += 1
            ctx.adam_step(batch, lr, theta, theta_target, m, v, t_adam)
            if t_adam % target_every == 0:
                theta_target.copy_(theta)
            ctx.publish_weights(theta)
        if it % report_every == 0 or it == iters:
            s = ctx.stats()
            n_ep = s["episodes_finished"] - last_eps
            mean_ret = (s["return_sum"] - last_ret) / n_ep if n_ep else float("nan")
            last_eps, last_ret = s["episodes_finished"], s["return_sum"]
            hist.append(dict(iter=it, env_steps=it * n_envs, updates=t_adam, episodes=int(n_ep), mean_return=float(mean_ret),
                             max_sampled_staleness=int(s["max_sampled_staleness"]), starved=starved))
    return hist


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--staleness", type=int, nargs="+", default=[8])
    ap.add_argument("--iters", type=int, default=1500)
    ap.add_argument("--envs", type=int, default=1024)
    ap.add_argument("--hidden", type=int, default=64)
    ap.add_argument("--seed", type=int, default=1)
    a = ap.parse_args()
    for S in a.staleness:
        h = train(staleness_bound=S, iters=a.iters, n_envs=a.envs, hidden=a.hidden, seed=a.seed)
        print(json.dumps(dict(staleness_bound=S, curve=[(r["env_steps"], round(r["mean_return"], 1)) for r in h],
                              final=h[-1])))


if __name__ == "__main__":
    main()
