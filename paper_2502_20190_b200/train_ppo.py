"""PPO on the vectorised CartPole env through the library's calls, with a chosen sample staleness.

    python -m paper_2502_20190_b200.train_ppo [--lag 0 1 2 4] [--iters 150]

Per iteration the actor rolls out one segment with the newest published parameters (tj_actor_step), the learner takes the
oldest unconsumed segment (tj_segment_acquire), computes advantages (tj_gae), runs a few epochs of minibatch updates
over shuffled rows (tj_normalize, tj_segment_minibatch, tj_ppo_step) and publishes the result as the next parameter
version (tj_publish_weights).  With `lag` segments rolled out
ahead of the first update, every consumed segment is exactly `lag` versions older than the learner -- the on-policy form of
the staleness that the paper controls through its production/consumption balance (Sec. 3.3; the "New / Lag" curves of
Sec. 4.3.2 and App. D.1).  lag = 0 is the synchronous mode of App. C.  The library's staleness bound is set to `lag`, so a
staler segment would be dropped, and the statistics confirm none is.

Every arithmetic step runs in the library's kernels; torch only holds the device arrays."""
from __future__ import annotations

import argparse
import json

from . import binding, synth


def train(lag=0, iters=150, n_envs=1024, rollout=32, hidden=64, minibatch=4096, epochs=4, lr=1e-3, clip_eps=0.2, c_v=0.5,
          c_e=0.01, gamma=0.99, lam=0.95, seed=1, device=0):
    """Returns a list of dicts per iteration: env steps produced, mean return of the episodes finished in the iteration,
    version lag of the consumed segment, PPO statistics of the last minibatch."""
    import torch
    torch.cuda.set_device(device)
    f = synth.config_fields({}, env_kind=synth.ENV_CARTPOLE, n_envs=n_envs, obs_dim=4, n_actions=2, hidden=hidden,
                            policy_kind=1, seed=seed, replay_capacity=0, rollout_len=rollout, n_segments=lag + 2,
                            staleness_bound=lag, minibatch=minibatch, gamma=gamma, gae_lambda=lam, device=device)
    ctx = binding.Context(**f)
    theta = torch.from_numpy(synth.policy_blob(seed, 1, 4, hidden, 2, True)).cuda()
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ctx.publish_weights(theta)
    for _ in range(lag):                       # the producer runs `lag` segments ahead of the consumer
        ctx.actor_step(rollout)
    hist, t_adam, last_eps, last_ret = [], 0, 0, 0.0
    n_shuffles, mbs = 0, {}
    rows = rollout * n_envs
    for it in range(1, iters + 1):
        ctx.actor_step(rollout)
        st, seg = ctx.segment_acquire(allow=(0, binding.TJ_ERR_STARVED))
        if st != 0:
            continue
        seg_lag = ctx.stats()["learner_version"] - seg["version"]
        adv, ret = ctx.gae(seg["rew"], seg["val"], seg["done"], gamma, lam)
        ctx.normalize(adv, 1e-8, out=adv)              # advantages of the segment: mean 0, variance 1
        stats = None
        for _ in range(epochs):
            n_shuffles += 1                            # a fresh row order per epoch
            for r0 in range(0, rows, minibatch):
                n = min(rows, r0 + minibatch) - r0
                mb = mbs.get(n) or mbs.setdefault(n, ctx.alloc_minibatch(n))
                ctx.segment_minibatch(seg, adv, ret, n_shuffles, r0, mb)
                t_adam += 1
                stats = ctx.ppo_step(mb["obs"], mb["act"], mb["logp_old"], mb["adv"], mb["ret"], lr, theta, m, v, t_adam,
                                     clip_eps, c_v, c_e)
        ctx.publish_weights(theta)
        s = ctx.stats()
        n_ep = s["episodes_finished"] - last_eps
        mean_ret = (s["return_sum"] - last_ret) / n_ep if n_ep else float("nan")
        last_eps, last_ret = s["episodes_finished"], s["return_sum"]
        st_host = [float(x) for x in stats.cpu().tolist()]
        hist.append(dict(iter=it, env_steps=(it + lag) * rows, mean_return=float(mean_ret), episodes=int(n_ep),
                         segment_lag=int(seg_lag), loss=st_host[0], entropy=st_host[3], clip_fraction=st_host[4],
                         dropped_stale=int(s["dropped_stale"])))
    return hist


def env_steps_to(hist, threshold):
    """env steps at the first iteration from which three consecutive iteration means stay at or above the threshold"""
    r = [x["mean_return"] for x in hist]
    for i in range(len(r) - 2):
        if min(r[i:i + 3]) >= threshold:
            return hist[i]["env_steps"]
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--lag", type=int, nargs="+", default=[0])
    ap.add_argument("--iters", type=int, default=150)
    ap.add_argument("--seed", type=int, default=1)
    a = ap.parse_args()
    for lag in a.lag:
        h = train(lag=lag, iters=a.iters, seed=a.seed)
        print(json.dumps(dict(lag=lag, seed=a.seed, env_steps_to_300=env_steps_to(h, 300), env_steps_to_475=env_steps_to(h, 475),
                              max_segment_lag=max(r["segment_lag"] for r in h),
                              curve=[(r["env_steps"], round(r["mean_return"], 1)) for r in h[::5]], final=h[-1])))


if __name__ == "__main__":
    main()
