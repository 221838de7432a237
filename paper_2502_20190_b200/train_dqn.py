"""DQN on the vectorised CartPole env, driven entirely through the library's calls: tj_actor_step produces, tj_replay_sample
draws staleness-bounded minibatches, tj_adam_step learns, tj_publish_weights hands every new parameter version to the actor.

    python -m paper_2502_20190_b200.train_dqn [--staleness 1 8 64] [--iters 1500]

It is the paper's pipeline in miniature (Sec. 3.1: actor / buffer / learner; Sec. 3.3 and App. D.1: how stale the consumed
samples may be), used here to show that the pieces learn together and to compare staleness bounds on one GPU.  The mean
episode return is the episode length (reward 1 per step, cut at 500)."""
from __future__ import annotations

import argparse
import json
import time

import numpy as np

from . import balance, binding, synth


def train(staleness_bound=8, iters=1500, n_envs=1024, hidden=64, minibatch=1024, updates_per_iter=4, lr=5e-4,
          target_every=200, epsilon=0.1, seed=1, report_every=100, device=0, actor_steps_per_iter=1, rates_out=None,
          two_stream=False, auto_balance=False):
    """Runs `iters` iterations of (`actor_steps_per_iter` env steps of every env, `updates_per_iter` learner steps, each
    followed by a publish).  Returns a list of dicts: iteration, env steps, mean return of the episodes finished since the
    last report.  With `rates_out` (a dict) the per-kernel times are recorded and the dict receives the actor's and the
    learner's stand-alone rates (Eq. 3's TR_A, TR_L: env steps and consumed samples per second of their own kernel time),
    the balanced time split for the realised ratio and the throughput that split predicts.
    two_stream: the learner's calls run on a second CUDA stream; the iteration is software-pipelined (the learner works on what
    was produced up to the previous iteration while the actor produces the next block with the parameters published one
    iteration earlier), one parameter version per iteration.  auto_balance: every report interval the measured per-step
    kernel times of the two sides set the cadence for the next interval (balance.balanced_cadence: Eq. 3's TR_L ~ TR_A)."""
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
    if two_stream:
        ctx.use_learner_stream(True)
    if rates_out is not None or auto_balance:
        ctx.set_profiling(1)
    cadence_log = []
    hist, t_adam, last_eps, last_ret, starved = [], 0, 0, 0.0, 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    env_steps_done, win_actor, win_learner = 0, 0, 0
    lstream = getattr(ctx, "learner_stream", None) if two_stream else None
    if two_stream:
        ctx.actor_step(actor_steps_per_iter)           # the pipeline's first block
        env_steps_done += actor_steps_per_iter * n_envs
    for it in range(1, iters + 1):
        if not two_stream:
            ctx.actor_step(actor_steps_per_iter)
            env_steps_done += actor_steps_per_iter * n_envs
            win_actor += actor_steps_per_iter
        published = False
        for _ in range(updates_per_iter):
            st, _ = ctx.replay_sample(batch=batch, allow=(0, binding.TJ_ERR_WARMUP, binding.TJ_ERR_STARVED))
            if st != 0:
                starved += 1
                continue
            t_adam += 1
            win_learner += 1
            ctx.adam_step(batch, lr, theta, theta_target, m, v, t_adam)
            if t_adam % target_every == 0:
                if lstream is not None:
                    with torch.cuda.stream(lstream):
                        theta_target.copy_(theta)
                else:
                    theta_target.copy_(theta)
            if not two_stream:
                ctx.publish_weights(theta)
            published = True
        if two_stream:
            # the next block is produced while the updates above run; then one version for the iteration
            ctx.actor_step(actor_steps_per_iter)
            env_steps_done += actor_steps_per_iter * n_envs
            win_actor += actor_steps_per_iter
            if published:
                ctx.publish_weights(theta)
        if it % report_every == 0 or it == iters:
            s = ctx.stats()
            n_ep = s["episodes_finished"] - last_eps
            mean_ret = (s["return_sum"] - last_ret) / n_ep if n_ep else float("nan")
            last_eps, last_ret = s["episodes_finished"], s["return_sum"]
            hist.append(dict(iter=it, env_steps=env_steps_done, updates=t_adam, episodes=int(n_ep), mean_return=float(mean_ret),
                             max_sampled_staleness=int(s["max_sampled_staleness"]), starved=starved))
            if auto_balance and win_actor and win_learner:
                tau_a, tau_l = balance.step_times_from_stats(s, win_actor, win_learner)
                c = balance.balanced_cadence(tau_a, tau_l, minibatch, n_envs, staleness_bound)
                actor_steps_per_iter, updates_per_iter = c["actor_steps"], c["learner_steps"]
                cadence_log.append(dict(iter=it, actor_step_us=tau_a * 1e6, learner_step_us=tau_l * 1e6, **c))
                ctx.set_profiling(0)
                ctx.set_profiling(1)                   # a fresh window
                win_actor = win_learner = 0
    torch.cuda.synchronize()
    loop_s = time.perf_counter() - t0
    if rates_out is not None and auto_balance:
        rates_out.update(loop_s=loop_s, loop_produced_per_s=env_steps_done / loop_s, loop_consumed_per_s=t_adam * minibatch / loop_s,
                         cadence=cadence_log)
    elif rates_out is not None:
        produced, consumed = env_steps_done, t_adam * minibatch
        R_A, R_L = balance.rates_from_stats(ctx.stats(), produced, consumed)
        P = consumed / produced
        rates_out.update(R_A=R_A, R_L=R_L, P=P, loop_s=loop_s, loop_produced_per_s=produced / loop_s,
                         kernel_s=sum(ctx.stats()["kernel_ms"]) * 1e-3, **balance.time_share(R_A, R_L, P))
    return hist


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--staleness", type=int, nargs="+", default=[8])
    ap.add_argument("--iters", type=int, default=1500)
    ap.add_argument("--envs", type=int, default=1024)
    ap.add_argument("--hidden", type=int, default=64)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--ratio", type=float, default=None,
                    help="consumed : produced samples (Eq. 2's P); sets the actor / learner cadence through balance.schedule")
    ap.add_argument("--two-stream", action="store_true", help="learner on a second CUDA stream, iterations software-pipelined")
    ap.add_argument("--auto-balance", action="store_true", help="set the cadence from the measured step times (Eq. 3)")
    a = ap.parse_args()
    k, u = (1, 4) if a.ratio is None else balance.schedule(a.ratio, 1024, a.envs)
    for S in a.staleness:
        rates = {}
        h = train(staleness_bound=S, iters=a.iters, n_envs=a.envs, hidden=a.hidden, seed=a.seed, actor_steps_per_iter=k,
                  updates_per_iter=u, rates_out=rates, two_stream=a.two_stream, auto_balance=a.auto_balance)
        print(json.dumps(dict(staleness_bound=S, actor_steps_per_iter=k, updates_per_iter=u, balance=rates,
                              curve=[(r["env_steps"], round(r["mean_return"], 1)) for r in h], final=h[-1])))


if __name__ == "__main__":
    main()
