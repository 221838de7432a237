"""Production / consumption balance on one GPU (Sec. 3.3, Eq. 2-3 of the paper, read for a time-shared device).

The paper fixes the share of consumed to produced samples, P = B_s / N_s' (Eq. 2 with N_s' the samples produced per
consumed batch), and splits M cores between learners and actors so that the training and production throughputs meet
(Eq. 3: max min(TR_L, TR_A) s.t. N_c / N_s' = P, M_L + M_A = M, TR_L ~ TR_A).  On one GPU the resource that is split is
time: with R_A env steps per second while only the actor runs and R_L samples per second while only the learner runs, a
fraction f of the time on the actor produces f R_A and the rest consumes (1 - f) R_L.  The constraint
(1 - f) R_L = P f R_A gives f = R_L / (R_L + P R_A): both sides then run exactly as fast as the ratio allows, which is
the balanced point (more actor time would only produce samples that are never consumed, Table 1's L2A16 / L2A24 rows).
Host arithmetic only; nothing here touches the GPU."""
from __future__ import annotations

import math


def actor_steps_per_learner_step(P: float, minibatch: int, n_envs: int) -> int:
    """How many env steps of all n_envs the actor takes per learner step so that consumed / produced = P:
    minibatch / (k * n_envs) = P, k rounded to the nearest positive integer."""
    if P <= 0 or minibatch <= 0 or n_envs <= 0:
        raise ValueError("P, minibatch and n_envs must be positive")
    return max(1, int(round(minibatch / (P * n_envs))))


def realised_ratio(k: int, minibatch: int, n_envs: int, updates: int = 1) -> float:
    """consumed / produced with k actor steps per `updates` learner steps"""
    return updates * minibatch / (k * n_envs)


def schedule(P: float, minibatch: int, n_envs: int) -> tuple:
    """(k, u): k actor steps of all n_envs, then u learner steps, so that u * minibatch / (k * n_envs) is as close to P as
    whole numbers allow with one of the two equal to 1 (the cadence that keeps the consumed samples freshest: the learner
    never waits for more than one block when it consumes faster than one minibatch per block, and never runs more than
    its share ahead otherwise)."""
    if P <= 0 or minibatch <= 0 or n_envs <= 0:
        raise ValueError("P, minibatch and n_envs must be positive")
    per_block = P * n_envs / minibatch            # learner steps per actor step at ratio P
    if per_block >= 1.0:
        return 1, max(1, int(round(per_block)))
    return max(1, int(round(1.0 / per_block))), 1


def time_share(R_A: float, R_L: float, P: float) -> dict:
    """The balanced split of device time.  R_A: env steps/s of the actor alone, R_L: samples/s of the learner alone,
    P: consumed per produced sample.  Returns the actor's time fraction and the two throughputs at that point."""
    if R_A <= 0 or R_L <= 0 or P <= 0:
        raise ValueError("rates and P must be positive")
    f = R_L / (R_L + P * R_A)
    return dict(actor_fraction=f, produced_per_s=f * R_A, consumed_per_s=(1.0 - f) * R_L)


def rates_from_stats(stats: dict, produced: int, consumed: int) -> tuple:
    """(R_A, R_L) from a context's per-kernel-class times (tj_set_profiling on): classes 0-2 are the actor's kernels,
    3-5 and 7 the learner's (sample + gather, TD error, the publish that hands each new version over, update)."""
    ms = stats["kernel_ms"]
    t_a = (ms[0] + ms[1] + ms[2]) * 1e-3
    t_l = (ms[3] + ms[4] + ms[5] + ms[7]) * 1e-3
    if t_a <= 0 or t_l <= 0:
        raise ValueError("no timed launches: call tj_set_profiling(1) before the steps")
    return produced / t_a, consumed / t_l


def starved_fraction(staleness_bound: int, publishes_per_block: float) -> float:
    """Share of sample calls that find nothing eligible when every produced block (one actor step of all envs) is
    followed by `publishes_per_block` version bumps and only versions within `staleness_bound` may be consumed: a block
    written at version v is eligible for calls at versions v .. v + S, i.e. for S + 1 of the publishes_per_block calls
    that follow it before the next block arrives (the consumer-ahead-of-producer case of Sec. 3.3)."""
    if publishes_per_block <= 0:
        raise ValueError("publishes_per_block must be positive")
    return max(0.0, 1.0 - (staleness_bound + 1) / publishes_per_block)


def balanced_cadence(actor_step_s: float, learner_step_s: float, minibatch: int, n_envs: int, staleness_bound: int,
                     max_steps: int = 64) -> dict:
    """Cadence for CONCURRENT actor and learner streams (Sec. 3.1, Fig. 2; Eq. 3's TR_L ~ TR_A): per iteration the actor
    takes k env steps of all n_envs while the learner takes u steps on what was produced before, so an iteration lasts about
    max(k * actor_step_s, u * learner_step_s) and neither stream idles when the two are equal.  With one parameter version
    per iteration the consumed samples are at most one iteration behind, so any bound >= 1 admits the cadence; bound 0 needs
    the streams in lock step (k = u = 1 and no overlap).  Returns k, u (one of them 1, the other at most max_steps), the
    realised consumed : produced ratio P, both streams' busy time per iteration and the share of the iteration the slower
    one leaves the faster one idle."""
    if actor_step_s <= 0 or learner_step_s <= 0:
        raise ValueError("step times must be positive")
    if staleness_bound < 1:
        k, u = 1, 1
    elif actor_step_s >= learner_step_s:
        k, u = 1, max(1, min(max_steps, int(round(actor_step_s / learner_step_s))))
    else:
        k, u = max(1, min(max_steps, int(round(learner_step_s / actor_step_s)))), 1
    t_a, t_l = k * actor_step_s, u * learner_step_s
    return dict(actor_steps=k, learner_steps=u, P=realised_ratio(k, minibatch, n_envs, u), actor_busy_s=t_a, learner_busy_s=t_l,
                idle_share=abs(t_a - t_l) / max(t_a, t_l))


def step_times_from_stats(stats: dict, actor_steps: int, learner_steps: int) -> tuple:
    """(seconds per actor step of all envs, seconds per learner step) from a context's per-kernel-class times."""
    ms = stats["kernel_ms"]
    t_a = (ms[0] + ms[1] + ms[2]) * 1e-3
    t_l = (ms[3] + ms[4] + ms[5] + ms[7]) * 1e-3
    if actor_steps <= 0 or learner_steps <= 0 or t_a <= 0 or t_l <= 0:
        raise ValueError("no timed launches")
    return t_a / actor_steps, t_l / learner_steps
