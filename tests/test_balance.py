"""Host arithmetic of the production / consumption balance (Sec. 3.3, Eq. 2-3) and its agreement with the oracle's
sampler: the predicted share of starved sample calls is what the oracle's replay path shows."""
import numpy as np
import pytest

import oracle
from paper_2502_20190_b200 import balance, synth


def test_ratio_and_time_share_closed_forms():
    # cfg2's stated 4:1 producer:consumer cadence with minibatch 1,024 and 4,096 envs is P = 1/16
    assert balance.actor_steps_per_learner_step(1 / 16, 1024, 4096) == 4
    assert balance.realised_ratio(4, 1024, 4096) == 1 / 16
    # P = B_s / N_s (Eq. 2): consuming every produced sample once is one learner step per minibatch / n_envs actor steps
    assert balance.actor_steps_per_learner_step(1.0, 4096, 1024) == 4
    s = balance.time_share(R_A=2.0e8, R_L=1.0e7, P=1 / 16)
    assert s["consumed_per_s"] == pytest.approx(s["produced_per_s"] / 16)            # the constraint N_c / N_s' = P
    assert 0 < s["actor_fraction"] < 1
    # any other split lowers min(consumption, P * production): the balanced point is the maximum of Eq. 3's objective
    best = min(s["consumed_per_s"], s["produced_per_s"] / 16)
    for f in np.linspace(0.01, 0.99, 99):
        assert min((1 - f) * 1.0e7, f * 2.0e8 / 16) <= best * (1 + 1e-12)
    # a faster learner shifts time to the actor
    assert balance.time_share(2.0e8, 4.0e7, 1 / 16)["actor_fraction"] > s["actor_fraction"]
    with pytest.raises(ValueError):
        balance.time_share(0, 1, 1)


def test_schedule_realises_the_ratio_with_whole_steps():
    for P, B, N in [(1 / 16, 1024, 4096), (4.0, 1024, 1024), (1.0, 4096, 1024), (1 / 8, 512, 512), (1.0, 1024, 1024)]:
        k, u = balance.schedule(P, B, N)
        assert min(k, u) == 1
        assert balance.realised_ratio(k, B, N, u) == pytest.approx(P)
    # not representable exactly: the nearest whole cadence
    k, u = balance.schedule(0.3, 1024, 1024)
    assert (k, u) == (3, 1) and balance.realised_ratio(k, 1024, 1024, u) == pytest.approx(1 / 3)
    assert balance.schedule(2.4, 1024, 1024) == (1, 2)
    with pytest.raises(ValueError):
        balance.schedule(0, 1, 1)


@pytest.mark.parametrize("S,publishes", [(0, 4), (1, 4), (3, 4), (1, 2), (2, 8)])
def test_starved_share_matches_the_oracle_sampler(S, publishes):
    """One actor step (one block), then `publishes` rounds of sample + publish, repeated: the oracle's sampler starves in
    exactly the predicted share of calls."""
    N, D, A, H = 8, 4, 2, 8
    f = synth.config_fields({}, env_kind=synth.ENV_CARTPOLE, n_envs=N, obs_dim=D, n_actions=A, hidden=H, epsilon=0.1, seed=3,
                            replay_capacity=N * 64, minibatch=4, staleness_bound=S, warmup=1, target_sync_interval=1000,
                            gamma=0.99, huber_delta=1.0)
    o = oracle.Oracle(**f)
    ver = 1
    o.publish(synth.policy_blob(3, ver, D, H, A))
    calls = starved = 0
    for _ in range(12):
        o.actor_step(1)
        for _ in range(publishes):
            st, _, _ = o.sample()
            calls += 1
            starved += st != 0
            ver += 1
            o.publish(synth.policy_blob(3, ver, D, H, A))
    assert starved / calls == pytest.approx(balance.starved_fraction(S, publishes))


def test_balanced_cadence_for_concurrent_streams():
    """Eq. 3's TR_L ~ TR_A for two streams: the faster side takes as many steps as fit into one step of the slower one."""
    c = balance.balanced_cadence(actor_step_s=100e-6, learner_step_s=25e-6, minibatch=1024, n_envs=4096, staleness_bound=8)
    assert (c["actor_steps"], c["learner_steps"]) == (1, 4) and c["idle_share"] == pytest.approx(0.0)
    assert c["P"] == pytest.approx(4 * 1024 / 4096)
    c = balance.balanced_cadence(actor_step_s=10e-6, learner_step_s=72e-6, minibatch=256, n_envs=64, staleness_bound=4)
    assert (c["actor_steps"], c["learner_steps"]) == (7, 1) and c["idle_share"] < 0.05
    # both streams busy for about the same time: no other small-integer cadence with one side at 1 idles less
    for k in range(1, 20):
        assert abs(k * 10e-6 - 72e-6) / max(k * 10e-6, 72e-6) >= c["idle_share"] - 1e-12
    # bound 0 ("all samples new") cannot overlap production and consumption: lock step
    c0 = balance.balanced_cadence(10e-6, 72e-6, 256, 64, staleness_bound=0)
    assert (c0["actor_steps"], c0["learner_steps"]) == (1, 1)
    with pytest.raises(ValueError):
        balance.balanced_cadence(0.0, 1.0, 1, 1, 1)
    a, l = balance.step_times_from_stats(dict(kernel_ms=[8.0, 0, 0, 1.0, 2.0, 0.5, 0, 0.5]), actor_steps=4, learner_steps=2)
    assert a == pytest.approx(2e-3) and l == pytest.approx(2e-3)
