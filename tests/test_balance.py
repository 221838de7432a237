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
