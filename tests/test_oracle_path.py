"""Pins for the oracle's state machine (ring, versions, sampler, segments, counters):
brute force on tiny inputs, index formulas, invariants and the paper's special cases."""
import numpy as np
import pytest

from paper_2502_20190_b200 import synth


def _mk(orc, **kw):
    base = dict(env_kind=orc.ENV_CARTPOLE, n_envs=4, obs_dim=4, n_actions=2, hidden=8, epsilon=0.1, seed=1234,
                replay_capacity=16, minibatch=8, staleness_bound=2, warmup=4, target_sync_interval=3, gamma=0.99,
                huber_delta=1.0)
    base.update(kw)
    return orc.Oracle(**base)


def _uniform(orc, x, lo, width):
    """U(lo, lo+width) as one correctly rounded FP32 multiply-add of the exact uniform.  The product of two
    24-bit significands and the sum with a third of similar exponent are exact in double, so a single
    rounding to FP32 at the end is the fused result."""
    return np.float32(np.float64(orc.u01(int(x))) * np.float64(np.float32(width)) + np.float64(np.float32(lo)))


def _blob(o, version, seed=77):
    return synth.policy_blob(seed, version, o.D, o.H, o.A, o.value_head)


def test_statuses_before_weights_and_warmup(orc):
    o = _mk(orc, warmup=8)
    assert o.actor_step(1) == orc.ERR_NO_WEIGHTS
    assert o.sample()[0] == orc.ERR_NO_WEIGHTS
    assert o.publish(_blob(o, 1)) == 1
    assert o.sample()[0] == orc.ERR_WARMUP
    o.actor_step(1)
    assert o.sample()[0] == orc.ERR_WARMUP      # 4 < 8
    o.actor_step(1)
    assert o.sample()[0] == orc.OK
    with pytest.raises(ValueError):
        _mk(orc, replay_capacity=18)             # not a multiple of n_envs


def test_initial_state_comes_from_reset_stream(orc):
    o = _mk(orc)
    for e in range(o.N):
        w = orc.stream_words(1234, orc.STREAM_RESET, 0, e, 2**64 - 1)
        want = [_uniform(orc, x, -0.05, 0.1) for x in w]
        assert np.array_equal(o.state[e], np.array(want, np.float32))
        assert np.all(np.abs(o.state[e]) < 0.05)
    assert np.all(o.ep_step == 0)


def test_actor_step_is_the_composition_of_its_blocks(orc):
    """One env at a time in Python: observation -> MLP -> epsilon-greedy with the ACTION words of (e, t) ->
    CartPole step -> record at slot (cursor + e) mod C with the actor's version -> reset from RESET(e, t)."""
    o = _mk(orc, n_envs=3, replay_capacity=12, epsilon=0.3, max_episode_steps=7)
    blob = _blob(o, 1)
    o.publish(blob)
    thr = orc.explore_threshold(0.3)
    state = o.state.copy()
    ep = np.zeros(3, np.int32)
    ring = np.zeros((12, o.rec_words), np.float32)
    for t in range(30):
        if t == 11:
            blob = _blob(o, 2)
            o.publish(blob)
        ver = 1 if t < 11 else 2
        o.actor_step(1)
        for e in range(3):
            q = orc.mlp_forward(blob, 4, 8, 2, state[e])
            w = orc.stream_words(1234, orc.STREAM_ACTION, 0, e, t)
            a = orc.select_eps_greedy(q, w[0], w[1], thr)
            sn, r, term, _ = orc.cartpole_step(state[e], a)
            ep[e] += 1
            done = int(term or ep[e] >= 7)
            slot = (3 * t + e) % 12
            ring[slot, :4] = state[e]
            ring[slot, 4:8] = sn
            ring[slot].view(np.int32)[8] = a
            ring[slot, 9] = r
            ring[slot].view(np.int32)[10] = done
            ring[slot].view(np.int32)[11] = ver
            if done:
                rw = orc.stream_words(1234, orc.STREAM_RESET, 0, e, t)
                state[e] = [_uniform(orc, x, -0.05, 0.1) for x in rw]
                ep[e] = 0
            else:
                state[e] = sn
            assert o.last("act")[e] == a and o.last("done")[e] == done
        assert np.array_equal(o.state, state) and np.array_equal(o.ep_step, ep)
        assert np.array_equal(o.ring.view(np.int32), ring.view(np.int32))
        assert o.cursor == 3 * (t + 1)


def test_ring_index_arithmetic_against_a_list(orc):
    N, C = 4, 16
    o = _mk(orc, n_envs=N, replay_capacity=C)
    o.publish(_blob(o, 1))
    log = []  # (t, e) in write order
    for t in range(3 * (C // N) + 2):
        o.actor_step(1)
        log += [(t, e) for e in range(N)]
        assert o.cursor == len(log)
        resident = log[-C:]
        for (tt, e) in resident:
            slot = (tt % (C // N)) * N + e          # closed form of (cursor_at_write + e) mod C
            assert slot == (tt * N + e) % C
        # the resident steps are the last C/N steps; check through the stored observations' uniqueness of slots
        assert len({(tt * N + e) % C for tt, e in resident}) == min(len(log), C)
        assert sorted({tt for tt, _ in resident}) == list(range(max(0, t + 1 - C // N), t + 1))
    # each block carries the version in force when it was written
    assert np.all(o.block_version == 1)


def test_step_limit_truncates_at_exactly_500(orc):
    o = _mk(orc, n_envs=2, replay_capacity=4)
    o.publish(_blob(o, 1))
    upright = np.zeros((2, 4), np.float32)
    for t in range(1, 501):
        o.state[:] = upright                      # hold the pole upright so that only the limit can end it
        o.actor_step(1)
        done = o.last("done")
        assert np.all(done == (1 if t == 500 else 0)), t
    assert np.all(o.ep_step == 0)
    assert o.stats()["episodes_finished"] == 2 and o.stats()["return_sum"] == 1000.0


def _bruteforce_sample(orc, o, S, k, v_learner, valid):
    ver = o.ring.view(np.int32)[:, 2 * o.D + 3]
    E = [i for i in range(valid) if v_learner - int(ver[i]) <= S]
    idx = []
    for j in range(o.cfg.minibatch):
        w = orc.stream_words(o.cfg.seed, orc.STREAM_SAMPLE, 0, j, k)
        idx.append(E[(int(w[0]) * len(E)) >> 32] if E else -1)
    return E, idx


def test_sampler_against_bruteforce_enumeration(orc):
    o = _mk(orc, n_envs=4, replay_capacity=32, minibatch=16, staleness_bound=2, warmup=4)
    v = 0
    k = 0
    for t in range(40):
        if t % 3 == 0:
            v += 1
            o.publish(_blob(o, v))
        o.actor_step(1)
        valid = min(o.cursor, 32)
        for S in (0, 1, 2, 5, 1000):
            E, want = _bruteforce_sample(orc, o, S, k, v, valid)
            st, idx, rec = o.sample(S)
            assert st == orc.OK and idx.tolist() == want
            k += 1
            ver = rec.view(np.int32)[:, 2 * o.D + 3]
            assert np.all(v - ver <= S)                         # the staleness invariant
            assert np.array_equal(rec, o.ring[idx])             # gather copies rows bit for bit
            if S == 0:
                assert np.all(ver == v)                          # "all samples new"
            if S == 1000:
                assert len(E) == valid                           # no bound -> uniform over what is resident


def test_sampler_starved_and_determinism(orc):
    o = _mk(orc, n_envs=4, replay_capacity=16, minibatch=8, staleness_bound=0, warmup=0)
    o.publish(_blob(o, 1))
    o.actor_step(2)
    o.publish(_blob(o, 2))                                       # learner moves on, nothing fresh yet
    st, _, _ = o.sample()
    assert st == orc.ERR_STARVED and o.stats()["starved_calls"] == 1 and o.stats()["learner_steps"] == 0
    st, idx1, _ = o.sample(1)
    assert st == orc.OK
    o2 = _mk(orc, n_envs=4, replay_capacity=16, minibatch=8, staleness_bound=0, warmup=0)
    o2.publish(_blob(o2, 1)); o2.actor_step(2); o2.publish(_blob(o2, 2))
    o2.sample()
    assert np.array_equal(o2.sample(1)[1], idx1)                 # same seed, same k -> same indices


def test_sampler_uniform_over_eligible(orc):
    o = _mk(orc, n_envs=8, replay_capacity=64, minibatch=64, staleness_bound=100, warmup=0)
    o.publish(_blob(o, 1))
    o.actor_step(8)
    counts = np.zeros(64)
    draws = 0
    for _ in range(400):
        _, idx, _ = o.sample()
        np.add.at(counts, idx, 1)
        draws += 64
    chi2 = np.sum((counts - draws / 64) ** 2 / (draws / 64))
    assert chi2 < 63 + 5 * np.sqrt(2 * 63)


def test_eligible_fraction_in_steady_state(orc):
    """With p actor steps and one publish per learner step, a ring of C slots holds C/N steps and the records
    at most S versions old are the last (S+1)*p steps: |E|/C = min(1, (S+1) p N / C) up to one block."""
    N, C, p = 4, 64, 2
    o = _mk(orc, n_envs=N, replay_capacity=C, minibatch=4, warmup=0)
    v = 0
    for it in range(40):
        v += 1
        o.publish(_blob(o, v))
        o.actor_step(p)
    ver = o.ring.view(np.int32)[:, 2 * o.D + 3]
    for S in (0, 1, 3, 6, 20):
        frac = np.mean(v - ver <= S)
        assert abs(frac - min(1.0, (S + 1) * p * N / C)) <= N / C + 1e-12


def test_target_network_cadence(orc):
    o = _mk(orc, target_sync_interval=3, warmup=0, staleness_bound=100)
    b1 = _blob(o, 1)
    o.publish(b1)
    assert np.array_equal(o.target_blob, b1) and np.array_equal(o.online_blob, b1)
    o.actor_step(1)
    blobs = {1: b1}
    last_sync_k, target_v = 0, 1
    for v in range(2, 12):
        o.sample()                                               # learner step k = v - 1
        blobs[v] = _blob(o, v)
        o.publish(blobs[v])
        k = v - 1
        if k - last_sync_k >= 3:
            last_sync_k, target_v = k, v
        assert np.array_equal(o.online_blob, blobs[v])
        assert np.array_equal(o.target_blob, blobs[target_v])


def test_td_on_a_batch_reduces_to_algorithm_1_when_target_equals_online(orc):
    o = _mk(orc, warmup=0, target_sync_interval=1)
    blob = _blob(o, 1)
    o.publish(blob)
    o.actor_step(4)
    _, idx, rec = o.sample()
    st, td, hub, loss, qs, qn = o.td(rec)
    assert st == orc.OK
    r = orc.split_records(rec, 4)
    for j in range(rec.shape[0]):
        v_s = orc.mlp_forward(blob, 4, 8, 2, r["obs"][j])
        v_n = orc.mlp_forward(blob, 4, 8, 2, r["next_obs"][j])
        delta = float(r["rew"][j]) + 0.99 * (1 - r["done"][j]) * float(v_n.max()) - float(v_s[r["act"][j]])
        assert abs(td[j] - delta) < 1e-6
    assert abs(loss - hub.mean()) < 1e-12
    assert np.all(hub >= 0) and np.all((np.abs(td) <= 1) == (np.abs(hub - 0.5 * td * td) < 1e-15))


def test_bf16_mode_rounds_weight_matrices_only(orc):
    o = _mk(orc, weight_dtype=orc.W_BF16)
    blob = _blob(o, 1)
    blob[o.H * o.D: o.H * o.D + o.H] = 0.123456789               # a bias that is not bf16-representable
    o.publish(blob)
    got = o.online_blob
    W1 = got[:o.H * o.D]
    assert np.all((W1.view(np.uint32) & 0xFFFF) == 0)
    assert np.allclose(W1, blob[:o.H * o.D], rtol=2 ** -8)
    assert np.array_equal(got[o.H * o.D: o.H * o.D + o.H], blob[o.H * o.D: o.H * o.D + o.H])


def test_counters_follow_the_producer_consumer_ratio(orc):
    o = _mk(orc, n_envs=4, replay_capacity=64, minibatch=8, staleness_bound=50, warmup=0)
    o.publish(_blob(o, 1))
    for _ in range(10):
        o.actor_step(4)
        o.sample()
    s = o.stats()
    assert s["produced"] == 10 * 4 * 4 and s["consumed"] == 10 * 8
    assert s["actor_steps"] == 40 and s["learner_steps"] == 10
    assert sum(s["staleness_hist"]) == s["consumed"] and s["max_sampled_staleness"] == 0


# ------------------------------------------------------------------ on-policy segments
def _mk_seg(orc, **kw):
    base = dict(env_kind=orc.ENV_CARTPOLE, n_envs=3, obs_dim=4, n_actions=2, hidden=8, policy_kind=1, seed=99,
                replay_capacity=0, rollout_len=5, n_segments=3, staleness_bound=1, gamma=0.99, gae_lambda=0.95)
    base.update(kw)
    return orc.Oracle(**base)


def test_segment_contents_and_bootstrap_value(orc):
    o = _mk_seg(orc)
    blob = _blob(o, 1)
    o.publish(blob)
    assert o.segment_acquire()[0] == orc.ERR_STARVED
    states = []
    for t in range(5):
        states.append(o.state.copy())
        o.actor_step(1)
        if t < 4:
            assert o.segment_acquire()[0] == orc.ERR_STARVED   # still filling
    st, seg = o.segment_acquire()
    assert st == orc.OK and seg["version"] == 1 and seg["T"] == 5
    for t in range(5):
        for e in range(3):
            lg, v = orc.mlp_forward(blob, 4, 8, 2, states[t][e], value_head=True)
            u = orc.u01(int(orc.stream_words(99, orc.STREAM_ACTION, 0, e, t)[0]))
            a, logp, _ = orc.select_categorical(lg, u)
            assert np.array_equal(seg["obs"][t, e], states[t][e])
            assert seg["act"][t, e] == a and seg["val"][t, e] == np.float32(v)
            assert abs(seg["logp"][t, e] - logp) < 1e-6
    for e in range(3):
        _, v = orc.mlp_forward(blob, 4, 8, 2, o.state[e], value_head=True)
        assert seg["val"][5, e] == np.float32(v)
    assert o.segment_acquire()[0] == orc.ERR_STARVED            # consumed once only


def test_segment_staleness_drop_and_overwrite(orc):
    o = _mk_seg(orc, staleness_bound=1)
    o.publish(_blob(o, 1))
    o.actor_step(5)                     # segment 0, version 1
    o.publish(_blob(o, 2))
    o.actor_step(5)                     # segment 1, version 2
    o.publish(_blob(o, 3))              # learner at 3: segment 0 is 2 behind -> dropped, segment 1 is fine
    st, seg = o.segment_acquire()
    assert st == orc.OK and seg["version"] == 2
    s = o.stats()
    assert s["dropped_stale"] == 15 and s["consumed"] == 15 and s["max_sampled_staleness"] == 1
    # producer laps the consumer: 4 more segments into 3 slots, the oldest unconsumed one is overwritten
    o.actor_step(20)
    assert o.stats()["dropped_overwritten"] == 15
    versions = []
    while True:
        st, seg = o.segment_acquire()
        if st != orc.OK:
            break
        versions.append(seg["version"])
    assert versions == [3, 3, 3]


def test_gae_on_an_acquired_segment(orc):
    o = _mk_seg(orc, n_envs=4, rollout_len=40, max_episode_steps=9)
    o.publish(_blob(o, 1))
    o.actor_step(40)
    _, seg = o.segment_acquire()
    assert seg["done"].sum() > 0
    adv, ret = orc.gae(seg["rew"], seg["val"], seg["done"], 0.99, 0.95)
    # lambda-return identity: R_t = r_t + gamma (1-d_t) ((1-lambda) V_{t+1} + lambda R_{t+1}), R_T := V_T
    R_next = seg["val"][40].astype(np.float64)
    for t in range(39, -1, -1):
        nd = 1.0 - seg["done"][t]
        R = seg["rew"][t] + 0.99 * nd * ((1 - 0.95) * seg["val"][t + 1] + 0.95 * R_next)
        assert np.allclose(ret[t], R, atol=1e-9)
        R_next = R


# ------------------------------------------------------------------ the other two environments
# The building blocks used below (stream words, normals, uniforms, the env steps, the MLP, the selection rule) each have
# their own pins; these tests pin how the state machine puts them together for the linear-Gaussian and the Acrobot
# environments: which Philox stream, block, env and step index feeds what, the reset range, what the record holds.
def _mk_lingauss(orc, D, **kw):
    A, B = synth.lingauss_matrices(4321, D, 5)
    base = dict(env_kind=orc.ENV_LINGAUSS, n_envs=3, obs_dim=D, n_actions=5, hidden=8, epsilon=0.25, seed=4321,
                replay_capacity=12, minibatch=4, staleness_bound=2, warmup=0, gamma=0.99, huber_delta=1.0, lg_A=A, lg_B=B)
    base.update(kw)
    return orc.Oracle(**base), base["lg_A"], base["lg_B"]


def _bf16_weights(orc, blob, D, H, A):
    """The blob with its three weight matrices rounded to bfloat16 (biases untouched)."""
    out = blob.copy()
    spans = [(0, H * D), (H * D + H, H * D + H + H * H), (H * D + H + H * H + H, H * D + H + H * H + H + A * H)]
    for lo, hi in spans:
        out[lo:hi] = [orc.bf16_round(x) for x in blob[lo:hi]]
    return out


@pytest.mark.parametrize("D,done_norm,bf16", [(8, 1.9, False), (128, 7.2, False), (8, 1.9, True)])
def test_lingauss_actor_step_is_the_composition_of_its_blocks(orc, D, done_norm, bf16):
    o, A, B = _mk_lingauss(orc, D, lg_done_norm=done_norm, max_episode_steps=6,
                           weight_dtype=orc.W_BF16 if bf16 else orc.W_FP32)
    blob = _blob(o, 1)
    o.publish(blob)
    used = _bf16_weights(orc, blob, D, 8, 5) if bf16 else blob
    thr = orc.explore_threshold(0.25)
    # initial states: RESET words of block b, env e at the all-ones step, U(-0.1, 0.1), components 4b .. 4b+3
    state = np.zeros((3, D), np.float32)
    for e in range(3):
        for b in range(D // 4):
            w = orc.stream_words(4321, orc.STREAM_RESET, b, e, 2**64 - 1)
            state[e, 4 * b:4 * b + 4] = [_uniform(orc, x, -0.1, 0.2) for x in w]
    assert np.array_equal(o.state, state) and np.all(np.abs(state) < 0.1) and np.abs(state).max() > 0.05
    ep = np.zeros(3, np.int32)
    ring = np.zeros((12, o.rec_words), np.float32)
    n_term = n_trunc = n_alive = 0
    for t in range(14):
        o.actor_step(1)
        for e in range(3):
            if bf16:
                q = orc.mlp_forward(used, D, 8, 5, state[e], f64=True).astype(np.float32)
            else:
                q = orc.mlp_forward(used, D, 8, 5, state[e])
            w = orc.stream_words(4321, orc.STREAM_ACTION, 0, e, t)
            a = orc.select_eps_greedy(q, w[0], w[1], thr)
            noise = np.concatenate([orc.normal4(orc.stream_words(4321, orc.STREAM_NOISE, b, e, t)) for b in range(D // 4)])
            # the configuration holds both constants as FP32
            sn, r, term, _ = orc.lingauss_step(state[e], a, A, B, noise, float(np.float32(0.01)), float(np.float32(done_norm)))
            ep[e] += 1
            done = int(term or ep[e] >= 6)
            n_term += term
            n_trunc += int(not term and ep[e] >= 6)
            n_alive += 1 - done
            slot = (3 * t + e) % 12
            ring[slot, :D] = state[e]
            ring[slot, D:2 * D] = sn
            ring[slot].view(np.int32)[2 * D] = a
            ring[slot, 2 * D + 1] = r
            ring[slot].view(np.int32)[2 * D + 2] = done
            ring[slot].view(np.int32)[2 * D + 3] = 1
            assert np.array_equal(o.last("logits")[e], q)
            assert o.last("act")[e] == a and o.last("done")[e] == done and o.last("rew")[e] == np.float32(r)
            if done:
                for b in range(D // 4):
                    rw = orc.stream_words(4321, orc.STREAM_RESET, b, e, t)
                    state[e, 4 * b:4 * b + 4] = [_uniform(orc, x, -0.1, 0.2) for x in rw]
                ep[e] = 0
            else:
                state[e] = sn
        assert np.array_equal(o.state, state) and np.array_equal(o.ep_step, ep)
        assert np.array_equal(o.ring.view(np.int32), ring.view(np.int32))
    assert n_term > 0 and n_alive > 0        # the chosen threshold exercises both branches
    assert n_trunc > 0 or D == 128


def test_lingauss_noise_blocks_are_distinct_per_block_env_and_step(orc):
    """A wrong block, env or step index in the noise keying would repeat normals somewhere: with A = 0 and B = 0 the new
    state is 0.01 times the normals, so every component of every env at every step must differ."""
    D = 16
    o, _, _ = _mk_lingauss(orc, D, lg_A=np.zeros((D, D), np.float32), lg_B=np.zeros((5, D), np.float32), lg_done_norm=1e9)
    o.publish(_blob(o, 1))
    seen = []
    for t in range(3):
        o.actor_step(1)
        seen.append(o.last("next_obs").copy())
    allv = np.concatenate([s.ravel() for s in seen])
    assert len(np.unique(allv)) == allv.size
    assert abs(allv.std() / 0.01 - 1.0) < 0.2
    # and each is 0.01 * the normal of its (block, env, step)
    for t in range(3):
        for e in range(3):
            for b in range(D // 4):
                z = orc.normal4(orc.stream_words(4321, orc.STREAM_NOISE, b, e, t))
                assert np.array_equal(seen[t][e, 4 * b:4 * b + 4], (float(np.float32(0.01)) * z).astype(np.float32))


def test_lingauss_default_step_limit_is_200(orc):
    D = 8
    o, _, _ = _mk_lingauss(orc, D, lg_A=np.zeros((D, D), np.float32), lg_B=np.zeros((5, D), np.float32), lg_noise_std=0.0,
                           n_envs=2, replay_capacity=4)
    o.publish(_blob(o, 1))
    for t in range(1, 201):
        o.actor_step(1)
        assert np.all(o.last("done") == (1 if t == 200 else 0)), t
        assert np.all(o.last("rew") == 0.0)
    assert np.all(o.ep_step == 0) and o.stats()["episodes_finished"] == 2


def _mk_acrobot(orc, **kw):
    base = dict(env_kind=orc.ENV_ACROBOT, n_envs=3, obs_dim=6, n_actions=3, hidden=8, epsilon=0.3, seed=777,
                replay_capacity=12, minibatch=4, staleness_bound=2, warmup=0, gamma=0.99, huber_delta=1.0)
    base.update(kw)
    return orc.Oracle(**base)


def test_acrobot_actor_step_is_the_composition_of_its_blocks(orc):
    """The record holds the six-component observation of the state before and after the step, the state itself stays
    four angles and velocities; reset U(-0.1, 0.1)^4 from RESET block 0; reward 0 on a terminating step, -1 otherwise."""
    o = _mk_acrobot(orc, max_episode_steps=9)
    blob = _blob(o, 1)
    o.publish(blob)
    thr = orc.explore_threshold(0.3)
    state = np.zeros((3, 4), np.float32)
    for e in range(3):
        w = orc.stream_words(777, orc.STREAM_RESET, 0, e, 2**64 - 1)
        state[e] = [_uniform(orc, x, -0.1, 0.2) for x in w]
    assert np.array_equal(o.state, state) and np.abs(state).max() > 0.05
    # one env is started near the top so that a terminating step occurs within the run
    state[2] = np.array([3.0, 0.1, 0.5, 0.0], np.float32)
    o.state[2] = state[2]
    ep = np.zeros(3, np.int32)
    ring = np.zeros((12, o.rec_words), np.float32)
    n_term = 0
    for t in range(20):
        o.actor_step(1)
        for e in range(3):
            obs = orc.acrobot_obs(state[e])
            q = orc.mlp_forward(blob, 6, 8, 3, obs)
            w = orc.stream_words(777, orc.STREAM_ACTION, 0, e, t)
            a = orc.select_eps_greedy(q, w[0], w[1], thr)
            sn, r, term, _ = orc.acrobot_step(state[e], a)
            assert r == (0.0 if term else -1.0)
            n_term += term
            ep[e] += 1
            done = int(term or ep[e] >= 9)
            slot = (3 * t + e) % 12
            ring[slot, :6] = obs
            ring[slot, 6:12] = orc.acrobot_obs(sn)
            ring[slot].view(np.int32)[12] = a
            ring[slot, 13] = r
            ring[slot].view(np.int32)[14] = done
            ring[slot].view(np.int32)[15] = 1
            assert o.last("act")[e] == a and o.last("done")[e] == done
            if done:
                rw = orc.stream_words(777, orc.STREAM_RESET, 0, e, t)
                state[e] = [_uniform(orc, x, -0.1, 0.2) for x in rw]
                ep[e] = 0
            else:
                state[e] = sn
        assert np.array_equal(o.state, state) and np.array_equal(o.ep_step, ep)
        assert np.array_equal(o.ring.view(np.int32), ring.view(np.int32))
    assert n_term > 0


def test_acrobot_default_step_limit_is_500(orc):
    o = _mk_acrobot(orc, n_envs=2, replay_capacity=4)
    o.publish(_blob(o, 1))
    hanging = np.zeros((2, 4), np.float32)
    for t in range(1, 501):
        o.state[:] = hanging                       # at rest, hanging down: the tip stays far below the line
        o.actor_step(1)
        assert np.all(o.last("done") == (1 if t == 500 else 0)), t
        assert np.all(o.last("rew") == -1.0)
    assert o.stats()["episodes_finished"] == 2 and o.stats()["return_sum"] == -1000.0
