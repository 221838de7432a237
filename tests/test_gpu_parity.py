"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200).

Integer and index results (actions, slots, version tags, sampled indices, counters) must match bit for bit;
FP32 results within 1e-5 relative (|g-o| <= rtol*|o| + rtol*rms(o)).  Each actor step is compared from an
identical state: the GPU's state is copied into the oracle before the step.  Threshold decisions (done) are
compared exactly whenever the oracle's distance to the threshold exceeds the tolerance; the rest are counted.
"""
import numpy as np
import pytest

from parity_util import (RTOL_FP32, Tally, blob_for, close, compare_ring_step, fields_for, lockstep_step, make_pair,
                         measured_margin)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import oracle
    from paper_2502_20190_b200 import binding, build
    build.build()
    oracle.build()
    return torch, oracle, binding


def _small(**kw):
    base = dict(env_kind=0, n_envs=37, obs_dim=4, n_actions=2, hidden=24, epsilon=0.2, seed=4242, replay_capacity=37 * 8,
                minibatch=19, staleness_bound=2, warmup=37, target_sync_interval=3, gamma=0.99, huber_delta=1.0)
    base.update(kw)
    return fields_for(**base)


# ------------------------------------------------------------------------------------------------ set-up
@pytest.mark.parametrize("kind,D,A", [(0, 4, 2), (1, 6, 3), (2, 16, 5)])
def test_initial_states_are_bit_exact(env, kind, D, A):
    torch, orc, binding = env
    f = _small(env_kind=kind, obs_dim=D, n_actions=A, n_envs=70, replay_capacity=140)
    ctx, o = make_pair(orc, binding, **f)
    st = ctx.get_state()
    assert np.array_equal(st["state"].cpu().numpy(), o.state)
    assert np.all(st["ep_step"].cpu().numpy() == 0)
    assert st["cursor"] == 0 and st["t"] == 0 and st["actor_version"] == 0


def test_statuses(env):
    torch, orc, binding = env
    f = _small()
    ctx, o = make_pair(orc, binding, **f)
    b = binding
    assert b.tj_actor_step(ctx.h, 1, 0) == b.TJ_ERR_NO_WEIGHTS
    batch = ctx.alloc_batch()
    assert b.tj_replay_sample(ctx.h, -1, 0, batch["c"]) == b.TJ_ERR_NO_WEIGHTS
    assert b.tj_td_error(ctx.h, batch["c"], 0, 0, 0) == b.TJ_ERR_NO_WEIGHTS
    assert b.tj_publish_weights(ctx.h, 0, 0, 0)[0] == b.TJ_ERR_INVALID_ARG
    blob = blob_for(f, 1)
    assert b.tj_publish_weights(ctx.h, blob.ctypes.data, blob.size * 4 - 4, 0)[0] == b.TJ_ERR_INVALID_ARG
    assert ctx.publish_weights(blob) == 1
    assert b.tj_replay_sample(ctx.h, -1, 0, batch["c"]) == b.TJ_ERR_WARMUP
    assert b.tj_actor_step(ctx.h, -1, 0) == b.TJ_ERR_INVALID_ARG
    ctx.actor_step(1)
    assert b.tj_replay_sample(ctx.h, -1, 0, batch["c"]) == b.TJ_OK
    ctx.publish_weights(blob_for(f, 2))
    assert b.tj_replay_sample(ctx.h, 0, 0, batch["c"]) == b.TJ_ERR_STARVED
    assert "staleness" in b.tj_last_error(ctx.h)
    s = ctx.stats()
    assert s["starved_calls"] == 1 and s["learner_steps"] == 1 and s["device_error"] == 0


# ------------------------------------------------------------------------------------------------ actor
def test_cfg1_full_run_lockstep(env):
    """CartPole 64 envs x 1000 steps, 4-64-64-2, eps 0.1, version bump every 50 steps, learner step every 4."""
    torch, orc, binding = env
    f = fields_for("cfg1")
    ctx, o = make_pair(orc, binding, **f)
    tally = Tally()
    dbg = torch.empty((ctx.N, ctx.A), dtype=torch.float32, device=ctx.device)
    version = 0
    for t in range(1000):
        if t % 50 == 0:
            version += 1
            blob = blob_for(f, version)
            assert ctx.publish_weights(blob) == version == o.publish(blob)
        r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=0, tally=tally, dbg=dbg)
        compare_ring_step(r, o, rtol=RTOL_FP32, env_kind=0, tally=tally)
        if t % 4 == 3:
            gst, batch = ctx.replay_sample(allow=(0, -6, -7))
            ost, oidx, orec = o.sample()
            assert gst == ost
            if gst == 0:
                assert np.array_equal(batch["idx"].cpu().numpy(), oidx)
                assert np.array_equal(batch["ver"].cpu().numpy(), orec.view(np.int32)[:, 11])
                assert int((version - batch["ver"]).max().item()) <= f["staleness_bound"]
    tally.report("cfg1 lock-step")
    assert tally.ambiguous_done <= 0.001 * tally.total + 2
    gs, os_ = ctx.stats(), o.stats()
    for key in ("produced", "consumed", "dropped_stale", "starved_calls", "actor_steps", "learner_steps",
                "max_sampled_staleness", "episodes_finished", "staleness_hist", "actor_version"):
        assert gs[key] == os_[key], key
    assert abs(gs["return_sum"] - os_["return_sum"]) < 1e-6 * max(1.0, os_["return_sum"])
    assert gs["device_error"] == 0


@pytest.mark.parametrize("kind,D,A,H,N,steps", [(0, 4, 2, 24, 37, 120), (1, 6, 3, 40, 101, 150), (0, 4, 2, 128, 300, 40),
                                                (1, 6, 3, 256, 70, 30)])
def test_small_env_lockstep_ragged_shapes(env, kind, D, A, H, N, steps):
    torch, orc, binding = env
    f = _small(env_kind=kind, obs_dim=D, n_actions=A, hidden=H, n_envs=N, replay_capacity=N * 5, warmup=N,
               max_episode_steps=23)
    ctx, o = make_pair(orc, binding, **f)
    tally = Tally()
    for t in range(steps):
        if t % 17 == 0:
            blob = blob_for(f, t // 17 + 1)
            ctx.publish_weights(blob)
            o.publish(blob)
        r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=kind, tally=tally)
        scale = float(np.sqrt(np.mean(r["o_logits"].astype(np.float64) ** 2)))
        compare_ring_step(r, o, rtol=RTOL_FP32, env_kind=kind, tally=tally, act_exact=(kind != 1),
                          act_margin_scale=8 * RTOL_FP32 * scale)
    tally.report("small env lock-step kind %d H %d N %d" % (kind, H, N))
    assert tally.ambiguous_done <= 0.002 * tally.total + 2 and tally.ambiguous_act <= 0.002 * tally.total + 2
    assert ctx.stats()["episodes_finished"] > 0


@pytest.mark.parametrize("wd", [0, 1])
def test_lingauss_lockstep(env, wd):
    torch, orc, binding = env
    f = _small(env_kind=2, obs_dim=128, n_actions=16, hidden=48, n_envs=45, replay_capacity=45 * 4, warmup=45,
               weight_dtype=wd, max_episode_steps=6, lg_done_norm=9.5)
    ctx, o = make_pair(orc, binding, **f)
    tally = Tally()
    rtol = RTOL_FP32 if wd == 0 else 2e-2
    for t in range(25):
        if t % 10 == 0:
            blob = blob_for(f, t // 10 + 1)
            ctx.publish_weights(blob)
            o.publish(blob)
        r = lockstep_step(ctx, o, torch, rtol=rtol, env_kind=2, tally=tally, logits_exact=(wd == 0))
        compare_ring_step(r, o, rtol=RTOL_FP32, env_kind=2, tally=tally, act_exact=(wd == 0),
                          act_margin_scale=measured_margin(r["g_logits"], r["o_logits"]))
    st = ctx.stats()
    amb_act, _ = tally.report("LinGauss lock-step weight_dtype %d" % wd)
    assert st["episodes_finished"] > 0 and tally.ambiguous_done <= 0.01 * tally.total + 2
    assert amb_act <= 0.08


def test_lingauss_literal_constants_terminate_almost_every_step(env):
    """With B[a] ~ N(0,1) the post-step norm is about 7 > 4, so nearly every env finishes on every step."""
    torch, orc, binding = env
    f = _small(env_kind=2, obs_dim=128, n_actions=16, hidden=32, n_envs=64, replay_capacity=64 * 4, warmup=64)
    ctx, o = make_pair(orc, binding, **f)
    blob = blob_for(f, 1)
    ctx.publish_weights(blob)
    o.publish(blob)
    tally = Tally()
    for _ in range(5):
        r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=2, tally=tally)
        compare_ring_step(r, o, rtol=RTOL_FP32, env_kind=2, tally=tally)
    assert ctx.stats()["episodes_finished"] >= 0.95 * 5 * 64


def test_multi_step_launch_equals_single_steps(env):
    """n_steps inside one launch must give bit-identical states, rings and counters to n launches of one step."""
    torch, orc, binding = env
    for kind, D, A in ((0, 4, 2), (1, 6, 3), (2, 32, 7)):
        f = _small(env_kind=kind, obs_dim=D, n_actions=A, n_envs=77, replay_capacity=77 * 4, max_episode_steps=9,
                   lg_done_norm=3.0)
        a = binding.Context(**f)
        b_ = binding.Context(**f)
        blob = blob_for(f, 1)
        a.publish_weights(blob)
        b_.publish_weights(blob)
        a.actor_step(11)
        for _ in range(11):
            b_.actor_step(1)
        sa, sb = a.get_state(), b_.get_state()
        assert torch.equal(sa["state"], sb["state"]) and torch.equal(sa["ep_step"], sb["ep_step"])
        assert sa["cursor"] == sb["cursor"] == 77 * 11
        assert torch.equal(a.ring_view()[0].view(torch.int32), b_.ring_view()[0].view(torch.int32))
        assert torch.equal(a.ring_view()[1], b_.ring_view()[1])
        assert a.stats()["episodes_finished"] == b_.stats()["episodes_finished"] > 0


# ------------------------------------------------------------------------------------------------ learner
def test_sampler_indices_match_for_every_bound(env):
    torch, orc, binding = env
    f = _small(n_envs=16, replay_capacity=16 * 12, minibatch=64, warmup=16, staleness_bound=3)
    ctx, o = make_pair(orc, binding, **f)
    tally = Tally()
    v = 0
    for t in range(40):
        if t % 2 == 0:
            v += 1
            blob = blob_for(f, v)
            ctx.publish_weights(blob)
            o.publish(blob)
        lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=0, tally=tally)
        for S in (0, 1, 3, 7, 100):
            gst, batch = ctx.replay_sample(S, allow=(0, -7))
            ost, oidx, orec = o.sample(S)
            assert gst == ost == 0
            idx = batch["idx"].cpu().numpy()
            assert np.array_equal(idx, oidx)
            ring = ctx.ring_view()[0]
            rows = ring[batch["idx"].long()].cpu().numpy()
            D = 4
            assert np.array_equal(batch["obs"].cpu().numpy(), rows[:, :D])           # gather is a bit-exact copy
            assert np.array_equal(batch["next_obs"].cpu().numpy(), rows[:, D:2 * D])
            assert np.array_equal(batch["act"].cpu().numpy(), rows.view(np.int32)[:, 2 * D])
            assert np.array_equal(batch["rew"].cpu().numpy(), rows[:, 2 * D + 1])
            assert np.array_equal(batch["done"].cpu().numpy(), rows.view(np.int32)[:, 2 * D + 2])
            ver = batch["ver"].cpu().numpy()
            assert np.array_equal(ver, orec.view(np.int32)[:, 2 * D + 3]) and np.all(v - ver <= S)
    gs, os_ = ctx.stats(), o.stats()
    assert gs["staleness_hist"] == os_["staleness_hist"] and gs["consumed"] == os_["consumed"]
    assert gs["dropped_stale"] == os_["dropped_stale"] and gs["max_sampled_staleness"] == os_["max_sampled_staleness"]


def test_sampler_many_blocks(env):
    """More ring blocks than one pass of the eligible-list kernel handles (N small, C large)."""
    torch, orc, binding = env
    f = _small(n_envs=2, replay_capacity=2 * 3000, minibatch=257, warmup=2, staleness_bound=5, max_episode_steps=50)
    ctx, o = make_pair(orc, binding, **f)
    v = 0
    for it in range(30):
        v += 1
        blob = blob_for(f, v)
        ctx.publish_weights(blob)
        o.publish(blob)
        ctx.actor_step(150)
        o.actor_step(150)
        for S in (0, 5, 11):
            gst, batch = ctx.replay_sample(S)
            ost, oidx, _ = o.sample(S)
            assert gst == ost == 0 and np.array_equal(batch["idx"].cpu().numpy(), oidx)


@pytest.mark.parametrize("kind,D,A,H,B", [(0, 4, 2, 64, 256), (1, 6, 3, 256, 77), (2, 128, 16, 40, 50)])
def test_td_error_parity(env, kind, D, A, H, B):
    torch, orc, binding = env
    f = _small(env_kind=kind, obs_dim=D, n_actions=A, hidden=H, n_envs=32, replay_capacity=32 * 16, minibatch=B,
               warmup=32, staleness_bound=50, target_sync_interval=2, max_episode_steps=11, lg_done_norm=9.0)
    ctx, o = make_pair(orc, binding, **f)
    fresh = orc.Oracle(**dict(f, target_sync_interval=1))     # a learner whose target network never lags
    tally = Tally()
    lagging_versions = 0
    for v in range(1, 6):
        blob = blob_for(f, v)
        ctx.publish_weights(blob)
        o.publish(blob)
        fresh.publish(blob)
        for _ in range(4):
            lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=kind, tally=tally)
        _, batch = ctx.replay_sample()
        o.sample()
        fresh.set_counters(0, 0, v)                            # one learner step per version, as on the other two
        out = ctx.td_error(batch)
        # the oracle evaluates the batch the GPU gathered
        rec = np.zeros((B, 2 * D + 4), np.float32)
        rec[:, :D] = batch["obs"].cpu().numpy()
        rec[:, D:2 * D] = batch["next_obs"].cpu().numpy()
        rec.view(np.int32)[:, 2 * D] = batch["act"].cpu().numpy()
        rec[:, 2 * D + 1] = batch["rew"].cpu().numpy()
        rec.view(np.int32)[:, 2 * D + 2] = batch["done"].cpu().numpy()
        st, td, hub, loss, qs, qn = o.td(rec)
        assert st == 0
        # delta is a difference of O(1) numbers: its error is relative to the terms, not to the difference
        terms = np.abs(qs) + np.abs(qn) + np.abs(rec[:, 2 * D + 1])
        g_td = out["td"].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g_td - td) <= RTOL_FP32 * (np.abs(td) + terms))
        g_h = out["huber"].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g_h - hub) <= 2 * RTOL_FP32 * (hub + terms * np.maximum(1.0, np.abs(td))))
        assert abs(float(out["loss"].item()) - loss) <= 2 * RTOL_FP32 * (abs(loss) + float(terms.mean()))
        # The target network lags: refreshed on the first publish and then after every second learner step, it is the
        # newest parameters at versions 1, 3, 5 and one version behind at 2 and 4.  There the GPU's TD errors must
        # follow the lagging target, i.e. differ from those of a learner whose target is always the newest.
        assert np.array_equal(o.online_blob, blob)
        if v in (2, 4):
            assert np.array_equal(o.target_blob, blob_for(f, v - 1)) and not np.array_equal(o.target_blob, o.online_blob)
            _, td_fresh, _, _, _, _ = fresh.td(rec)
            moved = np.abs(td_fresh - td) > 100 * RTOL_FP32 * (np.abs(td) + terms)
            live = rec.view(np.int32)[:, 2 * D + 2] == 0       # a done row has no bootstrap term, so no target at all
            assert moved[live].mean() > 0.9
            assert np.all(np.abs(g_td - td_fresh)[moved] > RTOL_FP32 * (np.abs(td) + terms)[moved])
            lagging_versions += 1
        else:
            assert np.array_equal(o.target_blob, blob)
    assert lagging_versions == 2


def test_gae_parity_and_closed_forms(env):
    torch, orc, binding = env
    from paper_2502_20190_b200 import synth
    f = _small()
    ctx = binding.Context(**f)
    for T, N, rate in ((128, 1000, 0.02), (5, 33, 0.3), (1, 1, 0.0), (40, 4097, 0.0)):
        rew, val, done = synth.gae_inputs(7, T, N, rate)
        rew = (rew * np.random.default_rng(1).standard_normal((T, N))).astype(np.float32)
        adv, ret = ctx.gae(torch.from_numpy(rew).cuda(), torch.from_numpy(val).cuda(), torch.from_numpy(done).cuda(),
                           0.99, 0.95)
        o_adv, o_ret = orc.gae(rew, val, done, 0.99, 0.95)
        close(adv.cpu().numpy(), o_adv, RTOL_FP32, "adv")
        close(ret.cpu().numpy(), o_ret, RTOL_FP32, "ret")
    # full size of the on-policy workload: r = 1, V = 0, no dones => A_t = (1 - (g l)^(T-t)) / (1 - g l)
    T, N = 128, 65536
    rew = torch.ones((T, N), device="cuda")
    val = torch.zeros((T + 1, N), device="cuda")
    done = torch.zeros((T, N), dtype=torch.uint8, device="cuda")
    adv, ret = ctx.gae(rew, val, done, 0.99, 0.95)
    gl = 0.99 * 0.95
    want = (1 - gl ** (T - np.arange(T))) / (1 - gl)
    assert torch.equal(adv, ret)
    close(adv[:, ::4099].cpu().numpy(), np.repeat(want[:, None], adv[:, ::4099].shape[1], 1), RTOL_FP32, "closed form")
    assert torch.equal(adv[:, :1].expand(T, N), adv)
    # empty input is accepted and does nothing
    assert binding.tj_gae(ctx.h, rew.data_ptr(), val.data_ptr(), done.data_ptr(), 0, N, 0.99, 0.95, adv.data_ptr(),
                          ret.data_ptr()) == 0


# ------------------------------------------------------------------------------------------------ on-policy
def test_segment_mode_lockstep(env):
    torch, orc, binding = env
    f = fields_for(env_kind=0, n_envs=53, obs_dim=4, n_actions=2, hidden=32, policy_kind=1, seed=606, replay_capacity=0,
                   rollout_len=12, n_segments=3, staleness_bound=1, gamma=0.99, gae_lambda=0.95, max_episode_steps=9)
    ctx, o = make_pair(orc, binding, **f)
    tally = Tally()
    assert ctx.segment_acquire(allow=(0, -7))[0] == -7 == o.segment_acquire()[0]
    v = 0
    consumed = 0
    for seg_i in range(7):
        if seg_i != 3:            # one segment is produced without a fresh version in between
            v += 1
            blob = blob_for(f, v)
            ctx.publish_weights(blob)
            o.publish(blob)
        for p in range(12):
            r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=0, tally=tally)
            assert np.array_equal(r["g_ep"], o.ep_step) or tally.ambiguous_done > 0
        if seg_i in (1, 4, 5, 6):
            if seg_i == 4:        # learner runs ahead: older segments become too stale
                v += 1
                blob = blob_for(f, v)
                ctx.publish_weights(blob)
                o.publish(blob)
            while True:
                gst, gseg = ctx.segment_acquire(allow=(0, -7))
                ost, oseg = o.segment_acquire()
                assert gst == ost
                if gst != 0:
                    break
                consumed += 1
                assert gseg["version"] == oseg["version"]
                assert np.array_equal(gseg["obs"].cpu().numpy(), oseg["obs"])
                sure = np.ones_like(oseg["act"], bool)
                g_act = gseg["act"].cpu().numpy()
                same = g_act == oseg["act"]
                assert same.mean() > 0.999
                assert np.array_equal(gseg["val"].cpu().numpy()[:-1][same], oseg["val"][:-1][same])  # same FMA order
                close(gseg["logp"].cpu().numpy()[same], oseg["logp"][same], RTOL_FP32, "logp")
                assert np.array_equal(gseg["done"].cpu().numpy()[same], oseg["done"][same])
                assert np.array_equal(gseg["rew"].cpu().numpy(), oseg["rew"])
                # the bootstrap row is evaluated on the stepped state, which the two sides hold to FP32 rounding
                close(gseg["val"].cpu().numpy()[-1], oseg["val"][-1], 4 * RTOL_FP32, "bootstrap value")
                adv, ret = ctx.gae(gseg["rew"], gseg["val"], gseg["done"], 0.99, 0.95)
                o_adv, o_ret = orc.gae(oseg["rew"], oseg["val"], oseg["done"], 0.99, 0.95)
                close(adv.cpu().numpy(), o_adv, RTOL_FP32, "segment adv")
                close(ret.cpu().numpy(), o_ret, RTOL_FP32, "segment ret")
    assert consumed >= 3
    gs, os_ = ctx.stats(), o.stats()
    for key in ("produced", "consumed", "dropped_stale", "dropped_overwritten", "starved_calls",
                "max_sampled_staleness", "staleness_hist", "learner_steps"):
        assert gs[key] == os_[key], key
    assert gs["dropped_stale"] > 0
    # the producer laps the consumer: five more segments into three slots overwrite unconsumed ones
    ctx.actor_step(12 * 5)
    o.actor_step(12 * 5)
    while ctx.segment_acquire(allow=(0, -7))[0] == 0:
        assert o.segment_acquire()[0] == 0
    assert o.segment_acquire()[0] == -7
    gs, os_ = ctx.stats(), o.stats()
    for key in ("produced", "consumed", "dropped_stale", "dropped_overwritten", "starved_calls", "learner_steps"):
        assert gs[key] == os_[key], key
    assert gs["dropped_overwritten"] > 0


def test_categorical_actions_follow_the_margin_rule(env):
    torch, orc, binding = env
    f = fields_for(env_kind=1, n_envs=200, obs_dim=6, n_actions=3, hidden=64, policy_kind=1, seed=11, replay_capacity=0,
                   rollout_len=8, n_segments=2, staleness_bound=4, max_episode_steps=50)
    ctx, o = make_pair(orc, binding, **f)
    blob = blob_for(f, 1)
    ctx.publish_weights(blob)
    o.publish(blob)
    tally = Tally()
    margins, o_acts, o_logp = [], [], []
    for t in range(8):
        r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=1, tally=tally)
        margins.append(r["amargin"].copy())
        o_acts.append(r["o_act"].copy())
        o_logp.append(o.last("logp").copy())
    st, gseg = ctx.segment_acquire()
    assert st == 0
    g_act = gseg["act"].cpu().numpy()
    margins, o_acts, o_logp = np.array(margins), np.array(o_acts), np.array(o_logp)
    sure = margins > 8 * RTOL_FP32                 # distance of u*Z to the nearest cumulative boundary, relative to Z
    assert np.array_equal(g_act[sure], o_acts[sure])
    assert (~sure).sum() < 0.01 * sure.size
    same = g_act == o_acts
    close(gseg["logp"].cpu().numpy()[same], o_logp[same], RTOL_FP32, "logp")
    assert len(np.unique(g_act)) == 3


# ------------------------------------------------------------------------------------------------ tensor cores
@pytest.mark.parametrize("D,H,A,N", [(128, 512, 16, 300), (64, 64, 5, 130), (128, 320, 16, 128), (32, 256, 16, 257),
                                     (128, 256, 16, 300), (128, 128, 7, 200), (128, 384, 9, 140)])
def test_bf16_tensor_core_actor_lockstep(env, D, H, A, N):
    """BF16 weights on the tcgen05 path: network outputs within 2e-2 of the oracle (BF16-rounded weights, double
    accumulation), actions exact outside the oracle's top-2 margin, the selection rule exact on the GPU's own
    outputs, env step / ring / reset as in FP32."""
    torch, orc, binding = env
    f = _small(env_kind=2, obs_dim=D, n_actions=A, hidden=H, n_envs=N, replay_capacity=N * 4, warmup=N, weight_dtype=1,
               max_episode_steps=5, lg_done_norm=0.75 * np.sqrt(D), minibatch=200, staleness_bound=10)
    ctx, o = make_pair(orc, binding, **f)
    tally = Tally()
    for t in range(12):
        if t % 5 == 0:
            blob = blob_for(f, t // 5 + 1)
            ctx.publish_weights(blob)
            o.publish(blob)
        r = lockstep_step(ctx, o, torch, rtol=2e-2, env_kind=2, tally=tally, logits_exact=False)
        # outputs are held to 2e-2; the action must equal the oracle's wherever the oracle's top-2 gap exceeds twice the
        # deviation actually measured on this step (then no rounding can change the maximum)
        compare_ring_step(r, o, rtol=RTOL_FP32, env_kind=2, tally=tally, act_exact=False,
                          act_margin_scale=measured_margin(r["g_logits"], r["o_logits"]))
    assert ctx.stats()["device_error"] == 0 and ctx.stats()["episodes_finished"] > 0
    amb_act, _ = tally.report("BF16 tensor-core actor D %d H %d A %d N %d" % (D, H, A, N))
    assert amb_act <= 0.08                                  # a few per cent at most: the rule binds nearly every decision
    # TD error through the same tensor-core forward
    _, batch = ctx.replay_sample()
    out = ctx.td_error(batch)
    rec = np.zeros((200, 2 * D + 4), np.float32)
    rec[:, :D] = batch["obs"].cpu().numpy()
    rec[:, D:2 * D] = batch["next_obs"].cpu().numpy()
    rec.view(np.int32)[:, 2 * D] = batch["act"].cpu().numpy()
    rec[:, 2 * D + 1] = batch["rew"].cpu().numpy()
    rec.view(np.int32)[:, 2 * D + 2] = batch["done"].cpu().numpy()
    st, td, hub, loss, qs, qn = o.td(rec)
    assert st == 0
    g_td = out["td"].cpu().numpy().astype(np.float64)
    q_scale = np.sqrt(np.mean(qs ** 2) + np.mean(qn ** 2))
    assert np.all(np.abs(g_td - td) <= 2e-2 * (np.abs(qs) + np.abs(qn) + 2 * q_scale))
    assert abs(float(out["loss"].item()) - loss) <= 4e-2 * (abs(loss) + q_scale)
    assert ctx.stats()["device_error"] == 0


def test_launch_counter_and_kernel_timing(env):
    torch, orc, binding = env
    f = _small()
    ctx = binding.Context(**f)
    ctx.publish_weights(blob_for(f, 1))
    base = ctx.stats()["kernel_launches"]
    assert base >= 1 and sum(ctx.stats()["kernel_count"]) == 0
    ctx.set_profiling(1)
    ctx.actor_step(3)
    _, batch = ctx.replay_sample()
    ctx.td_error(batch)
    s = ctx.stats()
    # one fused actor launch, eligible list + sample/gather, TD + loss reduction
    assert s["kernel_launches"] - base == 1 + 2 + 2
    assert s["kernel_count"][0] == 1 and s["kernel_count"][3] == 1 and s["kernel_count"][4] == 1
    assert all(s["kernel_ms"][i] > 0 for i in (0, 3, 4))
    ctx.set_profiling(0)
    ctx.actor_step(1)
    assert ctx.stats()["kernel_count"][0] == 1 and ctx.stats()["kernel_launches"] - base == 6
