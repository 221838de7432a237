"""The FP32-accuracy tensor-core actor (weight mode TJ_W_FP32_TC) against the FP32 oracle, through the C ABI.

The hidden x hidden layer runs as three FP16 products of split operands (about 2^-22 per term), so network outputs are
held to the FP32 tolerance of 1e-5 (|g-o| <= rtol*|o| + rtol*rms(o)) rather than bit for bit.  Actions must be the
oracle's wherever the oracle's decision margin exceeds twice the deviation measured on that step, and must always be
what the oracle's selection rule gives on the GPU's own outputs; the shares inside the margins are reported.  Everything
downstream of an equal action (rewards, done flags, next states, reset draws, ring slots, version tags, counters) is
compared as in the FP32 tests.  The oracle itself always runs with FP32 weights.
"""
import numpy as np
import pytest

from parity_util import RTOL_FP32, Tally, blob_for, close, compare_ring_step, fields_for, lockstep_step, measured_margin

pytestmark = pytest.mark.gpu

W_FP32, W_FP32_TC = 0, 2


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


def _pair(orc, binding, **fields):
    ctx = binding.Context(**dict(fields, weight_dtype=W_FP32_TC))
    o = orc.Oracle(**dict(fields, weight_dtype=W_FP32))
    return ctx, o


def _ring_fields(kind, D, A, H, N, **kw):
    base = dict(env_kind=kind, n_envs=N, obs_dim=D, n_actions=A, hidden=H, epsilon=0.2, seed=777, replay_capacity=N * 5,
                minibatch=19, staleness_bound=2, warmup=N, target_sync_interval=3, gamma=0.99, huber_delta=1.0,
                max_episode_steps=23)
    base.update(kw)
    return fields_for(**base)


@pytest.mark.parametrize("kind,D,A,H,N,steps", [(0, 4, 2, 64, 37, 60), (1, 6, 3, 128, 300, 40), (0, 4, 2, 192, 129, 30),
                                                (1, 6, 3, 256, 1, 30), (1, 6, 3, 256, 700, 30), (0, 4, 2, 256, 128, 30)])
def test_ring_mode_lockstep(env, kind, D, A, H, N, steps):
    torch, orc, binding = env
    f = _ring_fields(kind, D, A, H, N)
    ctx, o = _pair(orc, binding, **f)
    tally = Tally()
    for t in range(steps):
        if t % 11 == 0:
            blob = blob_for(f, t // 11 + 1)
            ctx.publish_weights(blob)
            o.publish(blob)
        r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=kind, tally=tally, logits_exact=False)
        compare_ring_step(r, o, rtol=RTOL_FP32, env_kind=kind, tally=tally, act_exact=False,
                          act_margin_scale=measured_margin(r["g_logits"], r["o_logits"]))
    amb_act, amb_done = tally.report("split tensor-core actor kind %d H %d N %d" % (kind, H, N))
    assert tally.max_logit_dev <= 2 * RTOL_FP32       # the tolerance is rtol * (|o| + rms(o)); |o| = rms at this bound
    assert amb_act <= 0.002 + 2.0 / tally.total and amb_done <= 0.002 + 2.0 / tally.total
    st = ctx.stats()
    assert st["device_error"] == 0 and st["episodes_finished"] > 0
    assert st["produced"] == o.stats()["produced"]


def test_multi_step_launch_equals_single_steps_and_blocks_take_several_tiles(env):
    """One launch of n steps equals n launches of one step bit for bit (the chunk stream of the hidden x hidden matrix runs
    on across steps and tiles inside a launch); 20,000 envs give most blocks two tiles."""
    torch, orc, binding = env
    for kind, D, A, N in ((0, 4, 2, 77), (1, 6, 3, 20000)):
        f = _ring_fields(kind, D, A, 128, N, replay_capacity=N * 8, max_episode_steps=5)
        a = binding.Context(**dict(f, weight_dtype=W_FP32_TC))
        b_ = binding.Context(**dict(f, weight_dtype=W_FP32_TC))
        blob = blob_for(f, 1)
        a.publish_weights(blob)
        b_.publish_weights(blob)
        a.actor_step(7)
        for _ in range(7):
            b_.actor_step(1)
        sa, sb = a.get_state(), b_.get_state()
        assert torch.equal(sa["state"], sb["state"]) and torch.equal(sa["ep_step"], sb["ep_step"])
        assert sa["cursor"] == sb["cursor"] == N * 7
        rows = N * 7                                  # the rows written so far; the rest of the ring is not initialised
        assert torch.equal(a.ring_view()[0][:rows].view(torch.int32), b_.ring_view()[0][:rows].view(torch.int32))
        assert torch.equal(a.ring_view()[1][:7], b_.ring_view()[1][:7])
        assert a.stats()["episodes_finished"] == b_.stats()["episodes_finished"] > 0
        assert a.stats()["device_error"] == 0


def test_many_envs_against_the_fp32_kernel(env):
    """20,000 envs (several tiles per block, a ragged last tile): outputs within tolerance of the FP32 FMA kernel's, which the
    other tests hold to the oracle bit for bit, and equal actions wherever that kernel's top-2 gap exceeds the deviation."""
    torch, orc, binding = env
    N = 20000 + 37
    f = _ring_fields(1, 6, 3, 256, N, replay_capacity=N * 2)
    a = binding.Context(**dict(f, weight_dtype=W_FP32_TC))
    b_ = binding.Context(**dict(f, weight_dtype=W_FP32))
    blob = blob_for(f, 1)
    a.publish_weights(blob)
    b_.publish_weights(blob)
    da = torch.empty((N, 3), dtype=torch.float32, device=a.device)
    db = torch.empty_like(da)
    a.actor_step(1, da)
    b_.actor_step(1, db)
    ga, gb = da.cpu().numpy(), db.cpu().numpy()
    close(ga, gb, RTOL_FP32, "outputs of the two kernels")
    top2 = np.sort(gb, axis=1)
    sure = (top2[:, -1] - top2[:, -2]) > measured_margin(ga, gb)
    ra, rb = a.ring_view()[0][:N].cpu().numpy().view(np.int32), b_.ring_view()[0][:N].cpu().numpy().view(np.int32)
    assert sure.mean() > 0.99
    assert np.array_equal(ra[sure][:, 12], rb[sure][:, 12])          # the action word of an Acrobot record
    assert np.array_equal(ra[sure][:, 15], rb[sure][:, 15])          # version tag


def test_segment_mode_with_value_head(env):
    torch, orc, binding = env
    T = 6
    f = fields_for(env_kind=0, n_envs=150, obs_dim=4, n_actions=2, hidden=256, policy_kind=1, seed=31, replay_capacity=0,
                   rollout_len=T, n_segments=2, staleness_bound=4, gamma=0.99, gae_lambda=0.95, max_episode_steps=9)
    ctx, o = _pair(orc, binding, **f)
    blob = blob_for(f, 1)
    ctx.publish_weights(blob)
    o.publish(blob)
    tally = Tally()
    margins, o_acts, o_logp, o_val = [], [], [], []
    for t in range(T):
        r = lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=0, tally=tally, logits_exact=False)
        margins.append(r["amargin"].copy())
        o_acts.append(r["o_act"].copy())
        o_logp.append(o.last("logp").copy())
        o_val.append(r["o_logits"][:, -1].copy() if r["o_logits"].shape[1] > 2 else None)
    st, gseg = ctx.segment_acquire()
    ost, oseg = o.segment_acquire()
    assert st == 0 == ost
    g_act = gseg["act"].cpu().numpy()
    margins, o_acts, o_logp = np.array(margins), np.array(o_acts), np.array(o_logp)
    sure = margins > 8 * RTOL_FP32                  # distance of u*Z to the nearest cumulative boundary, relative to Z
    assert np.array_equal(g_act[sure], o_acts[sure])
    assert (~sure).sum() <= 0.01 * sure.size
    same = g_act == o_acts
    close(gseg["logp"].cpu().numpy()[same], o_logp[same], RTOL_FP32, "logp")
    # values: each row of the oracle's segment was computed from the GPU's state of that step (lock-step), bootstrap included
    close(gseg["val"].cpu().numpy()[:-1], oseg["val"][:-1], RTOL_FP32, "values")
    last_same = same[-1]
    close(gseg["val"].cpu().numpy()[-1][last_same], oseg["val"][-1][last_same], 4 * RTOL_FP32, "bootstrap value")
    assert np.array_equal(gseg["obs"].cpu().numpy(), oseg["obs"])
    assert np.array_equal(gseg["rew"].cpu().numpy(), oseg["rew"])
    assert ctx.stats()["device_error"] == 0


def test_unsupported_shapes_are_refused(env):
    torch, orc, binding = env
    for kw in (dict(hidden=24), dict(hidden=512), dict(env_kind=2, obs_dim=16, n_actions=5, hidden=64)):
        f = _ring_fields(0, 4, 2, 64, 32)
        f.update(kw)
        f = fields_for(**f)
        with pytest.raises(Exception) as ei:
            binding.Context(**dict(f, weight_dtype=W_FP32_TC))
        assert "TJ_W_FP32_TC" in str(ei.value)


@pytest.mark.parametrize("kind,D,A,H,B", [(0, 4, 2, 64, 256), (1, 6, 3, 256, 77), (1, 6, 3, 128, 300), (0, 4, 2, 256, 1)])
def test_td_error_in_this_weight_mode_follows_the_lagging_target(env, kind, D, A, H, B):
    """tj_td_error of a context in this weight mode runs both forwards with the split-operand hidden layer; the oracle's FP32
    TD error is the reference at the FP32 tolerance (relative to the terms the error is a difference of).  The target network
    lags one version at versions 2 and 4: there the GPU's errors must follow the lagging target, not the newest parameters."""
    torch, orc, binding = env
    f = _ring_fields(kind, D, A, H, 32, replay_capacity=32 * 16, minibatch=B, warmup=32, staleness_bound=50,
                     target_sync_interval=2, max_episode_steps=11)
    ctx, o = _pair(orc, binding, **f)
    fresh = orc.Oracle(**dict(f, target_sync_interval=1, weight_dtype=W_FP32))
    tally = Tally()
    for v in range(1, 6):
        blob = blob_for(f, v)
        ctx.publish_weights(blob)
        o.publish(blob)
        fresh.publish(blob)
        for _ in range(4):
            lockstep_step(ctx, o, torch, rtol=RTOL_FP32, env_kind=kind, tally=tally, logits_exact=False)
        _, batch = ctx.replay_sample()
        o.sample()
        fresh.set_counters(0, 0, v)
        out = ctx.td_error(batch)
        rec = np.zeros((B, 2 * D + 4), np.float32)
        rec[:, :D] = batch["obs"].cpu().numpy()
        rec[:, D:2 * D] = batch["next_obs"].cpu().numpy()
        rec.view(np.int32)[:, 2 * D] = batch["act"].cpu().numpy()
        rec[:, 2 * D + 1] = batch["rew"].cpu().numpy()
        rec.view(np.int32)[:, 2 * D + 2] = batch["done"].cpu().numpy()
        st, td, hub, loss, qs, qn = o.td(rec)
        assert st == 0
        rms = float(np.sqrt(np.mean(qs ** 2) + np.mean(qn ** 2)))
        terms = np.abs(qs) + np.abs(qn) + np.abs(rec[:, 2 * D + 1]) + rms
        g_td = out["td"].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g_td - td) <= RTOL_FP32 * (np.abs(td) + terms)), float(np.max(np.abs(g_td - td) / (np.abs(td) + terms)))
        g_h = out["huber"].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g_h - hub) <= 2 * RTOL_FP32 * (hub + terms * np.maximum(1.0, np.abs(td))))
        assert abs(float(out["loss"].item()) - loss) <= 2 * RTOL_FP32 * (abs(loss) + float(terms.mean()))
        if v in (2, 4) and B > 1:
            _, td_fresh, _, _, _, _ = fresh.td(rec)
            moved = np.abs(td_fresh - td) > 100 * RTOL_FP32 * (np.abs(td) + terms)
            live = rec.view(np.int32)[:, 2 * D + 2] == 0
            assert moved[live].mean() > 0.9
            assert np.all(np.abs(g_td - td_fresh)[moved] > RTOL_FP32 * (np.abs(td) + terms)[moved])
    assert ctx.stats()["device_error"] == 0


def test_activation_beyond_the_split_range_is_reported(env):
    """The hidden activations are split after a scaling by 16, so they must stay below 4,094; parameters that push them
    beyond that must not pass silently: the kernel latches device_error 5 (no fault, the context stays usable)."""
    torch, orc, binding = env
    f = _ring_fields(0, 4, 2, 64, 64)
    ctx = binding.Context(**dict(f, weight_dtype=W_FP32_TC))
    blob = blob_for(f, 1)
    ctx.publish_weights(blob)
    ctx.actor_step(2)
    assert ctx.stats()["device_error"] == 0
    big = blob.copy()
    big[:64 * 4] *= 1e6                      # first-layer weights: activations of the order of 1e4 and more
    ctx.publish_weights(big)
    ctx.actor_step(1)
    assert ctx.stats()["device_error"] == 5
