"""Actor and learner on two CUDA streams (run with -m gpu): the results must be those of the one-stream run with the same
host call order, bit for bit, and the bounded host-side wait must report a stalled stream without touching the GPU."""
import numpy as np
import pytest

from parity_util import blob_for, fields_for

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2502_20190_b200 import binding, build
    build.build()
    return torch, binding


def _run_replay(torch, binding, f, two_stream, iters=24):
    """Software-pipelined DQN iterations: the learner consumes what was produced before, the actor produces the next block
    with the parameters of the previous iteration, then one new version."""
    ctx = binding.Context(**f)
    theta = torch.from_numpy(blob_for(f, 1)).cuda()
    target = theta.clone()
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    batch = ctx.alloc_batch()
    out = dict(td=torch.empty(f["minibatch"], device="cuda"), huber=torch.empty(f["minibatch"], device="cuda"),
               loss=torch.empty(1, device="cuda"))
    ctx.publish_weights(theta)
    if two_stream:
        ctx.use_learner_stream(True)
    ctx.actor_step(3)
    idx_log, td_log = [], []
    for it in range(iters):
        st, _ = ctx.replay_sample(batch=batch, allow=(0, -6, -7))
        if st == 0:
            ctx.td_error(batch, out)
            ctx.adam_step(batch, 1e-3, theta, target, m, v, it + 1)
        ctx.actor_step(3)
        ctx.publish_weights(theta)
        if st == 0:
            assert ctx.wait(1, 20000) == 0          # results of the learner stream, before the host reads them
            idx_log.append(batch["idx"].cpu().numpy().copy())
            td_log.append(out["td"].cpu().numpy().copy())
    s = ctx.stats()
    ring, bv = ctx.ring_view()
    return dict(ring=ring.view(torch.int32).cpu().numpy().copy(), bv=bv.cpu().numpy().copy(), theta=theta.cpu().numpy().copy(),
                state=ctx.get_state()["state"].cpu().numpy().copy(), idx=idx_log, td=td_log, stats=s)


@pytest.mark.parametrize("kind,D,A,H,N,wd", [(0, 4, 2, 128, 4096, 0), (1, 6, 3, 256, 2000, 0), (2, 128, 16, 512, 1000, 1)])
def test_two_streams_give_the_one_stream_results_bit_for_bit(env, kind, D, A, H, N, wd):
    torch, binding = env
    f = fields_for(env_kind=kind, n_envs=N, obs_dim=D, n_actions=A, hidden=H, epsilon=0.1, seed=515, weight_dtype=wd,
                   replay_capacity=N * 16, minibatch=512, staleness_bound=4, warmup=N, target_sync_interval=5, gamma=0.99,
                   huber_delta=1.0, max_episode_steps=30, lg_done_norm=9.0)
    one = _run_replay(torch, binding, f, False)
    two = _run_replay(torch, binding, f, True)
    assert len(one["idx"]) == len(two["idx"]) > 10
    for a, b in zip(one["idx"], two["idx"]):
        assert np.array_equal(a, b)
    for a, b in zip(one["td"], two["td"]):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    assert np.array_equal(one["ring"], two["ring"]) and np.array_equal(one["bv"], two["bv"])
    assert np.array_equal(one["theta"].view(np.uint32), two["theta"].view(np.uint32))
    assert np.array_equal(one["state"].view(np.uint32), two["state"].view(np.uint32))
    for key in ("produced", "consumed", "dropped_stale", "starved_calls", "actor_steps", "learner_steps", "max_sampled_staleness",
                "episodes_finished", "staleness_hist", "actor_version", "kernel_launches", "device_error"):
        assert one["stats"][key] == two["stats"][key], key
    assert one["stats"]["device_error"] == 0


def test_two_streams_in_segment_mode(env):
    torch, binding = env
    f = fields_for(env_kind=0, n_envs=512, obs_dim=4, n_actions=2, hidden=64, policy_kind=1, seed=99, replay_capacity=0,
                   rollout_len=16, n_segments=3, staleness_bound=2, gamma=0.99, gae_lambda=0.95, minibatch=2048)

    def run(two):
        ctx = binding.Context(**f)
        theta = torch.from_numpy(blob_for(f, 1)).cuda()
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        ctx.publish_weights(theta)
        if two:
            ctx.use_learner_stream(True)
        ctx.actor_step(16)
        mb = ctx.alloc_minibatch(2048)
        t = 0
        for it in range(6):
            st, seg = ctx.segment_acquire(allow=(0, -7))
            ctx.actor_step(16)                     # the next segment is produced while this one is consumed
            if st == 0:
                adv, ret = ctx.gae(seg["rew"], seg["val"], seg["done"], 0.99, 0.95)
                ctx.normalize(adv, 1e-8, out=adv)
                for first in range(0, 16 * 512, 2048):
                    ctx.segment_minibatch(seg, adv, ret, it, first, mb)
                    t += 1
                    ctx.ppo_step(mb["obs"], mb["act"], mb["logp_old"], mb["adv"], mb["ret"], 1e-3, theta, m, v, t)
                assert ctx.segment_check(seg) == 0
            ctx.publish_weights(theta)
        s = ctx.stats()
        return theta.cpu().numpy().copy(), ctx.get_state()["state"].cpu().numpy().copy(), s

    th1, st1, s1 = run(False)
    th2, st2, s2 = run(True)
    assert np.array_equal(th1.view(np.uint32), th2.view(np.uint32)) and np.array_equal(st1.view(np.uint32), st2.view(np.uint32))
    for key in ("produced", "consumed", "dropped_stale", "dropped_overwritten", "starved_calls", "learner_steps", "episodes_finished"):
        assert s1[key] == s2[key], key
    assert s1["consumed"] > 0


def test_bounded_wait_reports_a_stalled_learner_stream(env):
    """A stream that is busy for about a second (a bounded sleep, not a fault): the 20 ms wait gives up with TJ_ERR_TIMEOUT,
    the idle actor stream answers at once, a longer wait succeeds, and the context keeps working."""
    torch, binding = env
    f = fields_for(env_kind=0, n_envs=256, obs_dim=4, n_actions=2, hidden=32, epsilon=0.1, seed=3, replay_capacity=256 * 8,
                   minibatch=128, staleness_bound=4, warmup=128, target_sync_interval=10, gamma=0.99, huber_delta=1.0)
    ctx = binding.Context(**f)
    ctx.publish_weights(blob_for(f, 1))
    ctx.use_learner_stream(True)
    ctx.actor_step(2)
    assert ctx.wait(0, 5000) == 0 and ctx.wait(1, 5000) == 0
    with torch.cuda.stream(ctx.learner_stream):
        torch.cuda._sleep(int(2.0e9))              # about a second of a sleeping kernel on the learner stream
    assert ctx.wait(1, 20) == binding.TJ_ERR_TIMEOUT
    assert "learner stream" in binding.tj_last_error(ctx.h)
    assert ctx.wait(0, 1000) == 0                  # the actor stream is not held up by it
    ctx.actor_step(1)
    assert ctx.wait(1, 20000) == 0
    st, batch = ctx.replay_sample(allow=(0,))
    assert st == 0 and ctx.stats()["device_error"] == 0
    assert binding.tj_wait(ctx.h, 2, 10) == binding.TJ_ERR_INVALID_ARG
