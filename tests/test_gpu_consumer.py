"""On-policy consumer on the GPU against the oracle: advantage normalisation and shuffled minibatches of segment rows
(run with -m gpu).  Row indices and gathered values are compared bit for bit; normalised values at the FP32 tolerance."""
import numpy as np
import pytest

from parity_util import RTOL_FP32, blob_for, close, fields_for

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


def _seg_ctx(binding, **kw):
    f = fields_for(env_kind=0, n_envs=53, obs_dim=4, n_actions=2, hidden=32, policy_kind=1, seed=606, replay_capacity=0,
                   rollout_len=12, n_segments=2, staleness_bound=3, gamma=0.99, gae_lambda=0.95, max_episode_steps=9, minibatch=128)
    f.update(kw)
    return binding.Context(**f), f


@pytest.mark.parametrize("n", [1, 2, 7, 1000, 4096, (1 << 20) + 3])
def test_normalize_matches_the_oracle(env, n):
    torch, orc, binding = env
    ctx, _ = _seg_ctx(binding)
    rng = np.random.default_rng(n)
    x = (3.0 + 2.0 * rng.standard_normal(n)).astype(np.float32)
    g = ctx.normalize(torch.from_numpy(x).cuda(), 1e-8).cpu().numpy()
    o = orc.normalize(x, 1e-8)
    if n == 1:
        assert g[0] == 0.0 and o[0] == 0.0
        return
    close(g, o, RTOL_FP32, "normalised values")
    # in place, and reproducible bit for bit
    t = torch.from_numpy(x).cuda()
    ctx.normalize(t, 1e-8, out=t)
    assert np.array_equal(t.cpu().numpy().view(np.uint32), g.view(np.uint32))
    assert binding.tj_normalize(ctx.h, t.data_ptr(), 0, 1e-8, t.data_ptr()) == 0           # empty input: nothing to do
    assert binding.tj_normalize(ctx.h, 0, 5, 1e-8, t.data_ptr()) == binding.TJ_ERR_INVALID_ARG


def test_normalize_constant_input_gives_zeros(env):
    torch, orc, binding = env
    ctx, _ = _seg_ctx(binding)
    g = ctx.normalize(torch.full((777,), 2.5, device="cuda"), 1e-8)
    assert torch.count_nonzero(g).item() == 0


def test_shuffled_minibatches_match_the_oracle_and_cover_every_row_once(env):
    torch, orc, binding = env
    ctx, f = _seg_ctx(binding)
    ctx.publish_weights(blob_for(f, 1))
    ctx.actor_step(12)
    st, seg = ctx.segment_acquire()
    assert st == 0
    T, N, D = seg["T"], seg["N"], 4
    R = T * N
    adv, ret = ctx.gae(seg["rew"], seg["val"], seg["done"], 0.99, 0.95)
    adv_n = ctx.normalize(adv)
    s_obs = seg["obs"].reshape(R, D).cpu().numpy()
    s_act, s_logp = seg["act"].reshape(R).cpu().numpy(), seg["logp"].reshape(R).cpu().numpy()
    a_np, r_np = adv_n.reshape(R).cpu().numpy(), ret.reshape(R).cpu().numpy()
    for shuffle_id in (0, 1, 2**33 + 5):
        seen = []
        mb_size = 100                                    # 636 rows: six full minibatches and a ragged one of 36
        for first in range(0, R, mb_size):
            n = min(mb_size, R - first)
            mb = ctx.alloc_minibatch(n)
            ctx.segment_minibatch(seg, adv_n, ret, shuffle_id, first, mb)
            rows = mb["row"].cpu().numpy()
            want = np.array([orc.shuffle_index(f["seed"], shuffle_id, R, first + j) for j in range(n)])
            assert np.array_equal(rows, want)                                  # the keyed order, bit for bit
            assert np.array_equal(mb["obs"].cpu().numpy(), s_obs[rows])          # gathers are copies
            assert np.array_equal(mb["act"].cpu().numpy(), s_act[rows])
            assert np.array_equal(mb["logp_old"].cpu().numpy(), s_logp[rows])
            assert np.array_equal(mb["adv"].cpu().numpy(), a_np[rows])
            assert np.array_equal(mb["ret"].cpu().numpy(), r_np[rows])
            seen.append(rows)
        assert sorted(np.concatenate(seen).tolist()) == list(range(R))          # every row exactly once per shuffle
    # positions outside the segment are refused on the host
    mb = ctx.alloc_minibatch(10)
    assert binding.tj_segment_minibatch(ctx.h, seg["c"], adv_n.data_ptr(), ret.data_ptr(), 0, R - 5, mb["c"]) == binding.TJ_ERR_INVALID_ARG
    assert binding.tj_segment_minibatch(ctx.h, seg["c"], adv_n.data_ptr(), ret.data_ptr(), 0, -1, mb["c"]) == binding.TJ_ERR_INVALID_ARG
    # a minibatch feeds the PPO update as it lies
    theta = torch.from_numpy(blob_for(f, 1)).cuda()
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    mb = ctx.alloc_minibatch(128)
    ctx.segment_minibatch(seg, adv_n, ret, 7, 0, mb)
    stats = ctx.ppo_step(mb["obs"], mb["act"], mb["logp_old"], mb["adv"], mb["ret"], 1e-3, theta, m, v, 1)
    assert torch.isfinite(stats).all()


def test_full_size_segment_shuffle(env):
    """The on-policy workload's segment (128 x 65,536 rows): a whole shuffle covers every row once; sampled positions match
    the oracle; normalised advantages have mean 0 and variance 1."""
    torch, orc, binding = env
    f = fields_for("cfg4")
    ctx = binding.Context(**f)
    ctx.publish_weights(blob_for(f, 1))
    ctx.actor_step(f["rollout_len"])
    st, seg = ctx.segment_acquire()
    assert st == 0
    R = seg["T"] * seg["N"]
    adv, ret = ctx.gae(seg["rew"], seg["val"], seg["done"], f["gamma"], f["gae_lambda"])
    adv_n = ctx.normalize(adv)
    a64 = adv_n.double()
    assert abs(a64.mean().item()) < 1e-5 and abs(a64.var(unbiased=False).item() - 1.0) < 1e-4
    mb_size = 1 << 20
    hit = torch.zeros(R, dtype=torch.int32, device="cuda")
    mb = ctx.alloc_minibatch(mb_size)
    rng = np.random.default_rng(1)
    for first in range(0, R, mb_size):
        ctx.segment_minibatch(seg, adv_n, ret, 3, first, mb)
        hit.index_add_(0, mb["row"].long(), torch.ones(mb_size, dtype=torch.int32, device="cuda"))
        rows = mb["row"].cpu().numpy()
        for j in rng.integers(0, mb_size, 6):
            assert rows[j] == orc.shuffle_index(f["seed"], 3, R, first + int(j))
    assert int(hit.min().item()) == 1 and int(hit.max().item()) == 1
    assert ctx.stats()["device_error"] == 0
