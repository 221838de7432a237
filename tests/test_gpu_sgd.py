"""GPU parity for the learner update (tj_sgd_step) against the oracle's orc_sgd_step.

The two sides get the same parameter blobs and the same minibatch (sampled by the GPU context from its own ring, whose
contents are parity-checked elsewhere).  Compared: the parameter *change* per group and the loss.  Tolerance: the GPU
accumulates each gradient entry over the n rows in FP32 (n sequential fused multiply-adds, error <= n * 2^-24 of the sum of
term magnitudes in the worst case, ~sqrt(n) * 2^-24 typically), the oracle in double; 1e-5 relative to each entry plus
1e-5 of the group's rms covers n up to a few thousand with the inputs used here, and is the FP32 tolerance of every other
test."""
import numpy as np
import pytest

from parity_util import REPORT, RTOL_FP32, blob_for, close, fields_for

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


def _groups(D, H, A):
    n1, n2, n3 = H * D, H * H, A * H
    names = ["W1", "b1", "W2", "b2", "W3", "b3"]
    sizes = [n1, H, n2, H, n3, A]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    return [(names[i], int(offs[i]), int(offs[i + 1])) for i in range(6)]


# the last four run the tiled matrix-product kernels (hidden >= 128 and >= 512 rows): hidden and row counts that are not
# multiples of the 64 x 128 tile, an obs_dim that rules out 16-byte loads, an action count above one k-step's quarter
@pytest.mark.parametrize("kind,D,A,H,N,B", [(0, 4, 2, 64, 64, 256), (1, 6, 3, 96, 50, 333), (2, 16, 5, 200, 40, 77), (2, 48, 4, 32, 40, 100),
                                            (0, 4, 2, 256, 128, 1024), (2, 16, 5, 200, 64, 600), (1, 6, 3, 136, 64, 700),
                                            (2, 20, 9, 130, 64, 513)])
def test_sgd_step_matches_oracle(env, kind, D, A, H, N, B):
    _check_sgd_step(env, kind, D, A, H, N, B, 0)


@pytest.mark.parametrize("kind,D,A,H,N,B", [(2, 32, 4, 64, 128, 300), (2, 128, 7, 128, 256, 500)])
def test_sgd_step_in_a_bf16_context_updates_the_fp32_master_copy(env, kind, D, A, H, N, B):
    """A BF16 context (the second shape runs the pipelined tensor-core actor) rounds the parameters at publish only: the
    update itself is the FP32 one, on the caller's FP32 blob, and matches the same oracle step."""
    _check_sgd_step(env, kind, D, A, H, N, B, 1)


RTOL_TF32X3 = 1e-4


def test_sgd_step_on_the_tensor_core_path_matches_oracle(env):
    """25 x 4 tiles of 128 x 128 (3,100 rows, hidden 500: ragged both ways) are enough for the hidden layers and dh1 to run
    as 3 x TF32 tensor-core products.  Their tolerance: an operand enters as a TF32 high part plus a remainder that the
    tensor core again reads with 11 significant bits, so each product carries up to 2 * 2^-22 from the two truncated
    remainders plus 2^-22 from the dropped low x low term, 3 * 2^-22 = 7e-7 against FP32's 2^-24 = 6e-8 per operation:
    twelve times the FP32 tolerance, rounded down to 1e-4."""
    _check_sgd_step(env, 2, 16, 5, 500, 512, 3100, 0, rtol=RTOL_TF32X3)


@pytest.mark.parametrize("D", [32, 128])
def test_sgd_step_on_the_presplit_tensor_core_path_matches_oracle(env, D):
    """Hidden 512 (two 256-column tiles) and 3,100 rows (25 row tiles, the last one ragged; row ranges of the weight
    gradients that end inside a chunk): both hidden layers of both networks and dh1 run as 128 x 256 tensor-core tiles
    whose weight operand was split once per update, and the weight gradients of W2 (256-column tiles) and, with 128
    inputs, of W1 (128-column tiles) as tensor-core products over the minibatch rows.  Same three products per tile as
    the path above, same tolerance."""
    _check_sgd_step(env, 2, D, 5, 512, 512, 3100, 0, rtol=RTOL_TF32X3)


def _relu_gate_allowance(theta, D, H, A, obs, act, lr, kappa, margin=2e-6):
    """The ReLU derivative is a step: where a pre-activation lies within the forward tolerance of zero the two sides may
    take different branches, and the whole contribution of that (row, unit) to the gradient appears or vanishes.  This
    returns, per parameter, an upper bound of what those gates can move (|dL/dq| <= kappa / rows at the selected action),
    and their number.  A layer-2 gate (r, n) reaches b2[n], W2[n, :] and, through dh1[r, :], b1 and W1; a layer-1 gate
    (r, j) reaches b1[j] and W1[j, :].  The forward pass here is a float64 matmul used only to find those gates."""
    th = theta.astype(np.float64)
    o = 0
    W1 = th[o:o + H * D].reshape(H, D); o += H * D
    b1 = th[o:o + H]; o += H
    W2 = th[o:o + H * H].reshape(H, H); o += H * H
    b2 = th[o:o + H]; o += H
    W3 = th[o:o + A * H].reshape(A, H)
    x = obs.astype(np.float64)
    rows = x.shape[0]
    pre1 = x @ W1.T + b1
    h1 = np.maximum(pre1, 0.0)
    pre2 = h1 @ W2.T + b2
    allow = np.zeros(th.size)
    aW1 = allow[0:H * D].reshape(H, D)
    ab1 = allow[H * D:H * D + H]
    aW2 = allow[H * D + H:H * D + H + H * H].reshape(H, H)
    ab2 = allow[H * D + H + H * H:H * D + 2 * H + H * H]
    g = lr * kappa / rows
    amb2 = np.argwhere(np.abs(pre2) <= margin * np.sqrt(np.mean(pre2 ** 2)))
    amb1 = np.argwhere(np.abs(pre1) <= margin * np.sqrt(np.mean(pre1 ** 2)))
    for r, n in amb2:
        t = g * abs(W3[act[r], n])
        ab2[n] += t
        aW2[n, :] += t * np.abs(h1[r])
        c = t * np.abs(W2[n, :])
        ab1 += c
        aW1 += np.outer(c, np.abs(x[r]))
    reach = np.abs(W3) @ np.abs(W2)                 # [A][H]: the most dh1[r][j] can be per unit of |dL/dq|
    for r, j in amb1:
        t = g * reach[act[r], j]
        ab1[j] += t
        aW1[j, :] += t * np.abs(x[r])
    return allow, len(amb1) + len(amb2)


def _check_sgd_step(env, kind, D, A, H, N, B, weight_dtype, rtol=RTOL_FP32):
    torch, orc, binding = env
    f = fields_for(env_kind=kind, n_envs=N, obs_dim=D, n_actions=A, hidden=H, epsilon=0.3, seed=777, replay_capacity=N * 16,
                   minibatch=B, staleness_bound=20, warmup=N, target_sync_interval=1000, gamma=0.99, huber_delta=1.0,
                   max_episode_steps=9, weight_dtype=weight_dtype)
    ctx = binding.Context(**f)
    theta_t = blob_for(f, 1)            # the first publish also becomes the target
    theta = blob_for(f, 2)
    ctx.publish_weights(theta_t)
    ctx.actor_step(6)
    ctx.publish_weights(theta)
    ctx.actor_step(6)
    _, batch = ctx.replay_sample()
    dev = ctx.device
    th = torch.from_numpy(theta.copy()).to(dev)
    tt = torch.from_numpy(theta_t.copy()).to(dev)
    lr = 0.05
    loss = ctx.sgd_step(batch, lr, th, tt)
    torch.cuda.synchronize()
    g_new = th.cpu().numpy()
    o_new, o_loss = orc.sgd_step(theta, theta_t, D, H, A, batch["obs"].cpu().numpy(), batch["act"].cpu().numpy(),
                                 batch["rew"].cpu().numpy(), batch["next_obs"].cpu().numpy(), batch["done"].cpu().numpy(),
                                 0.99, 1.0, lr)
    assert np.array_equal(tt.cpu().numpy(), theta_t)                        # the target blob is read only
    assert abs(float(loss.item()) - o_loss) <= 2 * RTOL_FP32 * (abs(o_loss) + 1e-3)
    dg = g_new.astype(np.float64) - theta.astype(np.float64)
    do = o_new.astype(np.float64) - theta.astype(np.float64)
    # the FP32 rounding of theta_new itself (half an ulp on each side) is part of the comparison floor; the stored value is
    # rounded at its own magnitude, which a large step can carry well above theta's
    ulp = 2 * np.spacing(np.maximum(np.abs(theta), np.abs(o_new)).astype(np.float32)).astype(np.float64)
    allow, n_gates = _relu_gate_allowance(theta, D, H, A, batch["obs"].cpu().numpy(), batch["act"].cpu().numpy(), lr, 1.0)
    REPORT.append("sgd step D %d H %d rows %d: %d of %d ReLU gates within the forward tolerance of zero" % (D, H, B, n_gates, 2 * B * H))
    for name, a, b in _groups(D, H, A):
        assert np.abs(do[a:b]).max() > 0, name                               # every group moves
        rms = np.sqrt(np.mean(do[a:b] ** 2))
        err = np.abs(dg[a:b] - do[a:b])
        bound = rtol * np.abs(do[a:b]) + rtol * rms + ulp[a:b] + allow[a:b]
        assert np.all(err <= bound), "%s: worst %.3e over bound %.3e" % (name, err.max(), bound[np.argmax(err - bound)])
        # a layer-2 gate reaches one row of W2 and one entry of b2 only: there the allowance may not carry the comparison
        if name in ("W2", "b2"):
            assert np.mean(allow[a:b] > rtol * rms) <= 0.05, name
    # a second step from the updated parameters stays on the oracle's trajectory
    loss2 = ctx.sgd_step(batch, lr, th, tt)
    o_new2, o_loss2 = orc.sgd_step(o_new, theta_t, D, H, A, batch["obs"].cpu().numpy(), batch["act"].cpu().numpy(),
                                   batch["rew"].cpu().numpy(), batch["next_obs"].cpu().numpy(), batch["done"].cpu().numpy(),
                                   0.99, 1.0, lr)
    assert abs(float(loss2.item()) - o_loss2) <= 1e-4 * (abs(o_loss2) + 1e-3)
    close(th.cpu().numpy(), o_new2, 1e-4, "theta after two steps")
    assert ctx.stats()["device_error"] == 0


def test_sgd_step_argument_checks(env):
    torch, orc, binding = env
    f = fields_for(env_kind=0, n_envs=32, obs_dim=4, n_actions=2, hidden=32, epsilon=0.1, seed=5, replay_capacity=32 * 8,
                   minibatch=64, staleness_bound=8, warmup=32, target_sync_interval=10, gamma=0.99, huber_delta=1.0)
    ctx = binding.Context(**f)
    blob = blob_for(f, 1)
    ctx.publish_weights(blob)
    ctx.actor_step(4)
    _, batch = ctx.replay_sample()
    th = torch.from_numpy(blob.copy()).to(ctx.device)
    st = binding.tj_sgd_step(ctx.h, batch["c"], 0.1, th.data_ptr(), th.data_ptr(), 0)
    assert st == binding.TJ_ERR_INVALID_ARG                                  # theta and target must differ
    big = ctx.alloc_batch(65)
    tt = th.clone()
    st = binding.tj_sgd_step(ctx.h, big["c"], 0.1, th.data_ptr(), tt.data_ptr(), 0)
    assert st == binding.TJ_ERR_INVALID_ARG and "minibatch" in binding.tj_last_error(ctx.h)
    # lr = 0 leaves the parameters untouched
    before = th.clone()
    ctx.sgd_step(batch, 0.0, th, tt)
    assert torch.equal(before, th)
    # a segment-mode context (categorical policy) has no Q-learning update
    f2 = fields_for(env_kind=0, n_envs=32, obs_dim=4, n_actions=2, hidden=32, policy_kind=1, seed=5, replay_capacity=0,
                    rollout_len=4, n_segments=2, staleness_bound=1, minibatch=64)
    c2 = binding.Context(**f2)
    st = binding.tj_sgd_step(c2.h, batch["c"], 0.1, th.data_ptr(), tt.data_ptr(), 0)
    assert st == binding.TJ_ERR_UNSUPPORTED


@pytest.mark.parametrize("kind,D,A,H,N,B", [(0, 4, 2, 64, 64, 256), (2, 16, 5, 200, 40, 333)])
def test_adam_step_matches_oracle(env, kind, D, A, H, N, B):
    """Adam on the same gradient.  Two regimes: (i) moments with history (t = 5, v0 > 0), where the update is smooth in the
    gradient and the FP32 tolerance applies to every entry; (ii) the first step from zero moments, a sign step of size lr:
    there an entry is compared only where the oracle's |g| exceeds 1e-3 of the group's rms (below that the FP32 summation
    error of g can move the ratio g / (|g| + eps) by O(1)), and everywhere the step must stay within lr."""
    torch, orc, binding = env
    f = fields_for(env_kind=kind, n_envs=N, obs_dim=D, n_actions=A, hidden=H, epsilon=0.3, seed=778, replay_capacity=N * 16,
                   minibatch=B, staleness_bound=20, warmup=N, target_sync_interval=1000, gamma=0.99, huber_delta=1.0,
                   max_episode_steps=9)
    ctx = binding.Context(**f)
    theta_t, theta = blob_for(f, 1), blob_for(f, 2)
    ctx.publish_weights(theta_t)
    ctx.actor_step(6)
    ctx.publish_weights(theta)
    ctx.actor_step(6)
    _, batch = ctx.replay_sample()
    dev = ctx.device
    bn = {k: batch[k].cpu().numpy() for k in ("obs", "act", "rew", "next_obs", "done")}
    rng = np.random.default_rng(1)
    # the oracle's gradient, for the scale of the moments and for the mask of regime (ii)
    o_sgd, _ = orc.sgd_step(theta, theta_t, D, H, A, bn["obs"], bn["act"], bn["rew"], bn["next_obs"], bn["done"], 0.99, 1.0, 1.0)
    g = theta.astype(np.float64) - o_sgd.astype(np.float64)
    g_rms = float(np.sqrt(np.mean(g * g)))
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    ulp = 2 * np.spacing(np.abs(theta).astype(np.float32)).astype(np.float64)      # rounding of theta_new, both sides
    # (i) with history
    m0 = (rng.standard_normal(theta.size) * g_rms).astype(np.float32)
    v0 = ((0.5 + rng.random(theta.size)) * g_rms ** 2).astype(np.float32)
    th, tt = torch.from_numpy(theta.copy()).to(dev), torch.from_numpy(theta_t.copy()).to(dev)
    m, v = torch.from_numpy(m0.copy()).to(dev), torch.from_numpy(v0.copy()).to(dev)
    loss = ctx.adam_step(batch, lr, th, tt, m, v, 5, b1, b2, eps)
    o_new, o_m, o_v, o_loss = orc.adam_step(theta, theta_t, D, H, A, bn["obs"], bn["act"], bn["rew"], bn["next_obs"], bn["done"],
                                            0.99, 1.0, lr, b1, b2, eps, 5, m0, v0)
    assert abs(float(loss.item()) - o_loss) <= 2 * RTOL_FP32 * (abs(o_loss) + 1e-3)
    close(m.cpu().numpy(), o_m, RTOL_FP32, "m")
    close(v.cpu().numpy(), o_v, 3 * RTOL_FP32, "v")      # quadratic in g: twice its relative error, plus rounding
    dg = th.cpu().numpy().astype(np.float64) - theta
    do = o_new.astype(np.float64) - theta
    for name, a, b in _groups(D, H, A):
        rms = np.sqrt(np.mean(do[a:b] ** 2))
        err = np.abs(dg[a:b] - do[a:b])
        assert np.all(err <= RTOL_FP32 * np.abs(do[a:b]) + RTOL_FP32 * rms + ulp[a:b]), (name, err.max(), rms)
    # (ii) first step from zero moments
    th = torch.from_numpy(theta.copy()).to(dev)
    m, v = torch.zeros_like(th), torch.zeros_like(th)
    ctx.adam_step(batch, lr, th, tt, m, v, 1, b1, b2, eps)
    z = np.zeros_like(theta)
    o_new, o_m, o_v, _ = orc.adam_step(theta, theta_t, D, H, A, bn["obs"], bn["act"], bn["rew"], bn["next_obs"], bn["done"],
                                       0.99, 1.0, lr, b1, b2, eps, 1, z, z)
    dg = th.cpu().numpy().astype(np.float64) - theta
    do = o_new.astype(np.float64) - theta
    assert np.all(np.abs(dg) <= lr * (1 + 1e-4) + ulp)
    n_cmp = 0
    for name, a, b in _groups(D, H, A):
        sure = np.abs(g[a:b]) > 1e-3 * np.sqrt(np.mean(g[a:b] ** 2))
        n_cmp += int(sure.sum())
        assert np.all(np.abs(dg[a:b] - do[a:b])[sure] <= 1e-4 * lr + ulp[a:b][sure]), name
        dead = o_m[a:b] == 0                                                   # the gradient is exactly zero there
        assert np.all(dg[a:b][dead] == 0) and np.all(do[a:b][dead] == 0)
    assert n_cmp > 0.5 * np.count_nonzero(g)
    close(m.cpu().numpy(), o_m, RTOL_FP32, "m after the first step")
    assert ctx.stats()["device_error"] == 0


def test_cartpole_dqn_learns_through_the_library(env):
    """The whole path as one system: actor -> ring -> staleness-bounded sampler -> Adam update -> publish.  A random policy
    keeps the pole up for about 10 steps; after 1.2 M env steps the 100-iteration window mean must have passed 60 (it
    reaches ~150 with this seed) and no sampled transition may be staler than the bound."""
    from paper_2502_20190_b200 import train_dqn
    hist = train_dqn.train(staleness_bound=8, iters=1200, seed=1)
    best = max(r["mean_return"] for r in hist if r["episodes"] > 0)
    assert hist[0]["mean_return"] < 15
    assert best > 60, [round(r["mean_return"], 1) for r in hist]
    assert hist[-1]["max_sampled_staleness"] <= 8 and hist[-1]["updates"] > 4000


@pytest.mark.gpu
def test_measured_rates_give_the_balanced_split():
    """Eq. 2-3 from measured rates: the loop at consumed : produced = 1 : 8 reports stand-alone actor and learner rates,
    and the balanced time split built from them predicts a throughput the measured loop cannot exceed (kernel time is part
    of the loop's wall time) and is not far below."""
    from paper_2502_20190_b200 import balance, train_dqn
    k, u = balance.schedule(0.125, 1024, 1024)
    assert (k, u) == (8, 1)
    rates = {}
    h = train_dqn.train(staleness_bound=8, iters=200, actor_steps_per_iter=k, updates_per_iter=u, rates_out=rates)
    assert h[-1]["env_steps"] == 200 * 8 * 1024 and h[-1]["updates"] > 0
    assert rates["P"] == pytest.approx(h[-1]["updates"] * 1024 / h[-1]["env_steps"])
    assert rates["R_A"] > 0 and rates["R_L"] > 0 and 0 < rates["actor_fraction"] < 1
    assert rates["consumed_per_s"] == pytest.approx(rates["P"] * rates["produced_per_s"])
    assert rates["kernel_s"] <= rates["loop_s"]
    assert rates["loop_produced_per_s"] <= rates["produced_per_s"] * 1.001
    assert rates["loop_produced_per_s"] >= 0.1 * rates["produced_per_s"]       # loose: first launches of a kernel are slow and 200 iterations are short
