"""Pins for the oracle's on-policy update (PPO's clipped surrogate, value loss and entropy bonus on the shared-trunk
network, Sec. 4.1 / Table 2 of the paper for the hyper-parameters; the objective is Schulman et al. 2017, Eq. 7 and 9).

The gradient is recovered from the first Adam step (from zero moments m_1 = (1 - beta1) g) and checked against central finite
differences of the loss written out here from the pinned forward pass; further pins are the cases with a closed form:
ratio 1 (the plain policy gradient), a saturated clip (no policy gradient), uniform logits (entropy log A, no entropy
gradient) and the value head alone."""
import numpy as np

import oracle

D, H, A = 4, 10, 3
CLIP, CV, CE = 0.2, 0.5, 0.01


def _blob(rng, scale=0.5):
    return (rng.standard_normal(oracle.blob_floats(D, H, A, True)) * scale).astype(np.float32)


def _forward(theta, x):
    logits, v = oracle.mlp_forward(theta, D, H, A, x, value_head=True, f64=True)
    return np.asarray(logits, np.float64), float(v)


def _batch(rng, theta_old, n, adv_scale=1.0):
    obs = rng.standard_normal((n, D)).astype(np.float32)
    act = rng.integers(0, A, n).astype(np.int32)
    logp = np.zeros(n, np.float32)
    for j in range(n):
        l, _ = _forward(theta_old, obs[j])
        logp[j] = l[act[j]] - (l.max() + np.log(np.exp(l - l.max()).sum()))
    return dict(obs=obs, act=act, logp_old=logp, adv=(rng.standard_normal(n) * adv_scale).astype(np.float32),
                ret=rng.standard_normal(n).astype(np.float32))


def _loss(theta, b, clip=CLIP, cv=CV, ce=CE):
    """The objective, written from its definition on top of the pinned forward pass; returns (loss, parts)."""
    pi = vl = ent = nclip = 0.0
    n = len(b["act"])
    for j in range(n):
        l, v = _forward(theta, b["obs"][j])
        logp_all = l - (l.max() + np.log(np.exp(l - l.max()).sum()))
        p = np.exp(logp_all)
        ratio = np.exp(logp_all[b["act"][j]] - float(b["logp_old"][j]))
        a = float(b["adv"][j])
        t1, t2 = ratio * a, np.clip(ratio, 1 - clip, 1 + clip) * a
        pi += -min(t1, t2)
        nclip += float(t2 < t1)
        vl += 0.5 * (v - float(b["ret"][j])) ** 2
        ent += -(p * logp_all).sum()
    return (pi + cv * vl - ce * ent) / n, np.array([pi, vl, ent, nclip]) / n


def _grad(theta, b, clip=CLIP, cv=CV, ce=CE):
    """gradient from the first Adam step: m_1 = (1 - beta1) g with beta1 = 0.5 (exact up to the float32 storage of m)"""
    z = np.zeros_like(theta)
    _, m, _, loss, stats = oracle.ppo_step(theta, D, H, A, b["obs"], b["act"], b["logp_old"], b["adv"], b["ret"], clip, cv, ce,
                                           1e-3, 0.5, 0.9, 1e-8, 1, z, z)
    return m.astype(np.float64) * 2.0, loss, stats


def test_gradient_matches_finite_differences_and_loss_parts():
    rng = np.random.default_rng(2)
    theta_old, theta = _blob(rng), None
    theta = (theta_old + rng.standard_normal(theta_old.size).astype(np.float32) * 0.05).astype(np.float32)   # ratios around 1
    b = _batch(rng, theta_old, 12)
    g, loss, stats = _grad(theta, b)
    ref, parts = _loss(theta, b)
    assert abs(loss - ref) < 1e-12 * (1 + abs(ref))
    np.testing.assert_allclose(stats, parts, rtol=1e-12, atol=1e-14)
    assert 0 < parts[3] < 1                                     # some rows clipped, some not: both branches are exercised
    eps = 1e-4            # small: the loss has kinks (ReLU, clip, min), a wide stencil would straddle them
    idx = rng.choice(theta.size, size=48, replace=False)
    idx = np.concatenate([idx, [theta.size - 1, theta.size - 2, theta.size - H - 2]])      # bv, Wv, b3 explicitly
    for i in idx:
        tp, tm = theta.copy(), theta.copy()
        tp[i] += eps
        tm[i] -= eps
        fd = (_loss(tp, b)[0] - _loss(tm, b)[0]) / (float(tp[i]) - float(tm[i]))
        assert abs(fd - g[i]) <= 1e-4 * max(1e-2, abs(fd)) + 1e-6, (i, fd, g[i])
    assert np.abs(g).max() > 1e-3


def test_ratio_one_is_the_plain_policy_gradient():
    """At theta = theta_old every ratio is 1 and nothing is clipped: with c_v = c_e = 0 the gradient of the head bias is
    -mean_j A_j (e_{a_j} - p_j), the REINFORCE form."""
    rng = np.random.default_rng(4)
    theta = _blob(rng)
    b = _batch(rng, theta, 9)
    g, _, stats = _grad(theta, b, cv=0.0, ce=0.0)
    assert stats[3] == 0.0
    want = np.zeros(A)
    for j in range(9):
        l, _ = _forward(theta, b["obs"][j])
        p = np.exp(l - l.max())
        p /= p.sum()
        e = np.zeros(A)
        e[b["act"][j]] = 1.0
        want += -float(b["adv"][j]) * (e - p) / 9
    o_b3 = H * D + H + H * H + H + A * H
    np.testing.assert_allclose(g[o_b3:o_b3 + A], want, rtol=1e-5, atol=1e-8)
    assert np.all(g[o_b3 + A:] == 0)                           # the value head is out of the game with c_v = 0


def test_saturated_clip_stops_the_policy_gradient_and_value_head_is_least_squares():
    rng = np.random.default_rng(6)
    theta = _blob(rng)
    b = _batch(rng, theta, 7)
    # make every ratio e^{+1} with positive advantages (clipped at 1 + eps) : the surrogate is flat in theta
    b["logp_old"] = (b["logp_old"] - 1.0).astype(np.float32)
    b["adv"] = np.abs(b["adv"]) + 0.1
    g, _, stats = _grad(theta, b, cv=0.0, ce=0.0)
    assert stats[3] == 1.0 and np.all(g == 0)
    # and with negative advantages the same ratios are on the unclipped side
    b2 = dict(b, adv=-b["adv"])
    g2, _, stats2 = _grad(theta, b2, cv=0.0, ce=0.0)
    assert stats2[3] == 0.0 and np.abs(g2).max() > 1e-3
    # value head alone: d/dbv of c_v/2 mean (V - R)^2 = c_v mean (V - R)
    g3, _, _ = _grad(theta, b, cv=0.7, ce=0.0)
    want = 0.7 * np.mean([_forward(theta, b["obs"][j])[1] - float(b["ret"][j]) for j in range(7)])
    assert abs(g3[-1] - want) < 1e-6 * (1 + abs(want))


def test_entropy_of_uniform_logits():
    """Zero head weights and biases: p is uniform, H = log A, and the entropy bonus has no gradient there."""
    rng = np.random.default_rng(9)
    theta = _blob(rng)
    o_W3 = H * D + H + H * H + H
    theta[o_W3:o_W3 + A * H + A] = 0.0
    b = _batch(rng, theta, 5)
    b["adv"][:] = 0.0
    g, loss, stats = _grad(theta, b, cv=0.0, ce=1.0)
    assert abs(stats[2] - np.log(A)) < 1e-12 and abs(loss + np.log(A)) < 1e-12
    assert np.abs(g).max() < 1e-9
