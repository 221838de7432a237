"""Pins for the oracle's learner update (Algorithm 1: theta <- theta + alpha * delta * grad V(s; theta), as a minibatch
semi-gradient step on the mean Huber loss with a target network).

The update is checked against things it does not compute itself: central finite differences of the loss assembled from
the already pinned forward pass and TD/Huber routine, the closed form of Algorithm 1's line for a single transition, and
invariants (zero error, clipping, batch mean)."""
import numpy as np
import pytest

import oracle

D, H, A = 5, 12, 3
GAMMA, KAPPA = 0.97, 1.0


def _blob(rng, scale=0.6):
    n = oracle.blob_floats(D, H, A)
    return (rng.standard_normal(n) * scale).astype(np.float32)


def _batch(rng, n):
    return dict(obs=rng.standard_normal((n, D)).astype(np.float32), act=rng.integers(0, A, n).astype(np.int32),
                rew=rng.standard_normal(n).astype(np.float32), next_obs=rng.standard_normal((n, D)).astype(np.float32),
                done=(rng.random(n) < 0.3).astype(np.int32))


def _loss(theta, theta_target, b, kappa=KAPPA):
    """mean Huber loss from the pinned building blocks: float64 forward passes and the one-transition TD routine"""
    tot = 0.0
    for j in range(len(b["act"])):
        q = oracle.mlp_forward(theta, D, H, A, b["obs"][j], f64=True)[b["act"][j]]
        qn = oracle.mlp_forward(theta_target, D, H, A, b["next_obs"][j], f64=True).max()
        _, hub = oracle.td_one(q, qn, float(b["rew"][j]), int(b["done"][j]), GAMMA, kappa)
        tot += hub
    return tot / len(b["act"])


def _step(theta, target, b, lr, kappa=KAPPA):
    return oracle.sgd_step(theta, target, D, H, A, b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], GAMMA, kappa, lr)


def test_update_is_minus_lr_times_finite_difference_gradient():
    rng = np.random.default_rng(5)
    theta, target, b = _blob(rng), _blob(rng), _batch(rng, 9)
    lr = 0.25
    new, loss = _step(theta, target, b, lr)
    assert abs(loss - _loss(theta, target, b)) < 1e-12 * (1 + abs(loss))
    grad = (theta.astype(np.float64) - new.astype(np.float64)) / lr
    # every parameter group, a few entries each; the float32 rounding of theta_new limits the agreement
    n1, n2, n3 = H * D, H * H, A * H
    offs = [0, n1, n1 + H, n1 + H + n2, n1 + 2 * H + n2, n1 + 2 * H + n2 + n3]
    sizes = [n1, H, n2, H, n3, A]
    eps = 1e-3
    checked = 0
    for o, sz in zip(offs, sizes):
        for i in rng.choice(sz, size=min(6, sz), replace=False):
            tp, tm = theta.copy(), theta.copy()
            tp[o + i] += eps
            tm[o + i] -= eps
            h = (float(tp[o + i]) - float(tm[o + i]))          # the step actually taken in float32
            fd = (_loss(tp, target, b) - _loss(tm, target, b)) / h
            assert abs(fd - grad[o + i]) <= 2e-3 * max(1e-2, abs(fd)) + 5e-6, (o, i, fd, grad[o + i])
            checked += 1
    assert checked >= 30
    assert np.abs(grad).max() > 1e-3                            # the comparison is not about zeros


def test_single_transition_is_algorithm_one_line():
    """n = 1, no clipping, target = online: theta += lr * delta * grad Q(s, a; theta)."""
    rng = np.random.default_rng(11)
    theta = _blob(rng)
    b = _batch(rng, 1)
    b["done"][:] = 0
    lr = 0.1
    new, _ = _step(theta, theta, b, lr, kappa=1e30)
    t = theta.astype(np.float64)
    n1, n2, n3 = H * D, H * H, A * H
    W1, b1 = t[:n1].reshape(H, D), t[n1:n1 + H]
    W2, b2 = t[n1 + H:n1 + H + n2].reshape(H, H), t[n1 + H + n2:n1 + 2 * H + n2]
    W3, b3 = t[n1 + 2 * H + n2:n1 + 2 * H + n2 + n3].reshape(A, H), t[n1 + 2 * H + n2 + n3:]
    x, a = b["obs"][0].astype(np.float64), int(b["act"][0])
    h1 = np.maximum(W1 @ x + b1, 0)
    h2 = np.maximum(W2 @ h1 + b2, 0)
    q = W3 @ h2 + b3
    xn = b["next_obs"][0].astype(np.float64)
    qn = (W3 @ np.maximum(W2 @ np.maximum(W1 @ xn + b1, 0) + b2, 0) + b3).max()
    delta = float(b["rew"][0]) + GAMMA * qn - q[a]
    d = new.astype(np.float64) - t
    ob3 = n1 + 2 * H + n2 + n3
    oW3 = n1 + 2 * H + n2
    assert abs(delta) > 1e-2
    for k in range(A):                                          # grad of Q(s,a) w.r.t. b3 is the unit vector e_a
        assert abs(d[ob3 + k] - (lr * delta if k == a else 0.0)) < 1e-6 * (1 + abs(delta))
    np.testing.assert_allclose(d[oW3 + a * H: oW3 + (a + 1) * H], lr * delta * h2, atol=2e-6 * (1 + abs(delta) * np.abs(h2).max()))
    other = [k for k in range(A) if k != a]
    for k in other:
        assert np.all(d[oW3 + k * H: oW3 + (k + 1) * H] == 0.0)


def test_zero_error_changes_nothing_and_clipping_saturates():
    rng = np.random.default_rng(3)
    theta, target, b = _blob(rng), _blob(rng), _batch(rng, 4)
    # choose the rewards that make every TD error vanish
    for j in range(4):
        q = oracle.mlp_forward(theta, D, H, A, b["obs"][j], f64=True)[b["act"][j]]
        qn = oracle.mlp_forward(target, D, H, A, b["next_obs"][j], f64=True).max()
        b["rew"][j] = np.float32(q - GAMMA * (0.0 if b["done"][j] else 1.0) * qn)
    new, loss = _step(theta, target, b, 1.0)
    assert loss < 1e-10 and np.max(np.abs(new - theta)) < 1e-6
    # far outside the quadratic zone the update no longer depends on the size of the error
    b1, b2 = dict(b), dict(b)
    b1["rew"] = b["rew"] + 50.0
    b2["rew"] = b["rew"] + 500.0
    n1, _ = _step(theta, target, b1, 0.3)
    n2, _ = _step(theta, target, b2, 0.3)
    assert np.array_equal(n1, n2) and np.max(np.abs(n1 - theta)) > 1e-3
    n3, _ = _step(theta, target, dict(b, rew=b["rew"] - 50.0), 0.3)
    np.testing.assert_allclose(n3 - theta, -(n1 - theta), atol=1e-6)


def test_update_is_a_batch_mean():
    rng = np.random.default_rng(8)
    theta, target, b = _blob(rng), _blob(rng), _batch(rng, 6)
    twice = {k: np.concatenate([v, v]) for k, v in b.items()}
    n1, l1 = _step(theta, target, b, 0.2)
    n2, l2 = _step(theta, target, twice, 0.2)
    np.testing.assert_allclose(n1, n2, atol=1e-7)
    assert abs(l1 - l2) < 1e-12


# ------------------------------------------------------------------------------------------------ Adam (Table 2)
def _adam(theta, target, b, lr, b1, b2, eps, t, m, v):
    return oracle.adam_step(theta, target, D, H, A, b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], GAMMA, KAPPA, lr,
                            b1, b2, eps, t, m, v)


def _gradient(theta, target, b):
    """the gradient the pinned SGD step applies (lr = 1 keeps the most digits)"""
    new, _ = _step(theta, target, b, 1.0)
    return theta.astype(np.float64) - new.astype(np.float64)


def test_adam_first_step_has_the_closed_form():
    """From m = v = 0 the bias-corrected moments are g and g^2: the first update is -lr * g / (|g| + eps)."""
    rng = np.random.default_rng(21)
    theta, target, b = _blob(rng), _blob(rng), _batch(rng, 7)
    g = _gradient(theta, target, b)
    z = np.zeros_like(theta)
    lr, b1, b2, eps = 0.01, 0.9, 0.999, 1e-8
    new, m, v, loss = _adam(theta, target, b, lr, b1, b2, eps, 1, z, z)
    assert abs(loss - _loss(theta, target, b)) < 1e-12 * (1 + abs(loss))
    big = np.abs(g) > 1e-4                                    # where the float32 storage of g, m and v does not blur the ratio
    assert big.sum() > 50
    d = new.astype(np.float64) - theta.astype(np.float64)
    np.testing.assert_allclose(d[big], -lr * np.sign(g[big]), rtol=2e-3)          # |g| >> eps: a sign step of size lr
    np.testing.assert_allclose(m[big], (1 - b1) * g[big], rtol=1e-3)
    np.testing.assert_allclose(v[big], (1 - b2) * g[big] ** 2, rtol=2e-3)
    assert np.all(d[g == 0] == 0)                             # untouched rows (other actions' head weights) do not move


def test_adam_recurrence_and_limits():
    rng = np.random.default_rng(22)
    theta, target, b = _blob(rng), _blob(rng), _batch(rng, 5)
    g = _gradient(theta, target, b)
    m0 = (rng.standard_normal(theta.size) * 1e-2).astype(np.float32)
    v0 = (rng.random(theta.size) * 1e-3).astype(np.float32)
    lr, b1, b2, eps, t = 0.003, 0.8, 0.95, 1e-6, 4
    new, m, v, _ = _adam(theta, target, b, lr, b1, b2, eps, t, m0, v0)
    m_ref = b1 * m0.astype(np.float64) + (1 - b1) * g
    v_ref = b2 * v0.astype(np.float64) + (1 - b2) * g * g
    np.testing.assert_allclose(m, m_ref, rtol=1e-5, atol=1e-9)
    np.testing.assert_allclose(v, v_ref, rtol=1e-5, atol=1e-12)
    upd = -lr * (m_ref / (1 - b1 ** t)) / (np.sqrt(v_ref / (1 - b2 ** t)) + eps)
    np.testing.assert_allclose(new.astype(np.float64) - theta, upd, rtol=1e-3, atol=3e-7)
    # beta1 = beta2 = 0: no memory, every step is the first step's sign rule whatever m and v held
    n0, _, _, _ = _adam(theta, target, b, lr, 0.0, 0.0, 1e-12, 9, m0, v0)
    big = np.abs(g) > 1e-4
    np.testing.assert_allclose((n0.astype(np.float64) - theta)[big], -lr * np.sign(g[big]), rtol=2e-3)
    # lr = 0 moves nothing but still advances the moments
    n1, m1, _, _ = _adam(theta, target, b, 0.0, b1, b2, eps, t, m0, v0)
    assert np.array_equal(n1, theta) and not np.array_equal(m1, m0)
