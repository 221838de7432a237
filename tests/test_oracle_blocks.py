"""Pins for the oracle's building blocks: each is checked against something other
than itself -- published vectors, hand-worked values, physical invariants, closed
forms, library routines or brute force."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


# ------------------------------------------------------------------ Philox4x32-10
def _philox_bigint(ctr, key):
    """Independent restatement with Python integers (no fixed-width types)."""
    M0, M1, W0, W1, mask = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85, 0xFFFFFFFF
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        p0, p1 = M0 * c[0], M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & mask, (p0 >> 32) ^ c[3] ^ k[1], p0 & mask]
        k = [(k[0] + W0) & mask, (k[1] + W1) & mask]
    return c


def test_philox_known_answer_vectors(orc):
    for row in _rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in row]
        assert orc.philox4x32_10(v[0:4], v[4:6]).tolist() == v[6:10]


def test_philox_matches_bigint_restatement(orc):
    rng = np.random.default_rng(1)
    for _ in range(3000):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        assert orc.philox4x32_10(ctr, key).tolist() == _philox_bigint(ctr, key)


def test_philox_avalanche(orc):
    rng = np.random.default_rng(2)
    flips = []
    for _ in range(400):
        ctr = rng.integers(0, 2**32, 4).astype(np.uint32)
        key = rng.integers(0, 2**32, 2).astype(np.uint32)
        a = orc.philox4x32_10(ctr, key)
        c2 = ctr.copy()
        c2[rng.integers(0, 4)] ^= np.uint32(1 << int(rng.integers(0, 32)))
        b = orc.philox4x32_10(c2, key)
        flips.append(sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(a, b)))
    assert abs(np.mean(flips) / 128.0 - 0.5) < 0.02


def test_stream_keying(orc):
    seed, stream, block, c0, step = 0x1122334455667788, 2, 5, 77, (3 << 32) | 9
    want = _philox_bigint([c0, 9, stream | (block << 8), 3], [0x55667788, 0x11223344])
    assert orc.stream_words(seed, stream, block, c0, step).tolist() == want


def test_uniform_is_exact_fp32_and_open_interval(orc):
    for x in (0, 1, 511, 512, 2**31, 2**32 - 1, 123456789):
        want = Fraction(2 * (x >> 9) + 1, 2**24)
        got = orc.u01(x)
        assert Fraction(got) == want and 0.0 < got < 1.0
        assert np.float32(got) == got
    rng = np.random.default_rng(3)
    u = np.array([orc.u01(int(x)) for x in rng.integers(0, 2**32, 20000)])
    assert abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005


def test_mulhi_range_and_definition(orc):
    rng = np.random.default_rng(4)
    for _ in range(1000):
        x, n = int(rng.integers(0, 2**32)), int(rng.integers(1, 2**31))
        assert orc.mulhi(x, n) == (x * n) >> 32 < n


def test_normals_moments_and_unit_circle(orc):
    zs = []
    for i in range(5000):
        w = orc.stream_words(9, orc.STREAM_NOISE, 0, i, 0)
        z = orc.normal4(w)
        # a Box-Muller pair lies on the circle of radius sqrt(-2 ln u1)
        u1 = orc.u01(int(w[0]))
        assert abs(z[0] ** 2 + z[1] ** 2 - (-2.0 * math.log(u1))) < 1e-9
        zs.extend(z)
    zs = np.array(zs)
    assert abs(zs.mean()) < 0.03 and abs(zs.var() - 1.0) < 0.04
    assert abs(np.mean(zs ** 4) - 3.0) < 0.25  # Gaussian kurtosis


def test_explore_threshold(orc):
    assert orc.explore_threshold(0.0) == 0
    assert orc.explore_threshold(1.0) == 2**32
    assert orc.explore_threshold(0.5) == 2**31
    # 0.1 as FP32 is 13421773 * 2^-27; times 2^32 is an integer
    assert orc.explore_threshold(0.1) == 13421773 * 32


# ------------------------------------------------------------------ CartPole
def test_cartpole_hand_worked_step(orc):
    want = [Fraction(int(a), int(b)) for a, b in _rows("cartpole_hand_step.txt")]
    s, r, term, _ = orc.cartpole_step([0, 0, 0, 0], 1)
    for got, w in zip(s, want):
        assert got == np.float32(float(w))
    assert r == 1.0 and term == 0


def test_cartpole_mirror_symmetry(orc):
    rng = np.random.default_rng(5)
    for _ in range(200):
        s = (rng.uniform(-1, 1, 4) * [2.0, 2.0, 0.2, 2.0]).astype(np.float32)
        a = int(rng.integers(0, 2))
        s1, _, t1, _ = orc.cartpole_step(s, a)
        s2, _, t2, _ = orc.cartpole_step(-s, 1 - a)
        assert np.array_equal(s1, -s2) and t1 == t2


def test_cartpole_satisfies_coupled_equations_of_motion(orc):
    """The accelerations implied by one step must satisfy the cart and pole equations in their
    implicit (coupled) form, which the oracle's explicit formulas never write down:
      (m_c+m_p) x'' + m_p l (th'' cos th - th'^2 sin th) = F,   (4/3) l th'' = g sin th - x'' cos th."""
    rng = np.random.default_rng(6)
    g, mc, mp, l, tau = 9.8, 1.0, 0.1, 0.5, 0.02
    for _ in range(300):
        s = (rng.uniform(-1, 1, 4) * [1.0, 2.0, 0.2, 3.0]).astype(np.float32)
        a = int(rng.integers(0, 2))
        sn, _, _, _ = orc.cartpole_step(s, a)
        x, xd, th, thd = [float(v) for v in s]
        xacc = (float(sn[1]) - xd) / tau
        thacc = (float(sn[3]) - thd) / tau
        F = 10.0 if a == 1 else -10.0
        res1 = (mc + mp) * xacc + mp * l * (thacc * math.cos(th) - thd * thd * math.sin(th)) - F
        res2 = (4.0 / 3.0) * l * thacc - (g * math.sin(th) - xacc * math.cos(th))
        assert abs(res1) < 2e-4 and abs(res2) < 2e-4
        # positions move with the old velocities
        assert abs(float(sn[0]) - (x + tau * xd)) < 1e-6 and abs(float(sn[2]) - (th + tau * thd)) < 1e-6


def test_cartpole_termination_thresholds(orc):
    th = 12 * 2 * math.pi / 360
    assert orc.cartpole_step([2.39, 0, 0, 0], 0)[2] == 0
    assert orc.cartpole_step([2.41, 0, 0, 0], 0)[2] == 1
    assert orc.cartpole_step([-2.41, 0, 0, 0], 0)[2] == 1
    assert orc.cartpole_step([0, 0, th * 0.99, 0], 0)[2] == 0
    assert orc.cartpole_step([0, 0, th * 1.01, 0], 0)[2] == 1
    assert orc.cartpole_step([0, 0, -th * 1.01, 0], 0)[2] == 1


def test_cartpole_constant_push_falls_over(orc):
    s = np.zeros(4, np.float32)
    for n in range(1, 100):
        s, _, term, _ = orc.cartpole_step(s, 1)
        if term:
            break
    # pushed right from rest the pole tips backwards and leaves the 12 degree cone; small-angle estimate:
    # th'' ~ -600/41, th = -(300/41) t^2 > 12 deg after t ~ 0.169 s, i.e. within 8 to 12 steps of 0.02 s
    assert term and 8 <= n <= 12 and s[2] < 0


# ------------------------------------------------------------------ Acrobot
def test_acrobot_fixed_point(orc):
    s, r, term, _ = orc.acrobot_step([0, 0, 0, 0], 1)
    assert np.array_equal(s, np.zeros(4, np.float32)) and r == -1.0 and term == 0


def test_acrobot_energy_is_conserved_without_torque(orc):
    rng = np.random.default_rng(7)
    for _ in range(3):
        y = rng.uniform(-1, 1, 4) * [2.0, 2.0, 1.5, 1.5]
        e0 = orc.acrobot_energy(y)
        for _ in range(10000):  # 1 s at dt = 1e-4
            y = orc.acrobot_rk4(y, 0.0, 1e-4)
        assert abs(orc.acrobot_energy(y) - e0) / abs(e0) < 1e-8


def test_acrobot_torque_does_work_at_rate_tau_times_joint_speed(orc):
    # dE/dt = tau * dtheta2/dt for a torque on the second joint
    y = np.array([0.3, -0.4, 0.7, -0.2])
    e0 = orc.acrobot_energy(y)
    work = 0.0
    for _ in range(5000):
        yn = orc.acrobot_rk4(y, 1.0, 1e-4)
        work += 1.0 * 0.5 * (y[3] + yn[3]) * 1e-4
        y = yn
    assert abs((orc.acrobot_energy(y) - e0) - work) < 1e-6


def test_acrobot_rk4_fourth_order(orc):
    y0 = np.array([0.5, -0.3, 0.8, -0.6])
    ref = y0.copy()
    for _ in range(2000):
        ref = orc.acrobot_rk4(ref, 1.0, 1e-4)
    e1 = np.abs(orc.acrobot_rk4(y0, 1.0, 0.2) - ref).max()
    half = orc.acrobot_rk4(orc.acrobot_rk4(y0, 1.0, 0.1), 1.0, 0.1)
    e2 = np.abs(half - ref).max()
    assert 10.0 < e1 / e2 < 26.0


def test_acrobot_antisymmetry_and_obs(orc):
    rng = np.random.default_rng(8)
    for _ in range(100):
        s = (rng.uniform(-1, 1, 4) * [1.0, 1.0, 2.0, 2.0]).astype(np.float32)
        a = int(rng.integers(0, 3))
        s1 = orc.acrobot_step(s, a)[0]
        s2 = orc.acrobot_step(-s, 2 - a)[0]
        assert np.allclose(s1, -s2, atol=1e-6)
    o = orc.acrobot_obs([0.3, -1.2, 0.5, -0.7])
    assert np.allclose(o, [math.cos(0.3), math.sin(0.3), math.cos(-1.2), math.sin(-1.2), 0.5, -0.7], atol=1e-7)


def test_acrobot_wrap_clamp_and_termination(orc):
    s, _, _, _ = orc.acrobot_step([3.1, 0.0, 4.0, 0.0], 1)
    assert -math.pi <= s[0] < math.pi
    s, _, _, _ = orc.acrobot_step([0.0, 0.0, 12.5, 28.0], 2)
    assert abs(s[2]) <= np.float32(4 * math.pi) and abs(s[3]) <= np.float32(9 * math.pi)
    # tip height -cos(th1) - cos(th1+th2): straight up gives 2 > 1 (terminated, reward 0)
    s, r, term, _ = orc.acrobot_step([math.pi - 0.01, 0.0, 0.0, 0.0], 1)
    assert term == 1 and r == 0.0
    s, r, term, _ = orc.acrobot_step([0.1, 0.0, 0.0, 0.0], 1)
    assert term == 0 and r == -1.0


# ------------------------------------------------------------------ linear-Gaussian env
def test_lingauss_special_cases(orc):
    D = 8
    Z = np.zeros((D, D), np.float32)
    Bz = np.zeros((3, D), np.float32)
    s = np.linspace(-1, 1, D).astype(np.float32)
    sn, r, term, _ = orc.lingauss_step(s, 0, Z, Bz, np.zeros(D), 0.01, 4.0)
    assert np.array_equal(sn, np.zeros(D, np.float32)) and r == 0.0 and term == 0
    c = 0.25
    sn, r, term, _ = orc.lingauss_step(s, 1, c * np.eye(D, dtype=np.float32), Bz, np.zeros(D), 0.01, 4.0)
    assert np.allclose(sn, np.tanh(c * s.astype(np.float64)), atol=1e-7)
    assert abs(r + float(np.sum(sn.astype(np.float64) ** 2)) / D) < 1e-7
    noise = np.arange(D, dtype=np.float64)
    sn, _, _, _ = orc.lingauss_step(s, 0, Z, Bz, noise, 0.01, 4.0)
    assert np.allclose(sn, 0.01 * noise, atol=1e-8)


def test_lingauss_matches_library_matvec_and_norm_rule(orc):
    rng = np.random.default_rng(9)
    D, A_ = 128, 16
    A = (rng.standard_normal((D, D)) / math.sqrt(D)).astype(np.float32)
    Bm = rng.standard_normal((A_, D)).astype(np.float32)
    s = rng.uniform(-0.1, 0.1, D).astype(np.float32)
    noise = rng.standard_normal(D)
    for a in (0, 7, 15):
        sn, r, term, m = orc.lingauss_step(s, a, A, Bm, noise, 0.01, 4.0)
        want = np.tanh(A.astype(np.float64) @ s.astype(np.float64) + Bm[a]) + 0.01 * noise
        assert np.allclose(sn, want, atol=2e-7)
        nrm = float(np.linalg.norm(sn.astype(np.float64)))
        assert abs(r + nrm ** 2 / D) < 1e-6 and term == int(nrm > 4.0)
        assert abs(m - abs(nrm - 4.0) / 4.0) < 1e-12


# ------------------------------------------------------------------ MLP
def _round_f32(q: Fraction) -> Fraction:
    """Exact round-to-nearest-even of a rational to FP32 (normal range)."""
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    q = abs(q)
    e = q.numerator.bit_length() - q.denominator.bit_length() - 24
    while q / Fraction(2) ** e >= 2 ** 24:
        e += 1
    while q / Fraction(2) ** e < 2 ** 23:
        e -= 1
    scaled = q / Fraction(2) ** e
    n, rem = divmod(scaled.numerator, scaled.denominator)
    twice = 2 * rem
    if twice > scaled.denominator or (twice == scaled.denominator and (n & 1)):
        n += 1
    return sign * n * Fraction(2) ** e


def _mlp_exact_rounding(blob, D, H, A, x):
    """bias first, then one correctly rounded multiply-add per input in index order, in exact rationals."""
    def dense(W, b, xs, relu):
        out = []
        for i in range(W.shape[0]):
            acc = Fraction(float(b[i]))
            for k in range(W.shape[1]):
                acc = _round_f32(Fraction(float(W[i, k])) * xs[k] + acc)
            out.append(max(acc, Fraction(0)) if relu else acc)
        return out
    o = 0
    W1 = blob[o:o + H * D].reshape(H, D); o += H * D
    b1 = blob[o:o + H]; o += H
    W2 = blob[o:o + H * H].reshape(H, H); o += H * H
    b2 = blob[o:o + H]; o += H
    W3 = blob[o:o + A * H].reshape(A, H); o += A * H
    b3 = blob[o:o + A]
    h1 = dense(W1, b1, [Fraction(float(v)) for v in x], True)
    h2 = dense(W2, b2, h1, True)
    return [float(v) for v in dense(W3, b3, h2, False)]


def test_mlp_fp32_rounding_order_is_bias_then_fma_chain(orc):
    rng = np.random.default_rng(10)
    D, H, A = 4, 8, 3
    blob = rng.standard_normal(orc.blob_floats(D, H, A)).astype(np.float32)
    for _ in range(5):
        x = rng.standard_normal(D).astype(np.float32)
        got = orc.mlp_forward(blob, D, H, A, x)
        want = np.array(_mlp_exact_rounding(blob, D, H, A, x), np.float32)
        assert np.array_equal(got, want)


def test_mlp_matches_float64_library_matmul(orc):
    rng = np.random.default_rng(11)
    for D, H, A, vh in ((4, 64, 2, False), (6, 256, 3, False), (4, 256, 2, True), (128, 512, 16, False)):
        n = orc.blob_floats(D, H, A, vh)
        blob = (rng.standard_normal(n) * 0.2).astype(np.float32)
        x = rng.standard_normal(D).astype(np.float32)
        o = 0
        W1 = blob[o:o + H * D].reshape(H, D).astype(np.float64); o += H * D
        b1 = blob[o:o + H].astype(np.float64); o += H
        W2 = blob[o:o + H * H].reshape(H, H).astype(np.float64); o += H * H
        b2 = blob[o:o + H].astype(np.float64); o += H
        W3 = blob[o:o + A * H].reshape(A, H).astype(np.float64); o += A * H
        b3 = blob[o:o + A].astype(np.float64); o += A
        h2 = np.maximum(W2 @ np.maximum(W1 @ x + b1, 0) + b2, 0)
        want = W3 @ h2 + b3
        if vh:
            Wv = blob[o:o + H].astype(np.float64); o += H
            want_v = float(Wv @ h2 + blob[o])
            out64, v64 = orc.mlp_forward(blob, D, H, A, x, value_head=True, f64=True)
            out32, v32 = orc.mlp_forward(blob, D, H, A, x, value_head=True)
            assert abs(v64 - want_v) < 1e-12 * (1 + abs(want_v)) and abs(v32 - want_v) < 1e-5 * (1 + abs(want_v))
        else:
            out64 = orc.mlp_forward(blob, D, H, A, x, f64=True)
            out32 = orc.mlp_forward(blob, D, H, A, x)
        scale = np.sqrt(np.mean(want ** 2))
        assert np.allclose(out64, want, rtol=1e-12, atol=1e-12)
        assert np.abs(out32 - want).max() <= 1e-5 * (np.abs(want).max() + scale)


def test_mlp_hand_case_and_relu(orc):
    # D=1, H=1, A=1: out = w3 * relu(w2 * relu(w1 x + b1) + b2) + b3
    blob = np.array([2.0, 0.5, -1.0, 0.25, 3.0, -0.125], np.float32)
    assert orc.mlp_forward(blob, 1, 1, 1, [1.0])[0] == 3.0 * 0.0 - 0.125      # w2*2.5+0.25 < 0 -> relu
    blob[2] = 1.0
    assert orc.mlp_forward(blob, 1, 1, 1, [1.0])[0] == 3.0 * 2.75 - 0.125
    assert orc.mlp_forward(blob, 1, 1, 1, [-1.0])[0] == 3.0 * 0.25 - 0.125    # first relu clips 2*-1+0.5


def test_bf16_round_nearest_even(orc):
    assert orc.bf16_round(1.0) == 1.0
    assert orc.bf16_round(1.0 + 2 ** -8) == 1.0               # tie -> even mantissa
    assert orc.bf16_round(1.0 + 2 ** -7 + 2 ** -8) == 1.0 + 2 ** -6   # tie -> even (rounds up)
    assert orc.bf16_round(1.0 + 2 ** -8 + 2 ** -12) == 1.0 + 2 ** -7
    assert orc.bf16_round(-3.140625) == -3.140625


# ------------------------------------------------------------------ selection
def test_argmax_lowest_index_ties(orc):
    assert orc.argmax_lowest([1.0, 1.0, 1.0]) == 0
    assert orc.argmax_lowest([0.0, 2.0, 2.0]) == 1
    assert orc.argmax_lowest([-1.0, -3.0, -0.5]) == 2
    assert orc.argmax_lowest([float("nan"), 1.0]) == 1 or orc.argmax_lowest([float("nan"), 1.0]) == 0
    assert orc.argmax_lowest([1.0, float("nan")]) == 0


def test_eps_greedy_limits_and_frequency(orc):
    q = np.array([0.1, 0.7, 0.3], np.float32)
    rng = np.random.default_rng(12)
    thr0, thr1, thr = orc.explore_threshold(0.0), orc.explore_threshold(1.0), orc.explore_threshold(0.1)
    counts = np.zeros(3)
    explored = 0
    n = 30000
    for _ in range(n):
        x0, x1 = int(rng.integers(0, 2**32)), int(rng.integers(0, 2**32))
        assert orc.select_eps_greedy(q, x0, x1, thr0) == 1
        a = orc.select_eps_greedy(q, x0, x1, thr1)
        assert a == (x1 * 3) >> 32
        counts[a] += 1
        explored += orc.select_eps_greedy(q, x0, x1, thr) != 1 or (x0 < thr and ((x1 * 3) >> 32) == 1)
    assert np.all(np.abs(counts / n - 1 / 3) < 0.015)
    assert abs(explored / n - 0.1) < 3 * math.sqrt(0.1 * 0.9 / n) + 1e-3


def test_categorical_definition(orc):
    assert orc.select_categorical([0.0, 0.0], 0.49)[0] == 0
    assert orc.select_categorical([0.0, 0.0], 0.51)[0] == 1
    lg = np.array([0.2, -1.0, 1.3, 0.0], np.float32)
    p = np.exp(lg.astype(np.float64) - lg.max())
    p /= p.sum()
    cdf = np.cumsum(p)
    for u in np.linspace(0.001, 0.999, 97):
        a, logp, margin = orc.select_categorical(lg, np.float32(u))
        want = int(np.searchsorted(cdf, float(np.float32(u)), side="right"))
        assert a == min(want, 3)
        assert abs(logp - math.log(p[a])) < 1e-12
        assert abs(margin - np.min(np.abs(cdf[:-1] - float(np.float32(u))))) < 1e-12


# ------------------------------------------------------------------ TD / Huber, GAE
def test_td_hand_values(orc):
    for row in _rows("td_hand_values.txt"):
        r, gamma, qn, qs, done, y, delta, hub = [float(v) for v in row]
        td, h = orc.td_one(qs, qn, r, int(done), gamma, 1.0)
        assert abs(td - delta) < 1e-12 and abs(h - hub) < 1e-12 and abs((td + qs) - y) < 1e-12


def test_huber_continuity_and_symmetry(orc):
    k = 1.0
    lo = orc.td_one(0.0, 0.0, k * (1 - 1e-9), 0, 0.0, k)[1]
    hi = orc.td_one(0.0, 0.0, k * (1 + 1e-9), 0, 0.0, k)[1]
    assert abs(lo - hi) < 1e-8 and abs(lo - 0.5) < 1e-8
    assert orc.td_one(0.0, 0.0, 2.5, 0, 0.0, k)[1] == orc.td_one(0.0, 0.0, -2.5, 0, 0.0, k)[1] == 2.0
    # gamma = 0 -> delta = r - q
    assert orc.td_one(0.3, 9.0, 1.0, 0, 0.0, k)[0] == pytest.approx(0.7)


def test_gae_lambda_one_is_discounted_return_minus_value(orc):
    rng = np.random.default_rng(13)
    T, N, g = 17, 5, 0.97
    rew = rng.standard_normal((T, N)).astype(np.float32)
    val = rng.standard_normal((T + 1, N)).astype(np.float32)
    done = np.zeros((T, N), np.uint8)
    adv, ret = orc.gae(rew, val, done, g, 1.0)
    for t in range(T):
        G = sum(g ** k * rew[t + k].astype(np.float64) for k in range(T - t)) + g ** (T - t) * val[T]
        assert np.allclose(adv[t], G - val[t], atol=1e-10)
        assert np.allclose(ret[t], G, atol=1e-10)


def test_gae_lambda_zero_and_geometric_closed_form(orc):
    rng = np.random.default_rng(14)
    T, N, g, lam = 12, 4, 0.99, 0.95
    rew = rng.standard_normal((T, N)).astype(np.float32)
    val = rng.standard_normal((T + 1, N)).astype(np.float32)
    done = (rng.random((T, N)) < 0.2).astype(np.uint8)
    adv, _ = orc.gae(rew, val, done, g, 0.0)
    delta = rew + g * (1 - done) * val[1:].astype(np.float64) - val[:-1]
    assert np.allclose(adv, delta, atol=1e-12)
    ones, zeros = np.ones((T, N), np.float32), np.zeros((T + 1, N), np.float32)
    adv, ret = orc.gae(ones, zeros, np.zeros((T, N), np.uint8), g, lam)
    for t in range(T):
        assert np.allclose(adv[t], (1 - (g * lam) ** (T - t)) / (1 - g * lam), atol=1e-12)
    assert np.allclose(adv, ret)


def test_gae_done_cuts_the_future_and_matches_bruteforce_sum(orc):
    rng = np.random.default_rng(15)
    T, N, g, lam = 14, 6, 0.9, 0.8
    rew = rng.standard_normal((T, N)).astype(np.float32)
    val = rng.standard_normal((T + 1, N)).astype(np.float32)
    done = (rng.random((T, N)) < 0.25).astype(np.uint8)
    adv, ret = orc.gae(rew, val, done, g, lam)
    delta = rew + g * (1 - done) * val[1:].astype(np.float64) - val[:-1]
    for e in range(N):
        for t in range(T):
            tot, w = 0.0, 1.0
            for l in range(T - t):
                tot += w * delta[t + l, e]
                w *= g * lam * (1 - done[t + l, e])
            assert abs(adv[t, e] - tot) < 1e-10
    # changing anything after a done leaves earlier advantages untouched
    e, t = np.argwhere(done.T)[0]
    rew2 = rew.copy()
    rew2[t + 1:, e] += 100.0
    val2 = val.copy()
    val2[t + 1:, e] -= 50.0
    adv2, _ = orc.gae(rew2, val2, done, g, lam)
    assert np.array_equal(adv2[:t + 1, e], adv[:t + 1, e])
    assert np.allclose(ret, adv + val[:-1])
