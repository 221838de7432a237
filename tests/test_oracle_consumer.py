"""Pins for the oracle's on-policy consumer pieces: the keyed shuffle of segment rows and the advantage normalisation."""
import numpy as np
import pytest


@pytest.mark.parametrize("R", [1, 2, 3, 4, 5, 16, 17, 100, 255, 256, 257, 1000, 4097])
def test_shuffle_is_a_bijection_for_any_row_count(orc, R):
    for sid in (0, 1, 2**40 + 7):
        order = orc.shuffle_order(99, sid, R)
        assert sorted(order.tolist()) == list(range(R))


def test_shuffle_depends_on_seed_and_id_and_nothing_else(orc):
    a = orc.shuffle_order(5, 1, 500)
    assert np.array_equal(a, orc.shuffle_order(5, 1, 500))           # deterministic
    b, c = orc.shuffle_order(5, 2, 500), orc.shuffle_order(6, 1, 500)
    assert (a != b).mean() > 0.9 and (a != c).mean() > 0.9           # another id or seed: another order
    assert (a != np.arange(500)).mean() > 0.9                        # and not the identity
    assert orc.shuffle_index(5, 1, 500, 500) == -1 and orc.shuffle_index(5, 1, 0, 0) == -1


def test_shuffle_positions_are_uniform(orc):
    """Over many shuffle ids every row lands in every position about equally often (chi-square on a 24 x 24 table),
    and neighbours do not stay neighbours."""
    R, n = 24, 6000
    table = np.zeros((R, R))
    adjacent = 0
    for sid in range(n):
        order = orc.shuffle_order(1234, sid, R)
        table[np.arange(R), order] += 1
        adjacent += int(np.sum(np.abs(np.diff(order)) == 1))
    expect = n / R
    chi2 = np.sum((table - expect) ** 2 / expect)
    dof = (R - 1) ** 2
    assert chi2 < dof + 6 * np.sqrt(2 * dof)
    # in a uniform permutation a given adjacent pair differs by one with probability 2 / R
    assert abs(adjacent / (n * (R - 1)) - 2 / R) < 0.01


def test_shuffle_matches_a_big_integer_restatement_of_the_construction(orc):
    """Four Feistel rounds on 2*hb bits, round function = first SHUFFLE word of (right half, id, round), then cycle walking;
    restated with Python integers on top of the separately pinned Philox stream."""
    seed, sid, R = 77, 3, 300
    bits = (R - 1).bit_length()
    hb = max(1, (bits + 1) // 2)
    mask = (1 << hb) - 1

    def feistel(x):
        left, right = x >> hb, x & mask
        for rnd in range(4):
            f = int(orc.stream_words(seed, orc.STREAM_SHUFFLE, rnd, right, sid)[0]) & mask
            left, right = right, left ^ f
        return (left << hb) | right

    for i in range(0, R, 7):
        y = feistel(i)
        while y >= R:
            y = feistel(y)
        assert orc.shuffle_index(seed, sid, R, i) == y


def test_normalize_hand_values_and_moments(orc):
    out = orc.normalize([1.0, 2.0, 3.0], eps=0.0)
    assert np.allclose(out, [-np.sqrt(1.5), 0.0, np.sqrt(1.5)], atol=1e-12)
    rng = np.random.default_rng(3)
    x = (5.0 + 3.0 * rng.standard_normal(10001)).astype(np.float32)
    out = orc.normalize(x, eps=1e-8)
    assert abs(out.mean()) < 1e-12 and abs(out.var() - 1.0) < 1e-7
    # invariant under a positive affine map of the input
    y = (2.5 * x.astype(np.float64) - 7.0).astype(np.float32)
    assert np.allclose(orc.normalize(y, 1e-8), out, atol=5e-6)
    # a constant input has no spread: all zeros, not a division by zero
    assert np.array_equal(orc.normalize(np.full(10, 4.0, np.float32), 1e-8), np.zeros(10))
    # against the library routine
    assert np.allclose(out, (x.astype(np.float64) - x.astype(np.float64).mean()) / (x.astype(np.float64).std() + 1e-8), atol=1e-12)
