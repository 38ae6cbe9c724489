"""Pins for the oracle's action sampling from logits (policy interface)."""
import math

import numpy as np

import oracle


def test_expn_accuracy_and_special_values():
    assert oracle.expn(0.0) == 1.0
    for x in np.linspace(-1, 0, 2001):
        assert abs(oracle.expn(x) / math.exp(np.float32(x)) - 1) < 3e-7
    for x in np.linspace(-8, -1, 4001):
        assert abs(oracle.expn(x) / math.exp(np.float32(x)) - 1) < 1e-6
    for x in np.linspace(-80, -8, 2001):
        assert abs(oracle.expn(x) / math.exp(np.float32(x)) - 1) < 5e-6
    assert oracle.expn(-200.0) == 0.0 and oracle.expn(-1e30) == 0.0
    assert oracle.expn(3.0) == 1.0 and oracle.expn(float("nan")) == 1.0   # callers pass x <= 0
    xs = np.linspace(-30, 0, 3001)
    vals = [oracle.expn(x) for x in xs]
    assert all(b >= a for a, b in zip(vals, vals[1:]))                    # monotone on a grid


def test_frequencies_over_all_uniform_values_match_softmax():
    """Sweeping the 24-bit uniform number over a fine grid, the share of each
    action equals its softmax probability."""
    rng = np.random.Generator(np.random.PCG64(3))
    words = (np.arange(0, 1 << 24, 64, dtype=np.uint64) << 8).astype(np.uint32)   # 262144 values
    for logits in ([0.0, 0.0, 0.0], [1.0, 2.0, 3.0], [-4.0, 0.5, 0.25], [10.0, -10.0, 9.0],
                   list(rng.normal(0, 3, 3))):
        l = np.tile(np.array(logits, dtype=np.float32), (len(words), 1))
        a = oracle.sample_actions(l, words)
        z = np.exp(np.array(logits, dtype=np.float64) - max(logits))
        p = z / z.sum()
        freq = np.bincount(a, minlength=3) / len(words)
        assert np.abs(freq - p).max() < 2e-5, (logits, freq, p)
        # inverse CDF: the action is non-decreasing in the uniform number
        assert (np.diff(a.astype(np.int8)) >= 0).all()


def test_extreme_and_shifted_logits():
    words = np.array([0, 1 << 8, 0x7FFFFFFF, 0xFFFFFFFF, 0x80000000], dtype=np.uint32)
    for k in range(3):
        l = np.full((len(words), 3), -1000.0, dtype=np.float32)
        l[:, k] = 0.0
        assert (oracle.sample_actions(l, words) == k).all()
    # word = 0 always picks the first action with non-zero probability
    assert oracle.sample_actions([[0.0, 0.0, 0.0]], [0])[0] == 0
    assert oracle.sample_actions([[-1000.0, 0.0, 0.0]], [0])[0] == 1
    assert oracle.sample_actions([[0.0, 0.0, 0.0]], [0xFFFFFFFF])[0] == 2
    # only the top 24 bits of the word are used
    l = np.tile(np.array([[0.3, -0.2, 0.1]], dtype=np.float32), (4, 1))
    w = np.array([0x12345600, 0x123456FF, 0xABCDEF00, 0xABCDEF7F], dtype=np.uint32)
    a = oracle.sample_actions(l, w)
    assert a[0] == a[1] and a[2] == a[3]
    # adding the same power-of-two constant to all logits changes nothing (l - max is exact)
    rng = np.random.Generator(np.random.PCG64(9))
    l = rng.normal(0, 2, (5000, 3)).astype(np.float32)
    w = rng.integers(0, 1 << 32, 5000, dtype=np.uint64).astype(np.uint32)
    lq = np.round(l * 16) / 16
    assert np.array_equal(oracle.sample_actions(lq, w), oracle.sample_actions(lq + 64.0, w))


def test_fill_words_is_the_action_word_stream():
    o = oracle.OraclePong(6, 77, env_id_base=10)
    o.rollout(5, 0)
    w = o.fill_words(9)
    for t in range(9):
        for i in range(6):
            assert w[t, i] == oracle.action_word(77, 10 + i, 5 + t)
    acts = o.fill_actions(9, 1)
    assert np.array_equal(acts & 3, [[oracle.action_uniform(int(x)) for x in row] for row in w])
