"""Pins for the oracle's Philox4x32-10 and for the draws built on it.

The generator is pinned three ways that do not depend on the oracle's own
code: the published known answers, a second implementation on Python's
unbounded integers written in a different form (with the round keys
precomputed), and the inverse round function, which must recover the counter.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def py_philox(ctr, key, rounds=10):
    """Second implementation: keys of all rounds first, then the rounds."""
    keys = [((key[0] + r * W0) & MASK, (key[1] + r * W1) & MASK) for r in range(rounds)]
    c = list(ctr)
    for k0, k1 in keys:
        p0, p1 = M0 * c[0], M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k0, p1 & MASK, (p0 >> 32) ^ c[3] ^ k1, p0 & MASK]
    return c


def py_philox_inverse(out, key, rounds=10):
    """Undo the rounds: the multipliers are odd, hence invertible mod 2^32."""
    inv0, inv1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    c = list(out)
    for r in reversed(range(rounds)):
        k0, k1 = (key[0] + r * W0) & MASK, (key[1] + r * W1) & MASK
        c0 = (c[3] * inv0) & MASK           # lo(M0*c0) = c[3]
        c2 = (c[1] * inv1) & MASK           # lo(M1*c2) = c[1]
        c1 = c[0] ^ ((M1 * c2) >> 32) ^ k0
        c3 = c[2] ^ ((M0 * c0) >> 32) ^ k1
        c = [c0, c1, c2, c3]
    return c


def read_kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(x, 16) for x in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_known_answers():
    rows = read_kat()
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert oracle.philox4x32_10(ctr, key) == want
        assert py_philox(ctr, key) == want


def test_against_second_implementation_and_inverse():
    rng = np.random.Generator(np.random.PCG64(7))
    for _ in range(300):
        ctr = [int(x) for x in rng.integers(0, 1 << 32, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 1 << 32, 2, dtype=np.uint64)]
        out = oracle.philox4x32_10(ctr, key)
        assert out == py_philox(ctr, key)
        assert py_philox_inverse(out, key) == ctr


def test_single_bit_of_counter_or_key_changes_output():
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    for w in range(4):
        c = [1, 2, 3, 4]
        c[w] ^= 1
        assert oracle.philox4x32_10(c, [5, 6]) != base
    assert oracle.philox4x32_10([1, 2, 3, 4], [4, 6]) != base
    assert oracle.philox4x32_10([1, 2, 3, 4], [5, 7]) != base


def test_action_word_keying():
    """Action word of step t: counter {t/4, env, t>>34, 0}, key = the two
    halves of the seed, output word t%4."""
    seed = 0x0123456789ABCDEF
    key = [seed & MASK, seed >> 32]
    for env in (0, 1, 77, 65535, 1048575):
        for t in (0, 1, 2, 3, 4, 5, 127, 128, 10001, (1 << 34) + 6, (1 << 40) + 3):
            want = py_philox([(t >> 2) & MASK, env, (t >> 34) & MASK, 0], key)[t & 3]
            assert oracle.action_word(seed, env, t) == want


def test_uniform_action_exact_counts():
    """Over all 65,536 values of the low half-word the action takes the values
    0/1/2 exactly 21846/21845/21845 times, whatever the high half-word."""
    counts = [0, 0, 0]
    for u in range(65536):
        counts[oracle.action_uniform(u)] += 1
    assert counts == [21846, 21845, 21845]
    assert oracle.action_uniform(0xFFFF0000) == 0
    assert oracle.action_uniform(0x1234FFFF) == 2
    assert oracle.action_uniform(21845) == 0 and oracle.action_uniform(21846) == 1
    assert oracle.action_uniform(43690) == 1 and oracle.action_uniform(43691) == 2


def test_sticky_probability_exactly_one_quarter():
    reps = sum(oracle.action_repeat(s << 16) for s in range(65536))
    assert reps == 16384
    assert oracle.action_repeat(16383 << 16 | 0xFFFF) == 1
    assert oracle.action_repeat(16384 << 16) == 0


def test_spawn_keying_and_ranges():
    """Spawn of (seed, env, episode, point): counter {point, episode, env, 1};
    vx = +-512 from bit 0 of word 0; vy = floor(word1 * 769 / 2^32) - 384."""
    seed = 0xFEDCBA9876543210
    key = [seed & MASK, seed >> 32]
    seen_vx, vys = set(), []
    for env in (0, 3, 4095):
        for episode in (0, 1, 9):
            for point in (0, 1, 20, 40):
                out = py_philox([point, episode, env, 1], key)
                e = oracle.Env().spawn(seed, env, episode, point)
                assert e.bx == 20224 and e.by == 24320
                assert e.vx == (512 if out[0] & 1 else -512)
                assert e.vy == (out[1] * 769 >> 32) - 384
                seen_vx.add(e.vx)
                vys.append(e.vy)
    assert seen_vx == {-512, 512}
    assert min(vys) >= -384 and max(vys) <= 384
    # the multiply-high map reaches both ends and nothing outside
    assert (0 * 769 >> 32) - 384 == -384 and (MASK * 769 >> 32) - 384 == 384


def test_spawn_vy_roughly_uniform():
    """Loose check only (a tight distribution test would be sample-size
    sensitive): the mean of 769 equally likely values in [-384, 384] is 0."""
    vys = [oracle.Env().spawn(11, env, 0, 0).vy for env in range(4000)]
    assert abs(np.mean(vys)) < 20
    assert len(set(vys)) > 700


def test_reset_is_pure_function_of_counters():
    a = oracle.Env().reset(5, 17, 3).as_dict()
    b = oracle.Env(bx=1, by=2, vx=3, vy=4, apy=5, opy=6, score_a=7, score_o=8,
                   ep_len=9, episode=10, prev_action=2).reset(5, 17, 3).as_dict()
    assert a == b
    assert a["apy"] == 22528 and a["opy"] == 22528
    assert a["score_a"] == 0 and a["score_o"] == 0 and a["ep_len"] == 0
    assert a["prev_action"] == 0 and a["episode"] == 3
    out = py_philox([0, 3, 17, 1], [5, 0])
    assert a["vx"] == (512 if out[0] & 1 else -512)
    assert a["vy"] == (out[1] * 769 >> 32) - 384
