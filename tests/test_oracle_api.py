"""Composition properties of the oracle's batch surface: a rollout is a
sequence of steps, Philox modes equal the explicit mode fed with filled
actions, a restored state continues identically, and an env's trajectory does
not depend on the batch it sits in."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200.inputs import explicit_actions


@pytest.mark.parametrize("sticky", [0, 1])
def test_philox_modes_equal_explicit_mode_with_filled_actions(sticky):
    n, T, seed = 9, 400, 17
    a = oracle.OraclePong(n, seed)
    b = oracle.OraclePong(n, seed)
    for chunk in (3, 128, 1, 268):
        acts = b.fill_actions(chunk, sticky)
        assert set(np.unique(acts)) <= ({0, 1, 2, 4, 5, 6} if sticky else {0, 1, 2})
        oa = a.rollout(chunk, 1 if sticky else 0)
        ob = b.rollout(chunk, 2, acts)
        for x, y in zip(oa, ob):
            assert np.array_equal(x.view(np.uint8), y.view(np.uint8))
    assert np.array_equal(a.get_state()[0], b.get_state()[0])
    assert a.t == b.t == 400


def test_sticky_repeats_previous_action():
    n, T, seed = 64, 200, 5
    o = oracle.OraclePong(n, seed)
    acts = o.fill_actions(T, 1)
    frac = float((acts & 4).astype(bool).mean())
    assert 0.2 < frac < 0.3
    prev = np.zeros(n, dtype=np.int64)
    for t in range(T):
        o.rollout(1, 1)
        s, _ = o.get_state()
        want = np.where(acts[t] & 4, prev, acts[t] & 3)
        assert np.array_equal(s[10], want)
        prev = s[10].astype(np.int64)


def test_rollout_equals_repeated_step():
    n, T, seed = 6, 150, 8
    acts = explicit_actions(T, n, seed=9, repeat_fraction=0.2, odd_codes=True)
    a = oracle.OraclePong(n, seed)
    b = oracle.OraclePong(n, seed)
    obs, reward, done = a.rollout(T, 2, acts)
    for t in range(T):
        o1, r1, d1 = b.step(acts[t])
        assert np.array_equal(o1.view(np.uint32), obs[t].view(np.uint32))
        assert np.array_equal(r1, reward[t]) and np.array_equal(d1, done[t])
    assert np.array_equal(a.get_state()[0], b.get_state()[0])


def test_action_byte_decoding():
    assert [oracle.decode_action(b, 2) for b in range(8)] == [0, 1, 2, 0, 2, 2, 2, 2]
    assert [oracle.decode_action(b, 1) for b in (4, 7)] == [1, 1]


def test_save_restore_continues_identically():
    n, seed = 16, 99
    a = oracle.OraclePong(n, seed)
    a.rollout(777, 1)
    state, t = a.get_state()
    b = oracle.OraclePong(n, seed)
    b.set_state(state, t)
    ra = a.rollout(300, 1)
    rb = b.rollout(300, 1)
    for x, y in zip(ra, rb):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8))


def test_env_trajectory_independent_of_batch_partition():
    seed, T = 123, 600
    whole = oracle.OraclePong(32, seed)
    ow = whole.rollout(T, 1)
    lo = oracle.OraclePong(20, seed, env_id_base=0)
    hi = oracle.OraclePong(12, seed, env_id_base=20)
    ol, oh = lo.rollout(T, 1), hi.rollout(T, 1)
    for w, l, h in zip(ow, ol, oh):
        assert np.array_equal(w[:, :20], l) and np.array_equal(w[:, 20:], h)
    sw, sl, sh = whole.episode_stats(), lo.episode_stats(), hi.episode_stats()
    assert sw == tuple(x + y for x, y in zip(sl, sh))


def test_constant_action_mode_and_stats_clear():
    n, seed = 4, 2
    a = oracle.OraclePong(n, seed)
    b = oracle.OraclePong(n, seed)
    oa = a.rollout(12000, 3, 2)
    ob = b.rollout(12000, 2, np.full((12000, n), 2, dtype=np.uint8))
    for x, y in zip(oa, ob):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8))
    ep, ret, length = a.episode_stats(clear=True)
    assert ep >= n and ep == int(oa[2].sum())
    assert ret == int(oa[1].sum()) - sum(
        int(s) for s in (a.get_state()[0][6] - a.get_state()[0][7]))
    assert a.episode_stats() == (0, 0, 0)
