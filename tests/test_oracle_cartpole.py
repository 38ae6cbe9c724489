"""Pins for the CartPole oracle.  Expected values come from the textbook
cart-pole equations evaluated independently (closed forms by hand, a binary64
evaluation with the library sin / cos), from exact symmetries and from the
termination rule; never from the oracle itself."""
import itertools
import math

import numpy as np
import pytest

from oracle import cartpole as cp

TH_LIMIT = 12 * 2 * math.pi / 360


def reference_step64(state, a):
    """The same equations in binary64 with math.sin / math.cos."""
    x, xd, th, thd = state
    force = 10.0 if a else -10.0
    s, c = math.sin(th), math.cos(th)
    temp = (force + 0.05 * thd * thd * s) / 1.1
    thetaacc = (9.8 * s - c * temp) / (0.5 * (4.0 / 3.0 - 0.1 * c * c / 1.1))
    xacc = temp - 0.05 * thetaacc * c / 1.1
    return (x + 0.02 * xd, xd + 0.02 * xacc, th + 0.02 * thd, thd + 0.02 * thetaacc)


def test_first_step_from_rest_closed_form():
    # th = thd = 0: temp = 10/1.1, thetaacc = -temp / (0.5*(4/3 - 0.1/1.1)), xacc = temp - 0.05*thetaacc/1.1
    temp = 10.0 / 1.1
    thetaacc = -temp / (0.5 * (4.0 / 3.0 - 0.1 / 1.1))
    xacc = temp - 0.05 * thetaacc / 1.1
    for a, sign in ((1, 1.0), (0, -1.0)):
        e = cp.Env()
        assert e.step(a) == 0
        x, xd, th, thd = e.state()
        assert x == 0.0 and th == 0.0
        assert abs(xd - sign * 0.02 * xacc) < 2e-8 and abs(thd - sign * 0.02 * thetaacc) < 4e-8
    assert abs(0.02 * xacc - 0.1951219512) < 1e-9 and abs(0.02 * thetaacc + 0.2926829268) < 1e-9


def test_position_and_angle_integrate_the_old_velocities():
    e = cp.Env(x=0.5, xd=1.25, th=0.05, thd=-0.75)
    e.step(1)
    x, xd, th, thd = e.state()
    assert x == np.float32(0.5) + np.float32(0.02) * np.float32(1.25)
    assert th == np.float32(0.05) + np.float32(0.02) * np.float32(-0.75)


def test_polynomial_sine_and_cosine_accuracy():
    for th in np.linspace(-0.45, 0.45, 181):
        assert abs(cp.poly_sin(th) - math.sin(np.float32(th))) < 1.2e-7
        assert abs(cp.poly_cos(th) - math.cos(np.float32(th))) < 1.2e-7
    assert cp.poly_sin(0.0) == 0.0 and cp.poly_cos(0.0) == 1.0
    assert cp.poly_sin(-0.1) == -cp.poly_sin(0.1) and cp.poly_cos(-0.1) == cp.poly_cos(0.1)


def test_mirror_symmetry_is_exact():
    """Negating the state and swapping the action negates the next state bit for bit."""
    rng = np.random.Generator(np.random.PCG64(1))
    for _ in range(300):
        s = rng.uniform(-1, 1, 4) * np.array([2.0, 2.0, 0.2, 2.5])
        a = int(rng.integers(0, 2))
        e1 = cp.Env(*[float(np.float32(v)) for v in s])
        e2 = cp.Env(*[float(-np.float32(v)) for v in s])
        d1, d2 = e1.step(a), e2.step(1 - a)
        if d1 or d2:
            assert d1 == d2
            continue
        assert all(p == -q for p, q in zip(e1.state(), e2.state()))


def test_agrees_with_binary64_reference_over_short_horizons():
    rng = np.random.Generator(np.random.PCG64(2))
    worst = 0.0
    for trial in range(200):
        s = rng.uniform(-0.05, 0.05, 4)
        e = cp.Env(*[float(np.float32(v)) for v in s])
        ref = tuple(float(np.float32(v)) for v in s)
        for t in range(6):        # six steps cannot reach a threshold from a reset state
            a = int(rng.integers(0, 2))
            d = e.step(a)
            ref = reference_step64(ref, a)
            assert d == 0
            worst = max(worst, max(abs(float(p) - q) for p, q in zip(e.state(), ref)))
    assert worst < 5e-6


def test_every_action_sequence_against_binary64_reference():
    start = (0.01, -0.02, 0.03, 0.04)
    for seq in itertools.product((0, 1), repeat=7):
        e = cp.Env(*start)
        ref = tuple(float(np.float32(v)) for v in start)
        for a in seq:
            ref = reference_step64(ref, a)
            done_ref = abs(ref[0]) > 2.4 or abs(ref[2]) > TH_LIMIT
            d = e.step(a)
            if done_ref or d:
                assert d == int(done_ref)
                break
            assert max(abs(float(p) - q) for p, q in zip(e.state(), ref)) < 5e-6


def test_termination_thresholds_and_step_limit():
    lim = np.float32(TH_LIMIT)
    # angle: state lands exactly on the limit -> not done; one ulp beyond -> done
    below = np.nextafter(lim, np.float32(0))
    st = cp.new_stats()
    e = cp.Env(th=float(below), thd=0.0, steps=3, episode=4)
    # a step from rest changes thd but th only by tau*thd_old = 0 -> th stays `below`
    assert e.step(1, seed=5, env_id=6, stats=st) == 0 and e.state()[2] == below
    e = cp.Env(th=float(np.nextafter(lim, np.float32(1))), thd=0.0, steps=3, episode=4)
    assert e.step(1, seed=5, env_id=6, stats=st) == 1
    assert (st.episodes, st.sum_length) == (1, 4)
    assert e.as_tuple() == cp.Env().reset(5, 6, 5).as_tuple()
    e = cp.Env(th=float(-np.nextafter(lim, np.float32(1)))); assert e.step(0) == 1
    e = cp.Env(th=float(lim)); assert e.step(0) == 0             # exactly at the limit
    # position
    e = cp.Env(x=2.4); assert e.step(0) == 0                      # float32(2.4), not beyond
    e = cp.Env(x=float(np.nextafter(np.float32(2.4), np.float32(3)))); assert e.step(0) == 1
    e = cp.Env(x=-float(np.nextafter(np.float32(2.4), np.float32(3)))); assert e.step(1) == 1
    # step limit: the 500th step ends the episode
    st = cp.new_stats()
    e = cp.Env(steps=498, episode=0)
    assert e.step(1, stats=st) == 0 and e.c.steps == 499
    assert e.step(0, seed=1, env_id=2, stats=st) == 1
    assert (st.episodes, st.sum_length) == (1, 500)
    assert e.as_tuple() == cp.Env().reset(1, 2, 1).as_tuple()


def py_philox(ctr, key):
    M0, M1, W0, W1, MASK = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85, 0xFFFFFFFF
    c, k0, k1 = list(ctr), key[0], key[1]
    for _ in range(10):
        p0, p1 = M0 * c[0], M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k0, p1 & MASK, (p0 >> 32) ^ c[3] ^ k1, p0 & MASK]
        k0, k1 = (k0 + W0) & MASK, (k1 + W1) & MASK
    return c


def test_reset_and_action_keying():
    seed = 0x1122334455667788
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for env, ep in ((0, 0), (5, 3), (65535, 77)):
        out = py_philox([0, ep, env, 2], key)
        e = cp.Env(1, 2, 3, 4, 5, 6).reset(seed, env, ep)
        want = [np.float32((np.float32(w >> 8) * np.float32(2.0 ** -24) - np.float32(0.5))
                           * np.float32(0.1)) for w in out]
        assert list(e.state()) == want
        assert all(-0.05 <= float(v) < 0.05 for v in want)
        assert (e.c.steps, e.c.episode) == (0, ep)
    for env in (0, 9):
        for t in (0, 1, 2, 3, 4, 1023, (1 << 34) + 2):
            w = py_philox([(t >> 2) & 0xFFFFFFFF, env, t >> 34, 3], key)[t & 3]
            assert cp.action(seed, env, t) == (w & 1)


def test_batch_rollout_is_the_single_step_applied_to_every_env_and_invariants():
    n, T, seed = 7, 400, 11
    o = cp.OracleCartPole(n, seed, env_id_base=100)
    obs, reward, done = o.rollout(T, 0)
    assert (reward == 1.0).all()
    lengths = []
    for i in range(n):
        e = cp.Env().reset(seed, 100 + i, 0)
        run = 0
        for t in range(T):
            d = e.step(cp.action(seed, 100 + i, t), seed=seed, env_id=100 + i)
            run += 1
            assert d == done[t, i]
            assert tuple(obs[t, i]) == e.state()
            if d:
                lengths.append(run)
                run = 0
                assert all(-0.05 <= float(v) < 0.05 for v in e.state())
            else:
                assert abs(float(e.state()[0])) <= 2.4 and abs(float(e.state()[2])) <= TH_LIMIT + 1e-7
    ep, total = o.episode_stats()
    assert ep == len(lengths) == int(done.sum()) and total == sum(lengths)
    assert 8 <= min(lengths) and 15 < np.mean(lengths) < 32      # random policy: about 22 steps


def test_composition_partition_and_restore():
    seed = 3
    whole = cp.OracleCartPole(20, seed)
    a, b = cp.OracleCartPole(12, seed, 0), cp.OracleCartPole(8, seed, 12)
    ow, oa, ob = whole.rollout(300, 0), a.rollout(300, 0), b.rollout(300, 0)
    for w, p, q in zip(ow, oa, ob):
        assert np.array_equal(w[:, :12], p) and np.array_equal(w[:, 12:], q)
    f, i, t = whole.get_state()
    c = cp.OracleCartPole(20, seed)
    c.set_state(f, i, t)
    for x, y in zip(whole.rollout(100, 0), c.rollout(100, 0)):
        assert x.tobytes() == y.tobytes()
    # explicit actions reproduce the Philox mode; rollout = repeated step
    d = cp.OracleCartPole(6, seed)
    g = cp.OracleCartPole(6, seed)
    acts = np.array([[cp.action(seed, i, t) for i in range(6)] for t in range(50)], dtype=np.uint8)
    od = d.rollout(50, 0)
    for t in range(50):
        o1, r1, d1 = g.step(acts[t])
        assert o1.tobytes() == od[0][t].tobytes() and d1.tobytes() == od[2][t].tobytes()
