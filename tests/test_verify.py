"""The rollout-comparison harness and the equivalence test, on CPU: the oracle
against itself, against doubles with a planted fault, and the statistics
against scipy."""
import numpy as np
import pytest
from scipy import stats

import oracle
from paper_2603_12145_b200 import verify
from paper_2603_12145_b200.inputs import explicit_actions


class Faulty:
    """The oracle with one planted mistake: from global step `at` on, env `env`
    reports a wrong value in one output component."""

    def __init__(self, n, seed, at, env, component):
        self.o = oracle.OraclePong(n, seed)
        self.at, self.env, self.component = at, env, component

    def rollout(self, T, mode=0, actions=None):
        t0 = self.o.t
        obs, reward, done = self.o.rollout(T, mode, actions)
        for t in range(T):
            if t0 + t >= self.at:
                if self.component == "reward":
                    reward[t, self.env] += 1.0
                elif self.component == "done":
                    done[t, self.env] ^= 1
                else:
                    obs[t, self.env, self.component] = np.nextafter(
                        obs[t, self.env, self.component], np.float32(2.0))
        return obs, reward, done

    def get_state(self):
        return self.o.get_state()

    def set_state(self, s, t):
        self.o.set_state(s, t)

    def episode_stats(self):
        return self.o.episode_stats()


def test_identical_backends_compare_equal_over_many_episodes():
    n, seed = 16, 3
    a, b = oracle.OraclePong(n, seed), oracle.OraclePong(n, seed)
    schedule = [(128, 1)] * 60 + [(7, 0), (1, 0), (500, 2), (64, 3)]
    rep = verify.compare_rollouts(
        a, b, schedule,
        actions_for=lambda ci, T: explicit_actions(T, n, seed=ci) if schedule[ci][1] == 2 else 1)
    assert rep.equal, str(rep)
    assert rep.steps_compared == sum(T for T, _ in schedule)
    assert rep.env_steps_compared == rep.steps_compared * n
    assert rep.episodes_finished == a.episode_stats()[0] >= 40


@pytest.mark.parametrize("component,name", [(3, "obs.ball_vy"), (0, "obs.ball_x"),
                                            ("reward", "reward"), ("done", "done")])
def test_planted_fault_is_located_to_step_env_and_component(component, name):
    n, seed, at, env = 12, 9, 300 + 45, 7
    a = oracle.OraclePong(n, seed)
    b = Faulty(n, seed, at, env, component)
    rep = verify.compare_rollouts(a, b, [(100, 0), (100, 1), (100, 0), (100, 1), (100, 0)])
    assert not rep.equal
    d = rep.divergence
    assert (d.call, d.step, d.env, d.component) == (3, at, env, name)
    assert d.mismatching_elements == 1 and d.value_a != d.value_b
    assert any("single-step replay diverges at step %d, env %d" % (at, env) in s for s in rep.notes)
    assert rep.steps_compared == 300


def test_state_only_fault_is_reported():
    n, seed = 5, 1
    a, b = oracle.OraclePong(n, seed), oracle.OraclePong(n, seed)
    s, t = b.get_state()
    s[4, 2] += 768                      # agent paddle of env 2 somewhere else
    b.set_state(s, t)
    rep = verify.compare_rollouts(a, b, [(10, 0)])
    assert not rep.equal
    assert (rep.divergence.env, rep.divergence.component) == (2, "state.apy")


def test_episode_returns_match_the_episode_statistics():
    n, seed = 24, 4
    o = oracle.OraclePong(n, seed)
    carry, allr = None, []
    for T in (1000, 1, 2500, 37, 3000):
        _, reward, done = o.rollout(T, 1)
        r, carry = verify.episode_returns(reward, done, carry)
        allr.extend(r.tolist())
    ep, ret, _ = o.episode_stats()
    assert len(allr) == ep > 20 and sum(allr) == ret
    state, _ = o.get_state()
    assert np.array_equal(carry, (state[6] - state[7]).astype(np.float64))
    assert all(-21 <= x <= 21 for x in allr)


def test_tost_against_scipy_and_decisions():
    rng = np.random.Generator(np.random.PCG64(0))
    for na, nb, shift, margin in ((10, 10, 0.0, 1.0), (30, 12, 0.4, 1.0), (8, 50, 2.0, 1.0),
                                  (100, 100, 0.05, 0.3)):
        xa = rng.normal(28.0, 0.3, na)
        xb = rng.normal(28.0 + shift, 0.5, nb)
        r = verify.tost_equivalence(xa, xb, margin)
        p_lo = stats.ttest_ind(xa + margin, xb, equal_var=False, alternative="greater").pvalue
        p_hi = stats.ttest_ind(xa - margin, xb, equal_var=False, alternative="less").pvalue
        assert abs(r.p_lower - p_lo) < 1e-9 and abs(r.p_upper - p_hi) < 1e-9
        assert abs(r.p_value - max(p_lo, p_hi)) < 1e-9
        assert r.equivalent == (max(p_lo, p_hi) < 0.05)
    # clear decisions
    same = rng.normal(0.0, 1.0, 200)
    assert verify.tost_equivalence(same, same + 0.01, 0.5).equivalent
    assert not verify.tost_equivalence(same, same + 5.0, 0.5).equivalent
    # constant samples (zero variance): decided by the difference alone
    const = np.full(10, 19.0)
    assert verify.tost_equivalence(const, const, 1.0).equivalent
    assert not verify.tost_equivalence(const, const + 2.0, 1.0).equivalent
    with pytest.raises(ValueError):
        verify.tost_equivalence([1.0], [1.0, 2.0], 1.0)
    with pytest.raises(ValueError):
        verify.tost_equivalence([1.0, 2.0], [1.0, 2.0], 0.0)


def test_tost_on_returns_of_two_identically_seeded_backends():
    n, seed = 32, 8
    returns = []
    for _ in range(2):
        o = oracle.OraclePong(n, seed)
        _, reward, done = o.rollout(6000, 0)
        returns.append(verify.episode_returns(reward, done)[0])
    assert len(returns[0]) >= 60
    r = verify.tost_equivalence(returns[0], returns[1], margin=1.0)
    assert r.equivalent and r.difference == 0.0
