"""GPU parity of the CartPole library against its CPU oracle, through the C ABI.
Both sides compute in binary32 with the same operation order, so obs, reward,
done, state and statistics are compared bit for bit (0 ULP)."""
import numpy as np
import pytest

from oracle import cartpole as ocp
from paper_2603_12145_b200 import cartpole as cp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t
    assert t.cuda.is_available()
    cp.load(build_if_missing=True)
    return t


def cpu(x):
    return x.cpu().numpy()


def assert_equal(g, o, what=""):
    for name, a, b in zip(("obs", "reward", "done"), g, o):
        a = cpu(a)
        assert a.shape == b.shape and a.tobytes() == b.tobytes(), "%s %s differs" % (what, name)


def assert_state_equal(env, ora):
    gf, gi, gt = env.get_state()
    of, oi, ot = ora.get_state()
    assert gt == ot and gf.tobytes() == of.tobytes() and gi.tobytes() == oi.tobytes()
    assert env.episode_stats() == ora.episode_stats()


def actions(T, n, seed):
    return np.random.Generator(np.random.PCG64(seed)).integers(0, 2, (T, n), dtype=np.uint8)


@pytest.mark.parametrize("n", [1, 31, 128, 1000])
@pytest.mark.parametrize("mode", [0, 2, 3])
def test_rollout_every_mode_and_ragged_sizes(torch, n, mode):
    seed = 40 + n
    env, ora = cp.CartPoleEnv(n, seed), ocp.OracleCartPole(n, seed)
    assert cpu(env.reset()).tobytes() == ora.reset().tobytes()
    for k, T in enumerate((1, 2, 3, 5, 128, 64, 7, 501)):
        if mode == 2:
            a = actions(T, n, k) | (np.uint8(2) * (k % 2))      # upper bits are ignored
            g, o = env.rollout(T, 2, torch.from_numpy(a).cuda()), ora.rollout(T, 2, a)
        elif mode == 3:
            g, o = env.rollout(T, 3, k % 2), ora.rollout(T, 3, k % 2)
        else:
            g, o = env.rollout(T, 0), ora.rollout(T, 0)
        assert_equal(g, o, "n %d mode %d T %d" % (n, mode, T))
    assert_state_equal(env, ora)
    assert ora.episode_stats()[0] > 0


@pytest.mark.parametrize("n", [16, 48, 64, 1040, 4096])
@pytest.mark.parametrize("mode", [0, 2, 3])
def test_aligned_sizes_and_long_rollouts(torch, n, mode):
    """Batch sizes that are multiples of 16 with step counts that are and are not
    multiples of 4, long enough for several refills of the start-state table."""
    seed = 900 + n
    env, ora = cp.CartPoleEnv(n, seed), ocp.OracleCartPole(n, seed)
    for k, T in enumerate((8, 64, 16, 128, 200, 3, 8, 1, 24, 40, 512)):
        if mode == 2:
            a = actions(T, n, 50 + k)
            g, o = env.rollout(T, 2, torch.from_numpy(a).cuda()), ora.rollout(T, 2, a)
        elif mode == 3:
            g, o = env.rollout(T, 3, k % 2), ora.rollout(T, 3, k % 2)
        else:
            g, o = env.rollout(T, 0), ora.rollout(T, 0)
        assert_equal(g, o, "n %d mode %d T %d" % (n, mode, T))
    assert_state_equal(env, ora)
    assert ora.episode_stats()[0] > n


def test_step_api_and_composition(torch):
    n, seed, T = 257, 6, 200
    env, ora = cp.CartPoleEnv(n, seed), ocp.OracleCartPole(n, seed)
    a = actions(T, n, 1)
    da = torch.from_numpy(a).cuda()
    for t in range(T):
        assert_equal(env.step(da[t]), ora.step(a[t]), "t %d" % t)
    assert_state_equal(env, ora)
    # rollout == repeated step
    b = cp.CartPoleEnv(n, seed)
    obs, reward, done = b.rollout(T, 2, da)
    c = cp.CartPoleEnv(n, seed)
    for t in range(T):
        o1, r1, d1 = c.step(da[t])
        assert cpu(o1).tobytes() == cpu(obs[t]).tobytes() and cpu(d1).tobytes() == cpu(done[t]).tobytes()


def test_step_limit_truncation_with_balancing_actions(torch):
    """A bang-bang controller keeps the pole up long enough to reach 500 steps."""
    n, seed = 64, 9
    env, ora = cp.CartPoleEnv(n, seed), ocp.OracleCartPole(n, seed)
    obs = ora.reset()
    env.reset()
    lengths_before = ora.episode_stats()
    for t in range(1100):
        a = ((obs[:, 2] + 0.5 * obs[:, 3] + 0.02 * obs[:, 0] + 0.1 * obs[:, 1]) > 0).astype(np.uint8)
        g = env.step(torch.from_numpy(a).cuda())
        o = ora.step(a)
        assert_equal(g, o, "t %d" % t)
        obs = o[0]
    ep, total = ora.episode_stats()
    assert ep >= n and total // ep >= 400          # most episodes ran into the 500-step limit
    assert_state_equal(env, ora)


def test_extreme_in_play_states_divide_exactly(torch):
    """The kernel forms x / 1.1 by a multiply and two fused steps, which equals the division the
    oracle performs except for |x| <= 3.39e-32 and -0.  States at the edges of what set_state
    accepts (zero, signed-zero, subnormal and tiny angles, velocities up to +-1000, and angular
    velocities chosen so that force + 0.05 thd^2 sin(th) cancels to zero or to one ulp) must
    still agree with the oracle bit for bit."""
    th_vals = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-38, -1e-38, 1e-30, 3e-20, -3e-20, 1e-7, -1e-7,
                        0.05, -0.05, 0.2094, -0.2094, 0.20943951], np.float32)
    thd_vals = np.array([0.0, -0.0, 1e-38, 1e-20, -1e-20, 1.0, -1.0, 30.9, -30.9, 63.2, 100.0, -100.0,
                         999.0, -999.0, 1000.0, -1000.0], np.float32)
    th, thd = np.meshgrid(th_vals, thd_vals, indexing="ij")
    th, thd = th.ravel(), thd.ravel()
    # rows where t3 = 0.05 thd^2 sin(th) lands on -+10 exactly or within a few ulps: solve for thd
    extra_th = np.array([0.2, -0.2, 0.1, -0.1, 0.01, -0.01] * 40, np.float32)
    target = np.float32(10.0)
    base = np.sqrt(np.float64(target) / (0.05 * np.abs(np.sin(np.float64(extra_th))))).astype(np.float32)
    extra_thd = base.view(np.uint32) + np.tile(np.arange(-20, 20, dtype=np.int64).repeat(6), 1)[:len(base)]
    extra_thd = extra_thd.astype(np.uint32).view(np.float32)
    th = np.concatenate([th, extra_th])
    thd = np.concatenate([thd, extra_thd])
    keep = np.abs(thd) <= 1000.0
    th, thd = th[keep], thd[keep]
    n = len(th)
    rng = np.random.Generator(np.random.PCG64(8))
    f = np.stack([rng.uniform(-2.3, 2.3, n).astype(np.float32), rng.uniform(-50, 50, n).astype(np.float32),
                  th, thd])
    i = np.zeros((2, n), np.int32)
    for action in (0, 1):
        env, ora = cp.CartPoleEnv(n, 3), ocp.OracleCartPole(n, 3)
        env.set_state(f, i, 0)
        ora.set_state(f, i, 0)
        for t in range(3):
            g = env.rollout(1, cp.ACT_CONSTANT, action)
            o = ora.rollout(1, 3, action)
            assert_equal(g, o, "extreme states, action %d step %d" % (action, t))
        assert_state_equal(env, ora)
    # states outside the accepted range are refused
    for k, v in ((0, 2.5), (1, 1001.0), (2, 0.21), (3, -1000.5), (3, np.inf)):
        bad = f.copy(); bad[k, 0] = v
        with pytest.raises(cp.CartPoleError) as ei:
            env.set_state(bad, i, 0)
        assert ei.value.code == -1


def test_state_roundtrip_restore_partition_and_errors(torch):
    seed = 5
    whole = cp.CartPoleEnv(96, seed)
    lo, hi = cp.CartPoleEnv(50, seed, env_id_base=0), cp.CartPoleEnv(46, seed, env_id_base=50)
    gw, gl, gh = whole.rollout(300), lo.rollout(300), hi.rollout(300)
    for w, l, h in zip(gw, gl, gh):
        assert cpu(w[:, :50]).tobytes() == cpu(l).tobytes() and cpu(w[:, 50:]).tobytes() == cpu(h).tobytes()
    assert whole.episode_stats() == tuple(x + y for x, y in zip(lo.episode_stats(), hi.episode_stats()))
    f, i, t = whole.get_state()
    again = cp.CartPoleEnv(96, seed)
    again.set_state(f, i, t)
    for x, y in zip(whole.rollout(100), again.rollout(100)):
        assert cpu(x).tobytes() == cpu(y).tobytes()
    bad = f.copy(); bad[2, 3] = np.nan
    with pytest.raises(cp.CartPoleError) as ei:
        again.set_state(bad, i, 0)
    assert ei.value.code == -1
    badi = i.copy(); badi[0, 0] = 500
    with pytest.raises(cp.CartPoleError):
        again.set_state(f, badi, 0)
    obs = torch.empty((4, 96, 4), dtype=torch.float32, device="cuda")
    rew = torch.empty((4, 96), dtype=torch.float32, device="cuda")
    dn = torch.empty((4, 96), dtype=torch.uint8, device="cuda")
    for args, code in (((0, 0, None, obs, rew, dn), -1), ((4, 1, None, obs, rew, dn), -5),
                       ((4, 2, None, obs, rew, dn), -2), ((4, 0, None, None, rew, dn), -2),
                       ((4, 0, None, obs.data_ptr() + 4, rew, dn), -3)):
        with pytest.raises(cp.CartPoleError) as ei:
            cp.cartpole_rollout(again.h, *args)
        assert ei.value.code == code


def test_host_buffer_rollout(torch):
    n, T, seed = 300, 64, 3
    a, b = cp.CartPoleEnv(n, seed), cp.CartPoleEnv(n, seed)
    obs_h = torch.empty((T, n, 4), dtype=torch.float32).pin_memory()
    rew_h = torch.empty((T, n), dtype=torch.float32).pin_memory()
    done_h = torch.empty((T, n), dtype=torch.uint8).pin_memory()
    b._stream()
    cp.cartpole_rollout_host(b.h, T, 0, None, obs_h, rew_h, done_h)
    g = a.rollout(T, 0)
    assert cpu(g[0]).tobytes() == obs_h.numpy().tobytes() and cpu(g[2]).tobytes() == done_h.numpy().tobytes()
    assert bool((rew_h == 1.0).all())


def test_full_size_sampled(torch):
    """N = 1,048,576, T = 32: contiguous sample ranges recomputed by the oracle."""
    n, T, seed = 1 << 20, 32, 0
    env = cp.CartPoleEnv(n, seed)
    rng = np.random.Generator(np.random.PCG64(4))
    starts = sorted({0, n - 40} | {int(rng.integers(0, n - 40)) for _ in range(8)})
    oras = [ocp.OracleCartPole(40, seed, env_id_base=s) for s in starts]
    obs = torch.empty((T, n, 4), dtype=torch.float32, device="cuda")
    reward = torch.empty((T, n), dtype=torch.float32, device="cuda")
    done = torch.empty((T, n), dtype=torch.uint8, device="cuda")
    total_done = 0
    for k in range(4):
        env.rollout(T, 0, None, obs, reward, done)
        for s, o in zip(starts, oras):
            oo, orw, od = o.rollout(T, 0)
            assert cpu(obs[:, s:s + 40]).tobytes() == oo.tobytes(), (k, s)
            assert cpu(done[:, s:s + 40]).tobytes() == od.tobytes(), (k, s)
        total_done += int(done.sum().item())
        assert bool((reward == 1.0).all()) and bool((done <= 1).all())
    ep, length = env.episode_stats()
    assert ep == total_done > n and 15 < length / ep < 30


@pytest.mark.parametrize("n,T,mode", [
    (1, 4, 0), (40, 64, 0), (1000, 128, 2), (4097, 36, 3),
    (26048, 100, 0), (26033, 64, 2), (33152, 68, 0), (45056, 128, 0),
    (61568, 32, 0), (65536, 128, 0), (65536, 36, 2), (66304, 160, 3), (66290, 96, 0),
])
def test_chains_path_matches_the_oracle(torch, n, T, mode):
    """The balanced-chains kernel with the path forced, element by element: one chain per block,
    4 + 1 / 4 + 2 chains (leftovers alternating between two warps every 32 steps), 4 + 3 (whole
    leftovers), 8 + 1 / 8 + 2, 12 + 1 / 12 + 2, the largest batch, ragged last chains; rollouts of
    one span, whole spans and a short last span.  CartPole episodes end every ~22 steps, so every
    span crosses resets."""
    seed = 300 + n % 89
    env, ora = cp.CartPoleEnv(n, seed, env_id_base=11), ocp.OracleCartPole(n, seed, env_id_base=11)
    env.set_path(cp.PATH_CHAINS)
    for rep in range(2):
        if mode == 2:
            a = actions(T, n, rep)
            g, o = env.rollout(T, 2, torch.from_numpy(a).cuda()), ora.rollout(T, 2, a)
        elif mode == 3:
            g, o = env.rollout(T, 3, rep), ora.rollout(T, 3, rep)
        else:
            g, o = env.rollout(T, 0), ora.rollout(T, 0)
        assert_equal(g, o, "chains n %d T %d mode %d launch %d" % (n, T, mode, rep))
    # an unaligned call falls back to the plain kernel, and the chains kernel picks up again after it
    g, o = env.rollout(3, 0), ora.rollout(3, 0)
    assert_equal(g, o, "unaligned")
    g, o = env.rollout(1, 0), ora.rollout(1, 0)
    assert_equal(g, o, "realign")
    g, o = env.rollout(64, 0), ora.rollout(64, 0)
    assert_equal(g, o, "chains again")
    assert_state_equal(env, ora)
    with pytest.raises(cp.CartPoleError):
        env.set_path(5)
