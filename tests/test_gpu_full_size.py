"""Parity at the full benchmark sizes, in the launch configuration the
benchmark times.  The oracle cannot run a million envs in seconds, but an
env's trajectory depends only on its global id, so contiguous sample ranges
are recomputed by the oracle (with env_id_base) and compared bit for bit;
whole-batch properties are checked on top."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import pong

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t
    assert t.cuda.is_available()
    pong.load(build_if_missing=True)
    return t


def sample_ranges(n, width, count, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    starts = {0, n - width}
    while len(starts) < count:
        starts.add(int(rng.integers(0, n - width)))
    return sorted(starts)


def test_vector_rollout_65536_envs_T128(torch):
    n, T, seed, launches = 65536, 128, 0, 6
    env = pong.PongEnv(n, seed)
    starts = sample_ranges(n, 48, 10, 1)
    oras = [oracle.OraclePong(48, seed, env_id_base=s) for s in starts]
    obs = torch.empty((T, n, 6), dtype=torch.float32, device="cuda")
    reward = torch.empty((T, n), dtype=torch.float32, device="cuda")
    done = torch.empty((T, n), dtype=torch.uint8, device="cuda")
    total_done = 0
    total_reward = 0
    for k in range(launches):
        env.rollout(T, pong.ACT_PHILOX, None, obs, reward, done)
        for s, o in zip(starts, oras):
            oo, orw, od = o.rollout(T, 0)
            assert obs[:, s:s + 48].cpu().numpy().tobytes() == oo.tobytes(), (k, s)
            assert reward[:, s:s + 48].cpu().numpy().tobytes() == orw.tobytes(), (k, s)
            assert done[:, s:s + 48].cpu().numpy().tobytes() == od.tobytes(), (k, s)
        total_done += int(done.sum().item())
        total_reward += int(reward.sum(dtype=torch.float64).item())
        # whole-batch properties
        assert bool((done <= 1).all())
        assert bool(((reward == 0) | (reward == 1) | (reward == -1)).all())
        assert bool((obs[..., 0] >= 0).all()) and bool((obs[..., 0] <= 1).all())
        assert bool((obs[..., 1] >= 0).all()) and bool((obs[..., 1] <= 48640 / 40960).all())
        assert bool((obs[..., 4:] >= 0).all()) and bool((obs[..., 4:] <= 1.1).all())
    state, t = env.get_state()
    assert t == launches * T
    ep, ret, length = env.episode_stats()
    assert ep == total_done == int(state[9].sum())
    # sum of rewards = finished returns + points of the running episodes
    assert total_reward == ret + int((state[6] - state[7]).sum())
    for s, o in zip(starts, oras):
        assert state[:, s:s + 48].tobytes() == o.get_state()[0].tobytes()


def test_sticky_rollout_million_envs_T32(torch):
    n, T, seed, launches = 1048576, 32, 0, 4
    env = pong.PongEnv(n, seed)
    st0, _ = env.get_state()
    # bring a band of envs close to the episode end so that auto-resets and the
    # statistics reduction are exercised inside the few launches
    st0[6, ::7] = 20
    st0[8, ::5] = 9990
    env.set_state(st0, 0)
    starts = sample_ranges(n, 40, 12, 2)
    oras = []
    for s in starts:
        o = oracle.OraclePong(40, seed, env_id_base=s)
        o.set_state(st0[:, s:s + 40], 0)
        oras.append(o)
    obs = torch.empty((T, n, 6), dtype=torch.float32, device="cuda")
    reward = torch.empty((T, n), dtype=torch.float32, device="cuda")
    done = torch.empty((T, n), dtype=torch.uint8, device="cuda")
    total_done = 0
    for k in range(launches):
        env.rollout(T, pong.ACT_STICKY, None, obs, reward, done)
        for s, o in zip(starts, oras):
            oo, orw, od = o.rollout(T, 1)
            assert obs[:, s:s + 40].cpu().numpy().tobytes() == oo.tobytes(), (k, s)
            assert reward[:, s:s + 40].cpu().numpy().tobytes() == orw.tobytes(), (k, s)
            assert done[:, s:s + 40].cpu().numpy().tobytes() == od.tobytes(), (k, s)
        total_done += int(done.sum().item())
    state, t = env.get_state()
    ep, ret, length = env.episode_stats()
    assert ep == total_done and ep > n // 6
    assert ep == int((state[9] - st0[9]).sum())
    for s, o in zip(starts, oras):
        assert state[:, s:s + 40].tobytes() == o.get_state()[0].tobytes()
    part = [o.episode_stats() for o in oras]
    assert all(p[0] > 0 for p in part)


def test_step_api_4096_envs(torch):
    n, seed, T = 4096, 0, 600
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    acts = env.fill_actions(T, 0)
    acts_h = acts.cpu().numpy()
    assert acts_h.tobytes() == ora.fill_actions(T, 0).tobytes()
    obs = torch.empty((n, 6), dtype=torch.float32, device="cuda")
    reward = torch.empty((n,), dtype=torch.float32, device="cuda")
    done = torch.empty((n,), dtype=torch.uint8, device="cuda")
    for t in range(T):
        env.step(acts[t], obs, reward, done)
        if t % 50 == 49 or t < 3:
            oo, orw, od = ora.step(acts_h[t])
            assert obs.cpu().numpy().tobytes() == oo.tobytes(), t
            assert reward.cpu().numpy().tobytes() == orw.tobytes(), t
            assert done.cpu().numpy().tobytes() == od.tobytes(), t
        else:
            ora.step(acts_h[t])
    assert env.get_state()[0].tobytes() == ora.get_state()[0].tobytes()


def test_pixel_rollout_16384_envs_T64(torch):
    n, T, seed, launches = 16384, 64, 0, 2
    env = pong.PongEnv(n, seed, obs_mode=pong.OBS_PIXELS, frameskip=4)
    starts = sample_ranges(n, 24, 8, 3)
    oras = [oracle.OraclePong(24, seed, obs_mode=1, frameskip=4, env_id_base=s) for s in starts]
    reward = torch.empty((T, n), dtype=torch.float32, device="cuda")
    done = torch.empty((T, n), dtype=torch.uint8, device="cuda")
    for k in range(launches):
        env.rollout(T, pong.ACT_PHILOX, None, env.ring, reward, done)
        for s, o in zip(starts, oras):
            oring, orw, od = o.rollout(T, 0)
            assert env.ring[s:s + 24].cpu().numpy().tobytes() == oring.tobytes(), (k, s)
            assert reward[:, s:s + 24].cpu().numpy().tobytes() == orw.tobytes(), (k, s)
            assert done[:, s:s + 24].cpu().numpy().tobytes() == od.tobytes(), (k, s)
        # every frame: only 0 / 255; a paddle lights 7 rows of its two columns
        # (a missed ball passing behind it can add at most one row pair)
        ring = env.ring
        assert bool(((ring == 0) | (ring == 255)).all())
        for col in (78, 5):
            rows = (ring[:, :, :, col] == 255).sum(dim=2)
            assert int(rows.min()) == 7 and int(rows.max()) <= 8
        lit = (ring == 255).sum(dim=(2, 3))
        assert int(lit.min()) >= 28 - 4 and int(lit.max()) <= 28 + 4
    state, t = env.get_state()
    assert t == launches * T
    for s, o in zip(starts, oras):
        assert state[:, s:s + 24].tobytes() == o.get_state()[0].tobytes()


@pytest.mark.parametrize("mode", [0, 1])
def test_both_event_paths_of_the_tensor_store_kernel(torch, mode):
    """The tensor-store rollout has two forms of its score / episode-end path and picks by
    grid size (up to 1.75 waves of resident blocks: spawns from the per-lane queue; above:
    one Philox block per event).  Every env is compared with the oracle in both: 131,072 envs
    take the second form, and the same envs run as two handles of 65,536 take the first."""
    from paper_2603_12145_b200.inputs import random_states
    n, seed = 131072, 21
    st = random_states(n, seed=3, near_end=True)
    ora = oracle.OraclePong(n, seed)
    ora.set_state(st, 40)
    expect = [ora.rollout(T, mode) for T in (16, 24)]
    whole = pong.PongEnv(n, seed)
    whole.set_state(st, 40)
    halves = [pong.PongEnv(n // 2, seed, env_id_base=k * (n // 2)) for k in range(2)]
    for k, hv in enumerate(halves):
        hv.set_state(np.ascontiguousarray(st[:, k * (n // 2):(k + 1) * (n // 2)]), 40)
    for (eo, er, ed), T in zip(expect, (16, 24)):
        go, gr, gd = whole.rollout(T, mode)
        assert go.cpu().numpy().tobytes() == eo.tobytes()
        assert gr.cpu().numpy().tobytes() == er.tobytes()
        assert gd.cpu().numpy().tobytes() == ed.tobytes()
        for k, hv in enumerate(halves):
            sl = slice(k * (n // 2), (k + 1) * (n // 2))
            ho, hr, hd = hv.rollout(T, mode)
            assert ho.cpu().numpy().tobytes() == np.ascontiguousarray(eo[:, sl]).tobytes()
            assert hr.cpu().numpy().tobytes() == np.ascontiguousarray(er[:, sl]).tobytes()
            assert hd.cpu().numpy().tobytes() == np.ascontiguousarray(ed[:, sl]).tobytes()
    assert int(sum(e[2].sum() for e in expect)) > n // 4          # many episodes ended
    os_, ot = ora.get_state()
    gs, gt = whole.get_state()
    assert gt == ot and gs.tobytes() == os_.tobytes()
    assert whole.episode_stats() == ora.episode_stats()
    assert tuple(sum(v) for v in zip(*(hv.episode_stats() for hv in halves))) == ora.episode_stats()
