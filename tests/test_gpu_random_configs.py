"""GPU parity on seeded random configurations: batch size, seed, first env id,
frameskip, observation mode, start state, start step and a sequence of calls with
random lengths and action modes are all drawn from one generator, so that the
combinations nobody thought of listing get exercised too (aligned and ragged
sizes, fast and general kernels inside one run, episode ends at any phase).
Everything is compared bit for bit with the CPU oracle (0 ULP)."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import pong
from paper_2603_12145_b200.inputs import explicit_actions, random_states

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t
    assert t.cuda.is_available()
    pong.load(build_if_missing=True)
    return t


def same(a, b):
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    return a.shape == b.shape and a.dtype == b.dtype and a.tobytes() == b.tobytes()


def draw_config(case):
    rng = np.random.default_rng(1000 + case)
    pixels = case % 4 == 3
    if pixels:
        n = int(rng.integers(1, 120))
    else:
        n = int(rng.integers(1, 2500))
        if rng.random() < 0.5:
            n = max(16, n // 16 * 16)            # sizes the tensor-store kernel takes
    frameskip = int(rng.choice([1, 1, 1, 2, 3, 4])) if not pixels else int(rng.choice([1, 4, 4]))
    t0 = int(rng.choice([0, 4, 8, 1, 3, 2**32 - 8, 2**34 + 4, 2**40 + 1]))
    calls = []
    for _ in range(int(rng.integers(3, 7))):
        T = int(rng.choice([1, 2, 3, 4, 7, 8, 16, 24, 31, 64, 100, 128]))
        calls.append((T, int(rng.integers(0, 4))))
    return dict(n=n, seed=int(rng.integers(0, 2**63)), base=int(rng.choice([0, 1, 12345, 2**31 - 5000])),
                obs_mode=1 if pixels else 0, frameskip=frameskip, t0=t0, near_end=bool(rng.random() < 0.6),
                calls=calls, state_seed=int(rng.integers(0, 2**31)))


@pytest.mark.parametrize("case", range(24))
def test_random_configuration(torch, case):
    c = draw_config(case)
    n = c["n"]
    env = pong.PongEnv(n, c["seed"], obs_mode=c["obs_mode"], frameskip=c["frameskip"], env_id_base=c["base"])
    ora = oracle.OraclePong(n, c["seed"], obs_mode=c["obs_mode"], frameskip=c["frameskip"],
                            env_id_base=c["base"])
    st = random_states(n, seed=c["state_seed"], near_end=c["near_end"])
    env.set_state(st, c["t0"])
    ora.set_state(st, c["t0"])
    dones = 0
    for k, (T, mode) in enumerate(c["calls"]):
        what = "case %d call %d (n %d, T %d, mode %d, frameskip %d)" % (case, k, n, T, mode, c["frameskip"])
        if mode == 2:
            acts = explicit_actions(T, n, seed=case * 100 + k, repeat_fraction=0.2, odd_codes=True)
            g = env.rollout(T, 2, torch.from_numpy(acts).cuda())
            o = ora.rollout(T, 2, acts)
        elif mode == 3:
            g = env.rollout(T, 3, k % 3)
            o = ora.rollout(T, 3, k % 3)
        else:
            g = env.rollout(T, mode)
            o = ora.rollout(T, mode)
        for name, gv, ov in zip(("obs", "reward", "done"), g, o):
            assert same(gv.cpu().numpy(), ov), "%s: %s differs" % (what, name)
        dones += int(o[2].sum())
    gs, gt = env.get_state()
    os_, ot = ora.get_state()
    assert gt == ot and same(gs, os_)
    assert env.episode_stats() == ora.episode_stats()
    assert ora.episode_stats()[0] == dones
    env.close()


def draw_large_config(case):
    rng = np.random.default_rng(5000 + case)
    n = int(rng.choice([18944, 26048, 33152, 37888, 45056, 56832, 56848, 61568, 65536, 66304]))
    n -= int(rng.choice([0, 0, 16, 48]))                  # still a multiple of 16; the last chain ragged
    if rng.random() < 0.2:
        n -= 5                                            # no fast kernel takes it: general kernel throughout
    calls = []
    for _ in range(int(rng.integers(3, 6))):
        T = int(rng.choice([8, 16, 24, 40, 64, 72, 128, 136, 3, 1]))
        calls.append((T, int(rng.integers(0, 4)), int(rng.integers(0, 4))))     # T, action mode, kernel path
    return dict(n=n, seed=int(rng.integers(0, 2**63)), base=int(rng.choice([0, 7, 2**31 - 70000])),
                t0=int(rng.choice([0, 4, 2**34 + 8, 2])), near_end=bool(rng.random() < 0.5), calls=calls,
                state_seed=int(rng.integers(0, 2**31)))


@pytest.mark.parametrize("case", range(10))
def test_random_large_configuration_with_the_kernel_path_switched_between_calls(torch, case):
    """Batches of the sizes where the launcher's choice of vector kernel changes, with the path
    (auto, general, small blocks, balanced chains) drawn anew for every call of a run: whatever
    kernel ran last, the next one must pick the state up and give the oracle's bytes."""
    c = draw_large_config(case)
    n = c["n"]
    env = pong.PongEnv(n, c["seed"], env_id_base=c["base"])
    ora = oracle.OraclePong(n, c["seed"], env_id_base=c["base"])
    st = random_states(n, seed=c["state_seed"], near_end=c["near_end"])
    env.set_state(st, c["t0"])
    ora.set_state(st, c["t0"])
    for k, (T, mode, path) in enumerate(c["calls"]):
        what = "large case %d call %d (n %d, T %d, mode %d, path %d)" % (case, k, n, T, mode, path)
        env.set_vector_path(path)
        if mode == 2:
            acts = explicit_actions(T, n, seed=case * 100 + k, repeat_fraction=0.2, odd_codes=True)
            g = env.rollout(T, 2, torch.from_numpy(acts).cuda())
            o = ora.rollout(T, 2, acts)
        elif mode == 3:
            g = env.rollout(T, 3, k % 3)
            o = ora.rollout(T, 3, k % 3)
        else:
            g = env.rollout(T, mode)
            o = ora.rollout(T, mode)
        for name, gv, ov in zip(("obs", "reward", "done"), g, o):
            assert same(gv.cpu().numpy(), ov), "%s: %s differs" % (what, name)
    gs, gt = env.get_state()
    os_, ot = ora.get_state()
    assert gt == ot and same(gs, os_)
    assert env.episode_stats() == ora.episode_stats()
    env.close()
