"""Parity of the balanced-chains vector rollout (one block per SM, warp chains, leftover
chains alternating between two warps) with the CPU oracle, element by element, through
the C ABI with the path forced.  Sizes are chosen so that blocks on a 148-SM part hold
every mix the kernel distinguishes: one chain, 4 + 1 / 4 + 2 (alternating leftovers),
4 + 3 (whole leftovers), 8 + 1 / 8 + 2, 12 + 1 / 12 + 2, the largest batch the kernel
takes, a ragged last chain; stage counts 1, 2, 3 (no alternation), 5 and 9 (a last segment of one
stage), 6, 8, 16, and 17, 33, 49 (launches long enough for the block-wide rendezvous every 16 stages)."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import pong
from paper_2603_12145_b200.inputs import explicit_actions, random_states

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available()
    pong.load(build_if_missing=True)
    return torch


def same(got, want, what):
    for g, w, name in zip(got, want, ("obs", "reward", "done")):
        g = g.cpu().numpy()
        assert g.shape == w.shape and g.tobytes() == w.tobytes(), "%s: %s differs" % (what, name)


def run_pair(env, ora, T, mode, seed):
    acts = None
    if mode == pong.ACT_EXPLICIT:
        acts = explicit_actions(T, env.n, seed=seed, repeat_fraction=0.2, odd_codes=True)
    elif mode == pong.ACT_CONSTANT:
        acts = 2
    got = env.rollout(T, mode, acts if mode != pong.ACT_EXPLICIT else env.torch.from_numpy(acts).cuda())
    want = ora.rollout(T, mode, acts)
    return got, want


@pytest.mark.parametrize("n,T,mode", [
    (16, 8, 0), (48, 16, 1), (1040, 24, 2), (4112, 40, 3),
    (26048, 24, 0), (26048, 40, 1), (26048, 72, 0), (33152, 24, 0), (45056, 40, 2), (45056, 64, 1),
    (61568, 16, 0), (65536, 40, 0), (65536, 72, 1), (65536, 48, 2), (66304, 64, 3), (66288, 128, 0),
    (65536, 128, 0), (65536, 264, 0), (26048, 136, 1), (45056, 392, 0),
])
def test_chains_path_matches_the_oracle(torch_cuda, n, T, mode):
    seed, base = 1000 + n % 97, 3
    env = pong.PongEnv(n, seed, env_id_base=base)
    env.set_vector_path(pong.PATH_CHAINS)
    ora = oracle.OraclePong(n, seed, env_id_base=base)
    for rep in range(2):                       # the second launch starts from the first one's state
        got, want = run_pair(env, ora, T, mode, seed + rep)
        same(got, want, "n=%d T=%d mode=%d launch %d" % (n, T, mode, rep))
    s_gpu, t_gpu = env.get_state()
    s_cpu, t_cpu = ora.get_state()
    assert t_gpu == t_cpu and s_gpu.tobytes() == s_cpu.tobytes()
    assert tuple(env.episode_stats()) == tuple(ora.episode_stats())
    env.close()


def test_chains_path_through_episode_ends(torch_cuda):
    """Near-end start states: scores at 15-20 and frame counts close to 10,000, so that resets,
    the step limit and fresh spawn queues fall inside alternating segments."""
    n, T, seed = 65536, 64, 77
    env = pong.PongEnv(n, seed)
    env.set_vector_path(pong.PATH_CHAINS)
    ora = oracle.OraclePong(n, seed)
    st = random_states(n, seed, near_end=True)
    env.set_state(st, 4096)
    ora.set_state(st, 4096)
    for mode in (0, 1):
        got, want = run_pair(env, ora, T, mode, seed)
        same(got, want, "near-end mode %d" % mode)
    assert tuple(env.episode_stats()) == tuple(ora.episode_stats())
    assert env.episode_stats()[0] > n // 2
    s_gpu, _ = env.get_state()
    s_cpu, _ = ora.get_state()
    assert s_gpu.tobytes() == s_cpu.tobytes()
    env.close()


def test_every_path_gives_the_same_bytes_and_unaligned_calls_fall_through(torch_cuda):
    torch = torch_cuda
    n, seed = 61440, 5
    outs = []
    for path in (pong.PATH_AUTO, pong.PATH_GENERAL, pong.PATH_TMA, pong.PATH_CHAINS):
        env = pong.PongEnv(n, seed)
        env.set_vector_path(path)
        a = env.rollout(16, pong.ACT_PHILOX)      # aligned
        b = env.rollout(3, pong.ACT_STICKY)       # T % 8 != 0: every path falls through to the general kernel
        c = env.rollout(13, pong.ACT_PHILOX)      # t0 % 4 != 0
        outs.append([t.clone() for t in (*a, *b, *c)] + [torch.from_numpy(env.get_state()[0])])
        env.close()
    for other in outs[1:]:
        for x, y in zip(outs[0], other):
            assert torch.equal(x.cpu(), y.cpu())
    ora = oracle.OraclePong(n, seed)
    want = (*ora.rollout(16, 0), *ora.rollout(3, 1), *ora.rollout(13, 0))
    for g, w in zip(outs[0], want):
        assert g.cpu().numpy().tobytes() == w.tobytes()
    with pytest.raises(pong.PongError) as e:
        env = pong.PongEnv(16, 1)
        env.set_vector_path(7)
    assert e.value.code == -1


@pytest.mark.parametrize("n,path", [(65536, pong.PATH_AUTO), (65536, pong.PATH_CHAINS), (4096, pong.PATH_AUTO),
                                    (45056, pong.PATH_TMA)])
def test_calls_that_start_or_end_off_the_grid_are_cut_and_still_match(torch_cuda, n, path):
    """A call whose first step is no multiple of 4, or whose length is no multiple of 8, runs as a
    short general-kernel head, a fast-kernel middle and a general-kernel tail (1 to 3 kernels):
    the pieces must hand the state on exactly, in every action mode, and the kernel count shows
    that the cut was taken."""
    torch = torch_cuda
    seed = 17
    env = pong.PongEnv(n, seed, env_id_base=9)
    env.set_vector_path(path)
    ora = oracle.OraclePong(n, seed, env_id_base=9)
    for k, (T, mode, kernels) in enumerate([(100, 0, 2), (1, 1, 1), (128, 1, 3), (37, 2, 3), (21, 3, 3), (23, 0, 3),
                                            (128, 0, 3), (15, 0, 1), (3, 1, 1), (128, 0, 1)]):
        before = env.launches
        if mode == 2:
            acts = explicit_actions(T, n, seed=k, repeat_fraction=0.3, odd_codes=True)
            g, o = env.rollout(T, 2, torch.from_numpy(acts).cuda()), ora.rollout(T, 2, acts)
        elif mode == 3:
            g, o = env.rollout(T, 3, 1), ora.rollout(T, 3, 1)
        else:
            g, o = env.rollout(T, mode), ora.rollout(T, mode)
        same(g, o, "cut call %d (T %d, mode %d)" % (k, T, mode))
        assert env.launches - before == kernels, (k, T, env.launches - before)
    assert env.get_state()[0].tobytes() == ora.get_state()[0].tobytes()
    assert tuple(env.episode_stats()) == tuple(ora.episode_stats())
    env.close()
