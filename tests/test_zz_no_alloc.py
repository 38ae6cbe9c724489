"""pong_rollout_static, the entry point for hosts that cannot allocate device
memory while running (its env state sits in a fixed array inside the library),
must give exactly what the handle-based entry points give.  Checked on two
calls in a row that share the array, with different sizes, seeds and modes, so
that nothing left behind by the first call can leak into the second.  This file
is collected last on purpose."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import pong

pytestmark = pytest.mark.gpu


def run_both(torch, n, seed, base, T, mode, actions=None, with_stats=True, against_oracle=False):
    obs = torch.empty((T, n, 6), dtype=torch.float32, device="cuda")
    reward = torch.empty((T, n), dtype=torch.float32, device="cuda")
    done = torch.empty((T, n), dtype=torch.uint8, device="cuda")
    stats = torch.full((3,), -1, dtype=torch.int64, device="cuda") if with_stats else None
    stream = torch.cuda.current_stream().cuda_stream
    dev_actions = actions
    if mode == pong.ACT_CONSTANT:
        dev_actions = np.array([actions], dtype=np.uint8)            # a host byte
    pong.pong_rollout_static(n, seed, base, T, mode, dev_actions, obs, reward, done, stats, stream)
    env = pong.PongEnv(n, seed, env_id_base=base)
    want = env.rollout(T, mode, actions)
    torch.cuda.synchronize()
    for got, ref in zip((obs, reward, done), want):
        assert got.cpu().numpy().tobytes() == ref.cpu().numpy().tobytes()
    if with_stats:
        assert tuple(stats.cpu().tolist()) == env.episode_stats()
    if against_oracle:
        ora = oracle.OraclePong(n, seed, env_id_base=base)
        host_actions = actions.cpu().numpy() if hasattr(actions, "cpu") else actions
        for got, ref in zip((obs, reward, done), ora.rollout(T, mode, host_actions)):
            assert got.cpu().numpy().tobytes() == ref.tobytes()
        if with_stats:
            assert tuple(stats.cpu().tolist()) == tuple(ora.episode_stats())
    return env.episode_stats()


def test_static_rollout_matches_handle_rollout_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    pong.load(build_if_missing=True)
    # long enough for episodes to finish, so the counters are non-zero
    first = run_both(torch, 4096, 7, 0, 4000, pong.ACT_PHILOX)
    assert first[0] > 0
    # second call: other size (ragged), seed, id range and mode; shares the array
    second = run_both(torch, 1000, 0xABCDEF0123, 500, 2504, pong.ACT_STICKY)
    assert second[0] > 0 and second != first
    # and the first configuration again gives the first result again
    assert run_both(torch, 4096, 7, 0, 4000, pong.ACT_PHILOX) == first


def test_static_rollout_largest_batch_every_action_mode_and_the_oracle():
    """The largest batch the array holds (its last env's state sits directly before the three
    counters), through the aligned fast kernels and the general one, every action source, with
    and without the statistics output, and directly against the CPU oracle."""
    import torch
    pong.load(build_if_missing=True)
    n = pong.STATIC_MAX_ENVS
    run_both(torch, n, 21, 0, 8, pong.ACT_PHILOX, against_oracle=True)
    run_both(torch, n, 22, 128, 11, pong.ACT_STICKY, against_oracle=True)        # unaligned T: general kernel
    env = pong.PongEnv(n, 23)
    bytes_ = env.fill_actions(16, 1)                                           # explicit bytes, with repeats
    run_both(torch, n, 23, 0, 16, pong.ACT_EXPLICIT, actions=bytes_, against_oracle=True)
    run_both(torch, 4096, 24, 7, 24, pong.ACT_CONSTANT, actions=2, with_stats=False, against_oracle=True)
    run_both(torch, 1000, 7, 0, 2000, pong.ACT_PHILOX, against_oracle=True)      # finished episodes


def test_static_rollout_rejects_bad_sizes():
    import torch
    pong.load(build_if_missing=True)
    buf = torch.empty((64,), dtype=torch.float32, device="cuda")
    d = torch.empty((64,), dtype=torch.uint8, device="cuda")
    for n, code in ((pong.STATIC_MAX_ENVS + 1, -7), (0, -1)):
        with pytest.raises(pong.PongError) as ei:
            pong.pong_rollout_static(n, 0, 0, 1, 0, None, buf, buf, d)
        assert ei.value.code == code
    with pytest.raises(pong.PongError) as ei:
        pong.pong_rollout_static(8, 0, 0, 1, 0, None, None, buf, d)
    assert ei.value.code == -2
    with pytest.raises(pong.PongError) as ei:           # T * n beyond what the kernels address
        pong.pong_rollout_static(pong.STATIC_MAX_ENVS, 0, 0, 2 ** 31 - 1, 0, None, buf, buf, d)
    assert ei.value.code == -1
    assert "maximum" in pong.strerror(-7)
