"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs.  Everything is compared bit for bit: the
state is integer and the float32 obs is one correctly rounded multiply, so
the tolerance is 0 ULP (float arrays are compared as raw bytes)."""
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


def first_diff(a, b):
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    bad = np.argwhere(a.view(np.uint8).reshape(-1) != b.view(np.uint8).reshape(-1))
    return None if len(bad) == 0 else int(bad[0, 0])


def cpu(x):
    return x.cpu().numpy()


def assert_outputs_equal(gpu_out, ora_out, what=""):
    names = ("obs", "reward", "done")
    for name, g, o in zip(names, gpu_out, ora_out):
        g = cpu(g)
        assert same(g, o), "%s %s differs at byte %s" % (what, name, first_diff(g, o))


def assert_state_equal(env, ora, what=""):
    gs, gt = env.get_state()
    os_, ot = ora.get_state()
    assert gt == ot, what
    assert same(gs, os_), "%s state differs in fields %s" % (
        what, sorted({oracle.ENV_FIELDS[i] for i in np.argwhere(gs != os_)[:, 0]}))
    assert env.episode_stats() == ora.episode_stats(), what


# ---- small configuration: N = 64, T = 2000 ---------------------------------------------

@pytest.mark.parametrize("seed", [0, 1, 2, 0xDEADBEEF, 0x0123456789ABCDEF])
def test_small_config_rollout_philox(torch, seed):
    n, T = 64, 2000
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    assert same(cpu(env.reset()), ora.reset())
    for chunk in (128, 128, 744, 1000):
        assert_outputs_equal(env.rollout(chunk), ora.rollout(chunk), "seed %x" % seed)
    assert env.get_state()[1] == T
    assert_state_equal(env, ora)
    assert ora.episode_stats()[0] > 0


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
@pytest.mark.parametrize("n", [1, 31, 33, 1000])
def test_every_action_mode_ragged_sizes_unaligned_steps(torch, mode, n):
    seed = 7 + n
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    k = 0
    for T in (1, 2, 3, 5, 4, 127, 8, 64, 1, 129):
        k += 1
        if mode == 2:
            acts = explicit_actions(T, n, seed=100 + k, repeat_fraction=0.25, odd_codes=True)
            g = env.rollout(T, 2, torch.from_numpy(acts).cuda())
            o = ora.rollout(T, 2, acts)
        elif mode == 3:
            g = env.rollout(T, 3, k % 3)
            o = ora.rollout(T, 3, k % 3)
        else:
            g = env.rollout(T, mode)
            o = ora.rollout(T, mode)
        assert_outputs_equal(g, o, "mode %d n %d T %d" % (mode, n, T))
    assert_state_equal(env, ora)


@pytest.mark.parametrize("frameskip", [1, 2, 4, 16])
def test_auto_resets_from_states_near_episode_end(torch, frameskip):
    n, seed = 777, 99
    env = pong.PongEnv(n, seed, frameskip=frameskip)
    ora = oracle.OraclePong(n, seed, frameskip=frameskip)
    st = random_states(n, seed=5, near_end=True)
    env.set_state(st, 12345)
    ora.set_state(st, 12345)
    assert_state_equal(env, ora)
    total_done = 0
    for T, mode in ((40, 1), (3, 0), (64, 1), (200, 0)):
        g = env.rollout(T, mode)
        o = ora.rollout(T, mode)
        assert_outputs_equal(g, o, "fs %d" % frameskip)
        total_done += int(o[2].sum())
    assert total_done > n // 2
    assert_state_equal(env, ora)
    assert env.episode_stats(clear=True) == ora.episode_stats(clear=True)
    assert env.episode_stats() == (0, 0, 0)


def test_state_roundtrip_and_validation(torch):
    n = 100
    env = pong.PongEnv(n, 3)
    st = random_states(n, seed=8)
    env.set_state(st, 2**40 + 5)
    got, t = env.get_state()
    assert same(got, st) and t == 2**40 + 5
    for field, bad in ((0, -1), (0, 40961), (1, 48641), (2, 0), (2, 1025), (3, 769), (4, 45057),
                       (5, -1), (6, 21), (7, 21), (8, 10000), (9, -1), (10, 3)):
        s2 = st.copy()
        s2[field, 17] = bad
        with pytest.raises(pong.PongError) as ei:
            env.set_state(s2, 0)
        assert ei.value.code == -1
    got, t = env.get_state()
    assert same(got, st) and t == 2**40 + 5      # rejected states change nothing


def test_huge_step_counter_keys_philox_with_all_64_bits(torch):
    n, seed = 40, 11
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    st, _ = ora.get_state()
    t0 = (1 << 36) + 3
    env.set_state(st, t0)
    ora.set_state(st, t0)
    assert_outputs_equal(env.rollout(50, 1), ora.rollout(50, 1))
    assert_state_equal(env, ora)


@pytest.mark.parametrize("n", [16, 48, 64, 1040, 4096])
@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_tma_path_aligned_sizes_with_auto_resets(torch, n, mode):
    """Sizes and step counts that take the TMA-store kernel (n % 16 == 0,
    t % 4 == 0, T % 8 == 0), including a ragged last block, from states close
    to the episode end so that both rare paths run often; then a mix with
    calls that fall back to the general kernel."""
    seed = 500 + n
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    st = random_states(n, seed=n, near_end=True)
    env.set_state(st, 4096)
    ora.set_state(st, 4096)
    dones = 0
    for k, T in enumerate((8, 64, 16, 128, 3, 8, 1, 24, 40)):
        if mode == 2:
            acts = explicit_actions(T, n, seed=k, repeat_fraction=0.25, odd_codes=True)
            g = env.rollout(T, 2, torch.from_numpy(acts).cuda())
            o = ora.rollout(T, 2, acts)
        elif mode == 3:
            g = env.rollout(T, 3, (k + 1) % 3)
            o = ora.rollout(T, 3, (k + 1) % 3)
        else:
            g = env.rollout(T, mode)
            o = ora.rollout(T, mode)
        assert_outputs_equal(g, o, "n %d mode %d T %d" % (n, mode, T))
        dones += int(o[2].sum())
    assert dones >= n
    assert_state_equal(env, ora)


def test_tma_path_falls_back_on_unaligned_done_pointer(torch):
    n, T, seed = 256, 16, 77
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    obs = torch.empty((T, n, 6), dtype=torch.float32, device="cuda")
    reward = torch.empty((T, n), dtype=torch.float32, device="cuda")
    raw = torch.empty((T * n + 16,), dtype=torch.uint8, device="cuda")
    done = raw[1:1 + T * n].view(T, n)
    assert done.data_ptr() % 16 != 0
    env.rollout(T, 0, None, obs, reward, done)
    assert_outputs_equal((obs, reward, done), ora.rollout(T, 0))
    assert_state_equal(env, ora)


# ---- single-step API -------------------------------------------------------------------------

def test_step_api_against_oracle(torch):
    n, seed, T = 257, 21, 400
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    acts = explicit_actions(T, n, seed=1, repeat_fraction=0.1, odd_codes=True)
    d_acts = torch.from_numpy(acts).cuda()
    for t in range(T):
        g = env.step(d_acts[t])
        o = ora.step(acts[t])
        assert_outputs_equal(g, o, "t %d" % t)
    assert_state_equal(env, ora)


def test_rollout_equals_repeated_step_with_filled_actions(torch):
    n, seed, T = 300, 5, 96
    for sticky in (0, 1):
        a = pong.PongEnv(n, seed)
        b = pong.PongEnv(n, seed)
        ora = oracle.OraclePong(n, seed)
        a.rollout(7, sticky)
        b.rollout(7, sticky)
        ora.rollout(7, sticky)
        acts = b.fill_actions(T, sticky)
        assert same(cpu(acts), ora.fill_actions(T, sticky))
        obs, reward, done = a.rollout(T, sticky)
        for t in range(T):
            o1, r1, d1 = b.step(acts[t])
            assert same(cpu(o1), cpu(obs[t])) and same(cpu(r1), cpu(reward[t])) and \
                same(cpu(d1), cpu(done[t]))
        assert same(a.get_state()[0], b.get_state()[0])
        assert a.episode_stats() == b.episode_stats()


def test_save_restore_continues_identically(torch):
    n, seed = 128, 42
    a = pong.PongEnv(n, seed)
    a.rollout(555, 1)
    st, t = a.get_state()
    b = pong.PongEnv(n, seed)
    b.set_state(st, t)
    ga, gb = a.rollout(300, 1), b.rollout(300, 1)
    for x, y in zip(ga, gb):
        assert same(cpu(x), cpu(y))
    assert same(a.get_state()[0], b.get_state()[0])


def test_env_id_base_partition_reproduces_the_whole_batch(torch):
    seed, T = 123, 500
    whole = pong.PongEnv(96, seed)
    lo = pong.PongEnv(50, seed, env_id_base=0)
    hi = pong.PongEnv(46, seed, env_id_base=50)
    gw, gl, gh = whole.rollout(T, 1), lo.rollout(T, 1), hi.rollout(T, 1)
    for w, l, h in zip(gw, gl, gh):
        assert same(cpu(w[:, :50]), cpu(l)) and same(cpu(w[:, 50:]), cpu(h))
    sw, sl, sh = whole.episode_stats(), lo.episode_stats(), hi.episode_stats()
    assert sw == tuple(x + y for x, y in zip(sl, sh))


# ---- brute force: every action sequence ---------------------------------------------------------

def test_brute_force_every_action_sequence_near_the_paddles(torch):
    """All 3^8 sequences, one per env, from states in which the ball is about
    to reach a paddle or a court edge, so the outcome depends on the actions."""
    T = 8
    n = 3 ** T
    seqs = np.zeros((T, n), dtype=np.uint8)
    for i in range(n):
        v = i
        for t in range(T):
            seqs[t, i] = v % 3
            v //= 3
    starts = [
        dict(bx=36400, by=20000, vx=512, vy=0, apy=20000 + 512 + 768, opy=22528),
        dict(bx=35000, by=30000, vx=1024, vy=-700, apy=29000, opy=1000),
        dict(bx=38000, by=47000, vx=900, vy=768, apy=45056, opy=45056),
        dict(bx=4500, by=300, vx=-1000, vy=-768, apy=0, opy=0),
    ]
    for k, s in enumerate(starts):
        st = np.zeros((11, n), dtype=np.int32)
        for j, name in enumerate(oracle.ENV_FIELDS):
            st[j] = s.get(name, 0)
        st[6] = 20            # one more agent point ends the episode
        st[8] = 9996          # and so do four more frames
        env = pong.PongEnv(n, 1000 + k)
        ora = oracle.OraclePong(n, 1000 + k)
        env.set_state(st, 0)
        ora.set_state(st, 0)
        g = env.rollout(T, 2, torch.from_numpy(seqs).cuda())
        o = ora.rollout(T, 2, seqs)
        assert_outputs_equal(g, o, "start %d" % k)
        assert_state_equal(env, ora)
        assert o[2].sum() >= n   # every env ended an episode


# ---- pixels ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [1, 37, 300])
def test_pixel_rollout_and_step_against_oracle(torch, n):
    seed = 31
    env = pong.PongEnv(n, seed, obs_mode=1, frameskip=4)
    ora = oracle.OraclePong(n, seed, obs_mode=1, frameskip=4)
    assert same(cpu(env.ring), ora.ring)
    k = 0
    for T in (1, 1, 1, 3, 64, 2, 5):
        g = env.rollout(T, 1)
        o = ora.rollout(T, 1)
        assert_outputs_equal(g, o, "pixel T %d" % T)
    # single steps with explicit actions
    for t in range(9):
        acts = explicit_actions(1, n, seed=t)[0]
        g = env.step(torch.from_numpy(acts).cuda())
        o = ora.step(acts)
        assert_outputs_equal(g, o, "pixel step %d" % t)
    # episode ends: the reset frame fills all four slots
    st = random_states(n, seed=2, near_end=True)
    st[8] = np.where(np.arange(n) % 2 == 0, 9990, st[8])
    t_now = env.get_state()[1]
    env.set_state(st, t_now)
    ora.set_state(st, t_now)
    dones = 0
    for T in (1, 2, 7, 30):
        g = env.rollout(T, 0)
        o = ora.rollout(T, 0)
        assert_outputs_equal(g, o, "pixel resets T %d" % T)
        dones += int(o[2].sum())
    assert dones >= n // 2
    assert_state_equal(env, ora)
    assert same(cpu(env.reset()), ora.reset())


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_pixel_four_step_path_with_resets_inside_a_pass(torch, mode):
    """Aligned calls (t % 4 == 0, T % 4 == 0) take the kernel that paints a whole
    4-slot ring per pass; episode ends in the middle of a pass must leave every
    slot as the frame-at-a-time definition does."""
    n, seed = 203, 77
    env = pong.PongEnv(n, seed, obs_mode=1, frameskip=4)
    ora = oracle.OraclePong(n, seed, obs_mode=1, frameskip=4)
    st = random_states(n, seed=9, near_end=True)
    st[8] = 9999 - (np.arange(n) % 40)          # episodes end at every phase of a pass
    env.set_state(st, 64)
    ora.set_state(st, 64)
    dones = 0
    for k, T in enumerate((4, 8, 4, 12, 4, 4, 64)):
        if mode == 2:
            acts = explicit_actions(T, n, seed=k, repeat_fraction=0.2)
            g = env.rollout(T, 2, torch.from_numpy(acts).cuda())
            o = ora.rollout(T, 2, acts)
        elif mode == 3:
            g = env.rollout(T, 3, k % 3)
            o = ora.rollout(T, 3, k % 3)
        else:
            g = env.rollout(T, mode)
            o = ora.rollout(T, mode)
        assert_outputs_equal(g, o, "x4 mode %d T %d" % (mode, T))
        dones += int(o[2].sum())
    assert dones >= n
    assert_state_equal(env, ora)
    # then unaligned calls (frame-at-a-time kernel) and back
    for T in (3, 1, 4, 8):
        assert_outputs_equal(env.rollout(T, 0), ora.rollout(T, 0), "mixed T %d" % T)
    assert_state_equal(env, ora)


def test_pixel_one_env_per_block_long_rollouts_through_episode_ends(torch):
    """Few envs: every block (and warp) owns a single env, so consecutive steps re-store the same
    ring bytes from the same thread a few microseconds apart (a reset writes all four slots, the
    next step one of them).  Long enough for several episode ends per env, on both pixel kernels."""
    n, seed = 5, 123
    env = pong.PongEnv(n, seed, obs_mode=1, frameskip=4)
    ora = oracle.OraclePong(n, seed, obs_mode=1, frameskip=4)
    st = random_states(n, seed=4, near_end=True)
    st[8] = 9990 - 3 * np.arange(n)
    env.set_state(st, 0)
    ora.set_state(st, 0)
    dones = 0
    for T in (600, 1, 599, 2, 2, 600):          # aligned (four steps per pass), then unaligned, then aligned
        g, o = env.rollout(T, 0), ora.rollout(T, 0)
        assert_outputs_equal(g, o, "one env per block, T %d" % T)
        dones += int(o[2].sum())
    assert dones >= 2 * n
    assert_state_equal(env, ora)


def test_pixel_frameskip_one_and_constant_action(torch):
    n, seed = 50, 8
    env = pong.PongEnv(n, seed, obs_mode=1, frameskip=1)
    ora = oracle.OraclePong(n, seed, obs_mode=1, frameskip=1)
    for T, a in ((10, 2), (33, 1), (4, 0)):
        assert_outputs_equal(env.rollout(T, 3, a), ora.rollout(T, 3, a))
    assert_state_equal(env, ora)


# ---- boundary behaviour ------------------------------------------------------------------------------

def test_outputs_do_not_overrun_their_buffers(torch):
    n, T = 130, 9
    env = pong.PongEnv(n, 0)
    pad = 64
    obs = torch.full((T * n * 6 + pad,), 7.0, dtype=torch.float32, device="cuda")
    reward = torch.full((T * n + pad,), 7.0, dtype=torch.float32, device="cuda")
    done = torch.full((T * n + pad,), 7, dtype=torch.uint8, device="cuda")
    env.rollout(T, 0, None, obs, reward, done)
    torch.cuda.synchronize()
    assert bool((obs[T * n * 6:] == 7.0).all()) and bool((reward[T * n:] == 7.0).all())
    assert bool((done[T * n:] == 7).all())
    assert bool((done[:T * n] <= 1).all())
    penv = pong.PongEnv(10, 0, obs_mode=1, frameskip=4)
    ring = torch.full((10 * 4 * 84 * 84 + 256,), 9, dtype=torch.uint8, device="cuda")
    pong.pong_reset(penv.h, ring)
    reward = torch.empty((5, 10), dtype=torch.float32, device="cuda")
    done = torch.empty((5, 10), dtype=torch.uint8, device="cuda")
    penv.rollout(5, 0, None, ring, reward, done)
    torch.cuda.synchronize()
    assert bool((ring[10 * 4 * 84 * 84:] == 9).all())
    assert set(torch.unique(ring[:10 * 4 * 84 * 84]).tolist()) <= {0, 255}


def test_argument_errors(torch):
    n = 64
    env = pong.PongEnv(n, 0)
    obs = torch.empty((4, n, 6), dtype=torch.float32, device="cuda")
    reward = torch.empty((4, n), dtype=torch.float32, device="cuda")
    done = torch.empty((4, n), dtype=torch.uint8, device="cuda")
    acts = torch.zeros((4, n), dtype=torch.uint8, device="cuda")

    def code(fn, *args):
        with pytest.raises(pong.PongError) as ei:
            fn(*args)
        return ei.value.code

    assert code(pong.pong_rollout, env.h, 0, 0, None, obs, reward, done) == -1
    assert code(pong.pong_rollout, env.h, 4, 4, None, obs, reward, done) == -5
    assert code(pong.pong_rollout, env.h, 4, -1, None, obs, reward, done) == -5
    assert code(pong.pong_rollout, env.h, 4, 2, None, obs, reward, done) == -2
    assert code(pong.pong_rollout, env.h, 4, 0, None, None, reward, done) == -2
    assert code(pong.pong_rollout, env.h, 4, 0, None, obs.data_ptr() + 4, reward, done) == -3
    assert code(pong.pong_rollout, env.h, 4, 0, None, obs, reward.data_ptr() + 4, done) == -3
    assert code(pong.pong_rollout, env.h, 4, 3, np.array([3], dtype=np.uint8), obs, reward, done) == -1
    assert code(pong.pong_step, env.h, None, obs, reward, done) == -2
    assert code(pong.pong_step, env.h, acts, obs.data_ptr() + 8, reward, done) == -3
    assert code(pong.pong_fill_actions, env.h, 0, 0, acts) == -1
    assert code(pong.pong_fill_actions, env.h, 4, 0, None) == -2
    # nothing above advanced the step counter or touched the state
    ora = oracle.OraclePong(n, 0)
    assert_state_equal(env, ora)
    env.rollout(4, 2, acts, obs, reward, done)
    o = ora.rollout(4, 2, cpu(acts))
    assert_outputs_equal((obs, reward, done), o)


def test_rollout_host_matches_device_rollout(torch):
    n, T, seed = 500, 40, 9
    a = pong.PongEnv(n, seed)
    b = pong.PongEnv(n, seed)
    obs_h = torch.empty((T, n, 6), dtype=torch.float32).pin_memory()
    rew_h = torch.empty((T, n), dtype=torch.float32).pin_memory()
    done_h = torch.empty((T, n), dtype=torch.uint8).pin_memory()
    acts = explicit_actions(T, n, seed=3)
    acts_h = torch.from_numpy(acts).pin_memory()
    for mode, arg_h, arg_d in ((1, None, None), (2, acts_h, torch.from_numpy(acts).cuda()),
                               (1, None, None)):
        pong.pong_rollout_host(b.h, T, mode, arg_h, obs_h, rew_h, done_h)
        g = a.rollout(T, mode, arg_d)
        assert same(cpu(g[0]), obs_h.numpy()) and same(cpu(g[1]), rew_h.numpy()) and \
            same(cpu(g[2]), done_h.numpy())
    assert same(a.get_state()[0], b.get_state()[0])


def test_runs_on_a_side_stream(torch):
    n, seed = 256, 4
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        g = env.rollout(64, 1)
        g2 = env.rollout(64, 1)
    s.synchronize()
    assert_outputs_equal(g, ora.rollout(64, 1))
    assert_outputs_equal(g2, ora.rollout(64, 1))
