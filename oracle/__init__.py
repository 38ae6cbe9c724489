"""CPU oracle of the batched fixed-point Pong step -- TEST INFRASTRUCTURE.

Only the tests, the smoke check and the CPU-baseline timing of the benchmark
may import this package.  The CUDA library never does: the two share no code.

The arithmetic lives in ``pong_oracle.c`` (plain C, compiled here with gcc);
this module only builds it, loads it through ctypes and marshals numpy
arrays.  See the header of ``pong_oracle.c`` for what the oracle follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pong_oracle.c")
_LIB = os.path.join(_HERE, "libpong_oracle.so")
_lock = threading.Lock()
_lib = None

ENV_FIELDS = ("bx", "by", "vx", "vy", "apy", "opy", "score_a", "score_o",
              "ep_len", "episode", "prev_action")
FRAME_BYTES = 84 * 84


def build(force: bool = False) -> str:
    """Compile pong_oracle.c into libpong_oracle.so (no fast-math, no FMA
    contraction, so the fp32 obs multiply stays a single rounded multiply)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off",
           "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Env(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int32) for name in ENV_FIELDS]


class _Stats(ctypes.Structure):
    _fields_ = [("episodes", ctypes.c_int64), ("sum_return", ctypes.c_int64),
                ("sum_length", ctypes.c_int64)]


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            u32, u64, i32 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int
            vp = ctypes.c_void_p
            L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
            L.oracle_philox4x32_10.restype = None
            L.oracle_action_word.argtypes = [u64, u32, u64]
            L.oracle_action_word.restype = u32
            L.oracle_action_uniform.argtypes = [u32]
            L.oracle_action_uniform.restype = i32
            L.oracle_action_repeat.argtypes = [u32]
            L.oracle_action_repeat.restype = i32
            L.oracle_spawn.argtypes = [vp, u64, u32, u32, u32]
            L.oracle_spawn.restype = None
            L.oracle_reset_env.argtypes = [vp, u64, u32, u32]
            L.oracle_reset_env.restype = None
            L.oracle_frame.argtypes = [vp, i32, u64, u32, vp, vp]
            L.oracle_frame.restype = i32
            L.oracle_obs_vector.argtypes = [vp, vp]
            L.oracle_obs_vector.restype = None
            L.oracle_render.argtypes = [vp, vp]
            L.oracle_render.restype = None
            L.oracle_reset.argtypes = [vp, i32, u64, u32]
            L.oracle_reset.restype = None
            L.oracle_initial_obs.argtypes = [vp, i32, i32, vp, vp]
            L.oracle_initial_obs.restype = None
            L.oracle_decode_action.argtypes = [ctypes.c_uint8, i32]
            L.oracle_decode_action.restype = i32
            L.oracle_rollout.argtypes = [vp, i32, u64, u32, u64, i32, i32, vp,
                                         i32, i32, vp, vp, vp, vp, vp]
            L.oracle_rollout.restype = i32
            L.oracle_fill_actions.argtypes = [i32, u64, u32, u64, i32, i32, vp]
            L.oracle_fill_actions.restype = None
            L.oracle_expn.argtypes = [ctypes.c_float]
            L.oracle_expn.restype = ctypes.c_float
            L.oracle_sample_action.argtypes = [vp, u32]
            L.oracle_sample_action.restype = i32
            L.oracle_sample_actions.argtypes = [i32, vp, vp, vp]
            L.oracle_sample_actions.restype = None
            L.oracle_fill_words.argtypes = [i32, u64, u32, u64, i32, vp]
            L.oracle_fill_words.restype = None
            L.oracle_sizeof_env.argtypes = []
            L.oracle_sizeof_env.restype = i32
            assert L.oracle_sizeof_env() == ctypes.sizeof(_Env)
            _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return [int(x) for x in out]


def action_word(seed, env_id, t):
    return int(lib().oracle_action_word(seed, env_id, t))


def action_uniform(word):
    return int(lib().oracle_action_uniform(word))


def action_repeat(word):
    return int(lib().oracle_action_repeat(word))


def decode_action(byte, prev_action):
    return int(lib().oracle_decode_action(byte, prev_action))


def expn(x):
    return float(lib().oracle_expn(float(x)))


def sample_actions(logits, words):
    """uint8 [n] actions drawn from softmax(logits[n, 3]) with the uniform words[n]."""
    logits = np.ascontiguousarray(logits, dtype=np.float32).reshape(-1, 3)
    words = np.ascontiguousarray(words, dtype=np.uint32).reshape(-1)
    assert len(words) == len(logits)
    out = np.zeros(len(words), dtype=np.uint8)
    lib().oracle_sample_actions(len(words), _ptr(logits), _ptr(words), _ptr(out))
    return out


class Env:
    """One env, for unit tests of single frames."""

    def __init__(self, **fields):
        self.c = _Env()
        for k, v in fields.items():
            setattr(self.c, k, v)

    def __getattr__(self, name):
        if name in ENV_FIELDS:
            return getattr(self.c, name)
        raise AttributeError(name)

    def as_dict(self):
        return {k: getattr(self.c, k) for k in ENV_FIELDS}

    def reset(self, seed, env_id, episode):
        lib().oracle_reset_env(ctypes.byref(self.c), seed, env_id, episode)
        return self

    def spawn(self, seed, env_id, episode, point):
        lib().oracle_spawn(ctypes.byref(self.c), seed, env_id, episode, point)
        return self

    def frame(self, action, seed=0, env_id=0, stats=None):
        """One physics frame; returns (reward, done)."""
        done = ctypes.c_int(0)
        st = stats if stats is not None else _Stats()
        r = lib().oracle_frame(ctypes.byref(self.c), action, seed, env_id,
                               ctypes.byref(st), ctypes.byref(done))
        return int(r), int(done.value)

    def obs_vector(self):
        out = np.zeros(6, dtype=np.float32)
        lib().oracle_obs_vector(ctypes.byref(self.c), _ptr(out))
        return out

    def render(self):
        out = np.zeros(FRAME_BYTES, dtype=np.uint8)
        lib().oracle_render(ctypes.byref(self.c), _ptr(out))
        return out.reshape(84, 84)


def new_stats():
    return _Stats()


class OraclePong:
    """Batch of envs with the same call surface as the CUDA library's handle
    (create / reset / step / rollout / fill_actions / episode_stats /
    get_state / set_state), on numpy arrays."""

    def __init__(self, n_envs, seed, obs_mode=0, frameskip=1, env_id_base=0):
        self.n = int(n_envs)
        self.seed = int(seed) & 0xFFFFFFFFFFFFFFFF
        self.obs_mode = int(obs_mode)
        self.frameskip = int(frameskip)
        self.env_id_base = int(env_id_base)
        self.envs = (_Env * max(self.n, 1))()
        self.stats = _Stats()
        self.t = 0
        self.ring = (np.zeros((self.n, 4, 84, 84), dtype=np.uint8)
                     if self.obs_mode == 1 else None)
        self.reset()

    def reset(self):
        """All envs to episode 0, global step 0, stats cleared.  Returns the
        initial obs (vector [n,6]) or the ring (pixel)."""
        lib().oracle_reset(self.envs, self.n, self.seed, self.env_id_base)
        self.stats = _Stats()
        self.t = 0
        if self.obs_mode == 0:
            obs = np.zeros((self.n, 6), dtype=np.float32)
            lib().oracle_initial_obs(self.envs, self.n, 0, _ptr(obs), None)
            return obs
        lib().oracle_initial_obs(self.envs, self.n, 1, None, _ptr(self.ring))
        return self.ring

    def rollout(self, T, action_mode=0, actions=None):
        """Returns (obs, reward[T,n], done[T,n]); obs is [T,n,6] float32 or the
        persistent ring [n,4,84,84]."""
        T = int(T)
        n = self.n
        reward = np.zeros((T, n), dtype=np.float32)
        done = np.zeros((T, n), dtype=np.uint8)
        obs = np.zeros((T, n, 6), dtype=np.float32) if self.obs_mode == 0 else None
        act = None
        if action_mode == 2:
            act = np.ascontiguousarray(actions, dtype=np.uint8).reshape(T, n)
        elif action_mode == 3:
            act = np.array([int(actions)], dtype=np.uint8)
        rc = lib().oracle_rollout(self.envs, n, self.seed, self.env_id_base,
                                  self.t, T, action_mode, _ptr(act),
                                  self.frameskip, self.obs_mode, _ptr(obs),
                                  _ptr(self.ring), _ptr(reward), _ptr(done),
                                  ctypes.byref(self.stats))
        if rc != 0:
            raise ValueError("oracle_rollout: bad arguments")
        self.t += T
        return (obs if self.obs_mode == 0 else self.ring), reward, done

    def step(self, actions):
        obs, reward, done = self.rollout(1, 2, np.asarray(actions).reshape(1, self.n))
        if self.obs_mode == 0:
            obs = obs[0]
        return obs, reward[0], done[0]

    def fill_actions(self, T, sticky=0):
        out = np.zeros((int(T), self.n), dtype=np.uint8)
        lib().oracle_fill_actions(self.n, self.seed, self.env_id_base, self.t,
                                  int(T), int(sticky), _ptr(out))
        return out

    def fill_words(self, T):
        """uint32 [T, n]: the Philox action words of the next T global steps."""
        out = np.zeros((int(T), self.n), dtype=np.uint32)
        lib().oracle_fill_words(self.n, self.seed, self.env_id_base, self.t, int(T), _ptr(out))
        return out

    def episode_stats(self, clear=False):
        s = (int(self.stats.episodes), int(self.stats.sum_return),
             int(self.stats.sum_length))
        if clear:
            self.stats = _Stats()
        return s

    def get_state(self):
        """int32 [11, n] in ENV_FIELDS order, and the global step t."""
        raw = np.frombuffer(self.envs, dtype=np.int32,
                            count=self.n * len(ENV_FIELDS))
        return raw.reshape(self.n, len(ENV_FIELDS)).T.copy(), self.t

    def set_state(self, soa, t):
        soa = np.ascontiguousarray(np.asarray(soa, dtype=np.int32))
        assert soa.shape == (len(ENV_FIELDS), self.n)
        aos = np.ascontiguousarray(soa.T)
        ctypes.memmove(self.envs, aos.ctypes.data, aos.nbytes)
        self.t = int(t)
