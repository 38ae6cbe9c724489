"""ctypes wrapper of the CartPole CPU oracle -- TEST INFRASTRUCTURE (see the
header of cartpole_oracle.c).  Only tests, the smoke check and the CPU-baseline
timing of the benchmark may import it."""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cartpole_oracle.c")
_LIB = os.path.join(_HERE, "libcartpole_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Env(ctypes.Structure):
    _fields_ = [("x", ctypes.c_float), ("xd", ctypes.c_float), ("th", ctypes.c_float),
                ("thd", ctypes.c_float), ("steps", ctypes.c_int32), ("episode", ctypes.c_int32)]


class _Stats(ctypes.Structure):
    _fields_ = [("episodes", ctypes.c_int64), ("sum_length", ctypes.c_int64)]


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            u32, u64, i32, vp, f32 = (ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int,
                                      ctypes.c_void_p, ctypes.c_float)
            L.cp_oracle_sin.argtypes = [f32]
            L.cp_oracle_sin.restype = f32
            L.cp_oracle_cos.argtypes = [f32]
            L.cp_oracle_cos.restype = f32
            L.cp_oracle_action.argtypes = [u64, u32, u64]
            L.cp_oracle_action.restype = i32
            L.cp_oracle_reset_env.argtypes = [vp, u64, u32, u32]
            L.cp_oracle_reset_env.restype = None
            L.cp_oracle_step.argtypes = [vp, i32, u64, u32, vp]
            L.cp_oracle_step.restype = i32
            L.cp_oracle_reset.argtypes = [vp, i32, u64, u32]
            L.cp_oracle_reset.restype = None
            L.cp_oracle_obs.argtypes = [vp, i32, vp]
            L.cp_oracle_obs.restype = None
            L.cp_oracle_rollout.argtypes = [vp, i32, u64, u32, u64, i32, i32, vp, vp, vp, vp, vp]
            L.cp_oracle_rollout.restype = i32
            L.cp_oracle_sizeof_env.restype = i32
            assert L.cp_oracle_sizeof_env() == ctypes.sizeof(_Env)
            _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def poly_sin(th):
    return float(lib().cp_oracle_sin(float(th)))


def poly_cos(th):
    return float(lib().cp_oracle_cos(float(th)))


def action(seed, env_id, t):
    return int(lib().cp_oracle_action(seed, env_id, t))


class Env:
    """One env, for unit tests of single steps."""

    def __init__(self, x=0.0, xd=0.0, th=0.0, thd=0.0, steps=0, episode=0):
        self.c = _Env(x, xd, th, thd, steps, episode)

    def reset(self, seed, env_id, episode):
        lib().cp_oracle_reset_env(ctypes.byref(self.c), seed, env_id, episode)
        return self

    def step(self, a, seed=0, env_id=0, stats=None):
        st = stats if stats is not None else _Stats()
        return int(lib().cp_oracle_step(ctypes.byref(self.c), int(a), seed, env_id, ctypes.byref(st)))

    def state(self):
        return (np.float32(self.c.x), np.float32(self.c.xd), np.float32(self.c.th),
                np.float32(self.c.thd))

    def as_tuple(self):
        return (self.c.x, self.c.xd, self.c.th, self.c.thd, self.c.steps, self.c.episode)


def new_stats():
    return _Stats()


class OracleCartPole:
    """Batch of envs with the call surface of the CUDA library's handle."""

    def __init__(self, n_envs, seed, env_id_base=0):
        self.n = int(n_envs)
        self.seed = int(seed) & 0xFFFFFFFFFFFFFFFF
        self.env_id_base = int(env_id_base)
        self.envs = (_Env * max(self.n, 1))()
        self.stats = _Stats()
        self.t = 0
        self.reset()

    def reset(self):
        lib().cp_oracle_reset(self.envs, self.n, self.seed, self.env_id_base)
        self.stats = _Stats()
        self.t = 0
        obs = np.zeros((self.n, 4), dtype=np.float32)
        lib().cp_oracle_obs(self.envs, self.n, _ptr(obs))
        return obs

    def rollout(self, T, action_mode=0, actions=None):
        T, n = int(T), self.n
        obs = np.zeros((T, n, 4), dtype=np.float32)
        reward = np.zeros((T, n), dtype=np.float32)
        done = np.zeros((T, n), dtype=np.uint8)
        act = None
        if action_mode == 2:
            act = np.ascontiguousarray(actions, dtype=np.uint8).reshape(T, n)
        elif action_mode == 3:
            act = np.array([int(actions)], dtype=np.uint8)
        rc = lib().cp_oracle_rollout(self.envs, n, self.seed, self.env_id_base, self.t, T,
                                     action_mode, _ptr(act), _ptr(obs), _ptr(reward), _ptr(done),
                                     ctypes.byref(self.stats))
        if rc != 0:
            raise ValueError("cp_oracle_rollout: bad arguments")
        self.t += T
        return obs, reward, done

    def step(self, actions):
        obs, reward, done = self.rollout(1, 2, np.asarray(actions).reshape(1, self.n))
        return obs[0], reward[0], done[0]

    def episode_stats(self, clear=False):
        s = (int(self.stats.episodes), int(self.stats.sum_length))
        if clear:
            self.stats = _Stats()
        return s

    def get_state(self):
        """(float32 [4, n] x / xd / th / thd, int32 [2, n] steps / episode, t)."""
        raw = np.frombuffer(self.envs, dtype=np.uint8, count=self.n * ctypes.sizeof(_Env))
        rec = raw.view(np.dtype([("f", np.float32, 4), ("i", np.int32, 2)]))
        return rec["f"].T.copy(), rec["i"].T.copy(), self.t

    def set_state(self, fstate, istate, t):
        rec = np.zeros(self.n, dtype=np.dtype([("f", np.float32, 4), ("i", np.int32, 2)]))
        rec["f"] = np.asarray(fstate, dtype=np.float32).T
        rec["i"] = np.asarray(istate, dtype=np.int32).T
        ctypes.memmove(self.envs, rec.ctypes.data, rec.nbytes)
        self.t = int(t)
