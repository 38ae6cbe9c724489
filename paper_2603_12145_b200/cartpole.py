"""ctypes binding of libcartpole_b200.so: the entry points of include/cartpole.h
under their own names, plus a small wrapper that allocates output tensors with
torch.  Argument marshalling only; no CPU path."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

from . import build as _build

ACT_PHILOX, ACT_EXPLICIT, ACT_CONSTANT = 0, 2, 3

EXPORTS = ("cartpole_create", "cartpole_destroy", "cartpole_set_stream", "cartpole_reset",
           "cartpole_step", "cartpole_rollout", "cartpole_rollout_host", "cartpole_episode_stats",
           "cartpole_get_state", "cartpole_set_state", "cartpole_num_envs",
           "cartpole_launch_count", "cartpole_strerror", "cartpole_set_path")
PATH_AUTO, PATH_PLAIN, PATH_CHAINS = 0, 1, 2


class CartPoleError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (code %d)" % (where, strerror(code), code))


_lib = None


def load(build_if_missing: bool = False):
    global _lib
    if _lib is not None:
        return _lib
    path = _build.CARTPOLE_LIB
    if build_if_missing:
        _build.build_one("libcartpole_b200.so")
    if not os.path.exists(path):
        raise ImportError("CUDA library %s is not built; run `python -m paper_2603_12145_b200.build`"
                          " (needs nvcc). There is no CPU fallback." % path)
    L = ctypes.CDLL(path)
    vp, i32, u64, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64, ctypes.c_int64
    L.cartpole_create.argtypes = [ctypes.POINTER(vp), i32, u64, i32]
    L.cartpole_destroy.argtypes = [vp]
    L.cartpole_set_stream.argtypes = [vp, vp]
    L.cartpole_reset.argtypes = [vp, vp]
    L.cartpole_step.argtypes = [vp, vp, vp, vp, vp]
    L.cartpole_rollout.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.cartpole_rollout_host.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.cartpole_episode_stats.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), i32]
    L.cartpole_get_state.argtypes = [vp, vp, vp, ctypes.POINTER(u64)]
    L.cartpole_set_state.argtypes = [vp, vp, vp, u64]
    L.cartpole_num_envs.argtypes = [vp]
    L.cartpole_set_path.argtypes = [vp, i32]
    L.cartpole_launch_count.argtypes = [vp]
    L.cartpole_launch_count.restype = i64
    L.cartpole_strerror.argtypes = [i32]
    L.cartpole_strerror.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("cartpole_launch_count", "cartpole_strerror"):
            getattr(L, name).restype = i32
    _lib = L
    return L


def strerror(code: int) -> str:
    return load().cartpole_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise CartPoleError(code, where)


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def _const(actions):
    return actions if isinstance(actions, np.ndarray) else np.array([int(actions)], dtype=np.uint8)


def cartpole_create(n_envs: int, seed: int, env_id_base: int = 0) -> int:
    h = ctypes.c_void_p()
    _check(load().cartpole_create(ctypes.byref(h), int(n_envs), int(seed) & (2**64 - 1),
                                  int(env_id_base)), "cartpole_create")
    return h.value


def cartpole_destroy(h: int) -> None:
    _check(load().cartpole_destroy(h), "cartpole_destroy")


def cartpole_set_stream(h: int, cuda_stream: int) -> None:
    _check(load().cartpole_set_stream(h, cuda_stream), "cartpole_set_stream")


def cartpole_reset(h: int, obs_out=None) -> None:
    _check(load().cartpole_reset(h, _ptr(obs_out)), "cartpole_reset")


def cartpole_step(h: int, actions, obs, reward, done) -> None:
    _check(load().cartpole_step(h, _ptr(actions), _ptr(obs), _ptr(reward), _ptr(done)),
           "cartpole_step")


def cartpole_rollout(h: int, T: int, action_mode: int, actions, obs, reward, done) -> None:
    keep = _const(actions) if action_mode == ACT_CONSTANT else actions
    _check(load().cartpole_rollout(h, int(T), int(action_mode), _ptr(keep), _ptr(obs), _ptr(reward),
                                   _ptr(done)), "cartpole_rollout")


def cartpole_rollout_host(h: int, T: int, action_mode: int, actions_host, obs_host, reward_host,
                          done_host) -> None:
    keep = _const(actions_host) if action_mode == ACT_CONSTANT else actions_host
    _check(load().cartpole_rollout_host(h, int(T), int(action_mode), _ptr(keep), _ptr(obs_host),
                                        _ptr(reward_host), _ptr(done_host)), "cartpole_rollout_host")


def cartpole_episode_stats(h: int, clear: bool = False) -> Tuple[int, int]:
    e, l = ctypes.c_int64(), ctypes.c_int64()
    _check(load().cartpole_episode_stats(h, ctypes.byref(e), ctypes.byref(l), 1 if clear else 0),
           "cartpole_episode_stats")
    return int(e.value), int(l.value)


def cartpole_get_state(h: int):
    n = load().cartpole_num_envs(h)
    f = np.zeros((4, n), dtype=np.float32)
    i = np.zeros((2, n), dtype=np.int32)
    t = ctypes.c_uint64()
    _check(load().cartpole_get_state(h, f.ctypes.data, i.ctypes.data, ctypes.byref(t)),
           "cartpole_get_state")
    return f, i, int(t.value)


def cartpole_set_state(h: int, fstate, istate, t: int) -> None:
    n = load().cartpole_num_envs(h)
    f = np.ascontiguousarray(fstate, dtype=np.float32)
    i = np.ascontiguousarray(istate, dtype=np.int32)
    if f.shape != (4, n) or i.shape != (2, n):
        raise ValueError("state must be float32 [4, %d] and int32 [2, %d]" % (n, n))
    _check(load().cartpole_set_state(h, f.ctypes.data, i.ctypes.data, int(t)), "cartpole_set_state")


def cartpole_set_path(h: int, path: int) -> None:
    _check(load().cartpole_set_path(h, int(path)), "cartpole_set_path")


def cartpole_num_envs(h: int) -> int:
    return int(load().cartpole_num_envs(h))


def cartpole_launch_count(h: int) -> int:
    return int(load().cartpole_launch_count(h))


class CartPoleEnv:
    """Owns a handle; allocates output tensors with torch when none are given.
    Every call runs on torch's current CUDA stream."""

    device_actions = True

    def __init__(self, n_envs: int, seed: int, env_id_base: int = 0, device: Optional[str] = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("CartPoleEnv needs a CUDA device; there is no CPU fallback")
        self.torch = torch
        self.device = torch.device(device or "cuda:%d" % torch.cuda.current_device())
        self.n = int(n_envs)
        with torch.cuda.device(self.device):
            self.h = cartpole_create(n_envs, seed, env_id_base)

    def _stream(self):
        cartpole_set_stream(self.h, self.torch.cuda.current_stream(self.device).cuda_stream)

    def close(self):
        if getattr(self, "h", None):
            cartpole_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        self._stream()
        obs = self.torch.empty((self.n, 4), dtype=self.torch.float32, device=self.device)
        cartpole_reset(self.h, obs)
        return obs

    def _outputs(self, shape, obs, reward, done):
        t = self.torch
        if obs is None:
            obs = t.empty(shape + (4,), dtype=t.float32, device=self.device)
        if reward is None:
            reward = t.empty(shape, dtype=t.float32, device=self.device)
        if done is None:
            done = t.empty(shape, dtype=t.uint8, device=self.device)
        return obs, reward, done

    def step(self, actions, obs=None, reward=None, done=None):
        self._stream()
        obs, reward, done = self._outputs((self.n,), obs, reward, done)
        cartpole_step(self.h, actions, obs, reward, done)
        return obs, reward, done

    def rollout(self, T, action_mode=ACT_PHILOX, actions=None, obs=None, reward=None, done=None):
        self._stream()
        obs, reward, done = self._outputs((int(T), self.n), obs, reward, done)
        cartpole_rollout(self.h, T, action_mode, actions, obs, reward, done)
        return obs, reward, done

    def episode_stats(self, clear=False):
        self._stream()
        return cartpole_episode_stats(self.h, clear)

    def get_state(self):
        self._stream()
        return cartpole_get_state(self.h)

    def set_path(self, path: int):
        cartpole_set_path(self.h, path)

    def set_state(self, fstate, istate, t):
        self._stream()
        cartpole_set_state(self.h, fstate, istate, t)

    @property
    def launches(self):
        return cartpole_launch_count(self.h)
