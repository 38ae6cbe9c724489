"""ctypes binding of libpong_b200.so: the same entry points as include/pong.h.

Argument marshalling only.  Device buffers are torch tensors (torch is used
for device memory and streams, nothing else); every step of the environment
runs in the library's CUDA kernels.  There is no CPU path: loading fails
loudly if the library has not been built, and creating a handle fails if no
CUDA device is usable.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

from . import build as _build

OBS_VECTOR, OBS_PIXELS = 0, 1
ACT_PHILOX, ACT_STICKY, ACT_EXPLICIT, ACT_CONSTANT = 0, 1, 2, 3
STATE_FIELDS = 11
FRAME_BYTES = 84 * 84

EXPORTS = ("pong_create", "pong_create_ex", "pong_destroy", "pong_set_stream", "pong_reset",
           "pong_step", "pong_rollout", "pong_rollout_host", "pong_fill_actions",
           "pong_episode_stats", "pong_get_state", "pong_set_state", "pong_num_envs",
           "pong_launch_count", "pong_strerror", "pong_rollout_static", "pong_fill_words",
           "pong_sample_actions", "pong_get_step_counter", "pong_set_step_counter",
           "pong_set_vector_path", "pong_measure_alu_rate")
PATH_AUTO, PATH_GENERAL, PATH_TMA, PATH_CHAINS = 0, 1, 2, 3
STATIC_MAX_ENVS = 65536


class PongError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (code %d)" % (where, strerror(code), code))


class _Config(ctypes.Structure):
    _fields_ = [("obs_mode", ctypes.c_int), ("frameskip", ctypes.c_int),
                ("env_id_base", ctypes.c_int)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = False):
    """Load libpong_b200.so.  Raises if it is missing (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if build_if_missing:
        _build.build()
    if not os.path.exists(path):
        raise ImportError(
            "CUDA library %s is not built; run `python -m paper_2603_12145_b200.build` "
            "(needs nvcc). There is no CPU fallback." % path)
    L = ctypes.CDLL(path)
    vp, i32, u64, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64, ctypes.c_int64
    L.pong_create.argtypes = [ctypes.POINTER(vp), i32, u64]
    L.pong_create_ex.argtypes = [ctypes.POINTER(vp), i32, u64, ctypes.POINTER(_Config)]
    L.pong_destroy.argtypes = [vp]
    L.pong_set_stream.argtypes = [vp, vp]
    L.pong_set_vector_path.argtypes = [vp, i32]
    L.pong_measure_alu_rate.argtypes = [vp, ctypes.POINTER(ctypes.c_double)]
    L.pong_reset.argtypes = [vp, vp]
    L.pong_step.argtypes = [vp, vp, vp, vp, vp]
    L.pong_rollout.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.pong_rollout_host.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.pong_fill_actions.argtypes = [vp, i32, i32, vp]
    L.pong_fill_words.argtypes = [vp, i32, vp]
    L.pong_sample_actions.argtypes = [vp, vp, vp, vp]
    L.pong_get_step_counter.argtypes = [vp, ctypes.POINTER(u64)]
    L.pong_set_step_counter.argtypes = [vp, u64]
    L.pong_episode_stats.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64),
                                     ctypes.POINTER(i64), i32]
    L.pong_get_state.argtypes = [vp, vp, ctypes.POINTER(u64)]
    L.pong_set_state.argtypes = [vp, vp, u64]
    L.pong_num_envs.argtypes = [vp]
    L.pong_launch_count.argtypes = [vp]
    L.pong_launch_count.restype = i64
    L.pong_rollout_static.argtypes = [i32, u64, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    L.pong_strerror.argtypes = [i32]
    L.pong_strerror.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("pong_launch_count", "pong_strerror"):
            getattr(L, name).restype = i32
    _lib = L
    return L


def strerror(code: int) -> str:
    return load().pong_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise PongError(code, where)


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array, or an integer address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


# ---- the C entry points under their own names ------------------------------------

def pong_create(n_envs: int, seed: int) -> int:
    h = ctypes.c_void_p()
    _check(load().pong_create(ctypes.byref(h), int(n_envs), int(seed) & (2**64 - 1)), "pong_create")
    return h.value


def pong_create_ex(n_envs: int, seed: int, obs_mode: int = 0, frameskip: int = 1,
                   env_id_base: int = 0) -> int:
    h = ctypes.c_void_p()
    cfg = _Config(int(obs_mode), int(frameskip), int(env_id_base))
    _check(load().pong_create_ex(ctypes.byref(h), int(n_envs), int(seed) & (2**64 - 1),
                                 ctypes.byref(cfg)), "pong_create_ex")
    return h.value


def pong_destroy(h: int) -> None:
    _check(load().pong_destroy(h), "pong_destroy")


def pong_set_stream(h: int, cuda_stream: int) -> None:
    _check(load().pong_set_stream(h, cuda_stream), "pong_set_stream")


def pong_set_vector_path(h: int, path: int) -> None:
    _check(load().pong_set_vector_path(h, int(path)), "pong_set_vector_path")


def pong_measure_alu_rate(cuda_stream: Optional[int] = None) -> float:
    """Integer-ALU warp instructions per second the current device sustains."""
    out = ctypes.c_double(0.0)
    _check(load().pong_measure_alu_rate(cuda_stream, ctypes.byref(out)), "pong_measure_alu_rate")
    return out.value


def pong_reset(h: int, obs_out=None) -> None:
    _check(load().pong_reset(h, _ptr(obs_out)), "pong_reset")


def pong_step(h: int, actions, obs, reward, done) -> None:
    _check(load().pong_step(h, _ptr(actions), _ptr(obs), _ptr(reward), _ptr(done)), "pong_step")


def pong_rollout(h: int, T: int, action_mode: int, actions, obs_buf, reward_buf, done_buf) -> None:
    keep = None
    if action_mode == ACT_CONSTANT and not isinstance(actions, np.ndarray):
        keep = np.array([int(actions)], dtype=np.uint8)
        actions = keep
    _check(load().pong_rollout(h, int(T), int(action_mode), _ptr(actions), _ptr(obs_buf),
                               _ptr(reward_buf), _ptr(done_buf)), "pong_rollout")


def pong_rollout_host(h: int, T: int, action_mode: int, actions_host, obs_host, reward_host,
                      done_host) -> None:
    keep = None
    if action_mode == ACT_CONSTANT and not isinstance(actions_host, np.ndarray):
        keep = np.array([int(actions_host)], dtype=np.uint8)
        actions_host = keep
    _check(load().pong_rollout_host(h, int(T), int(action_mode), _ptr(actions_host),
                                    _ptr(obs_host), _ptr(reward_host), _ptr(done_host)),
           "pong_rollout_host")


def pong_fill_actions(h: int, T: int, sticky: int, actions_out) -> None:
    _check(load().pong_fill_actions(h, int(T), int(sticky), _ptr(actions_out)), "pong_fill_actions")


def pong_fill_words(h: int, T: int, words_out) -> None:
    _check(load().pong_fill_words(h, int(T), _ptr(words_out)), "pong_fill_words")


def pong_sample_actions(h: int, logits, words, actions_out) -> None:
    _check(load().pong_sample_actions(h, _ptr(logits), _ptr(words), _ptr(actions_out)),
           "pong_sample_actions")


def pong_get_step_counter(h: int) -> int:
    t = ctypes.c_uint64()
    _check(load().pong_get_step_counter(h, ctypes.byref(t)), "pong_get_step_counter")
    return int(t.value)


def pong_set_step_counter(h: int, t: int) -> None:
    _check(load().pong_set_step_counter(h, int(t)), "pong_set_step_counter")


def pong_episode_stats(h: int, clear: bool = False) -> Tuple[int, int, int]:
    e, r, l = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(load().pong_episode_stats(h, ctypes.byref(e), ctypes.byref(r), ctypes.byref(l),
                                     1 if clear else 0), "pong_episode_stats")
    return int(e.value), int(r.value), int(l.value)


def pong_get_state(h: int) -> Tuple[np.ndarray, int]:
    n = load().pong_num_envs(h)
    soa = np.zeros((STATE_FIELDS, n), dtype=np.int32)
    t = ctypes.c_uint64()
    _check(load().pong_get_state(h, soa.ctypes.data, ctypes.byref(t)), "pong_get_state")
    return soa, int(t.value)


def pong_set_state(h: int, soa: np.ndarray, t: int) -> None:
    n = load().pong_num_envs(h)
    soa = np.ascontiguousarray(soa, dtype=np.int32)
    if soa.shape != (STATE_FIELDS, n):
        raise ValueError("state must be int32 [%d, %d]" % (STATE_FIELDS, n))
    _check(load().pong_set_state(h, soa.ctypes.data, int(t)), "pong_set_state")


def pong_rollout_static(n_envs: int, seed: int, env_id_base: int, T: int, action_mode: int,
                        actions, obs_buf, reward_buf, done_buf, stats_out=None,
                        cuda_stream: Optional[int] = None) -> None:
    """Reset + rollout without any allocation inside the library: the env state
    lives in a fixed device array of the library (at most STATIC_MAX_ENVS envs).
    For hosts that may not call cudaMalloc while running.  Calls that overlap
    on the GPU race on that array."""
    keep = None
    if action_mode == ACT_CONSTANT and not isinstance(actions, np.ndarray):
        keep = np.array([int(actions)], dtype=np.uint8)
        actions = keep
    _check(load().pong_rollout_static(int(n_envs), int(seed) & (2**64 - 1), int(env_id_base), int(T),
                                      int(action_mode), _ptr(actions), _ptr(obs_buf),
                                      _ptr(reward_buf), _ptr(done_buf), _ptr(stats_out),
                                      cuda_stream), "pong_rollout_static")


def pong_num_envs(h: int) -> int:
    return int(load().pong_num_envs(h))


def pong_launch_count(h: int) -> int:
    return int(load().pong_launch_count(h))


# ---- convenience wrapper: allocates output tensors with torch --------------------

class PongEnv:
    """Owns a handle plus (optionally) torch output tensors.  Every call runs
    on torch's current CUDA stream."""

    device_actions = True  # explicit action buffers must be device tensors

    def __init__(self, n_envs: int, seed: int, obs_mode: int = OBS_VECTOR, frameskip: int = 1,
                 env_id_base: int = 0, device: Optional[str] = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("PongEnv needs a CUDA device; there is no CPU fallback")
        self.torch = torch
        self.device = torch.device(device or "cuda:%d" % torch.cuda.current_device())
        self.n = int(n_envs)
        self.obs_mode = int(obs_mode)
        self.frameskip = int(frameskip)
        with torch.cuda.device(self.device):
            self.h = pong_create_ex(n_envs, seed, obs_mode, frameskip, env_id_base)
        self.ring = None
        if self.obs_mode == OBS_PIXELS:
            self.ring = torch.zeros((self.n, 4, 84, 84), dtype=torch.uint8, device=self.device)
            self.reset()

    def _stream(self):
        pong_set_stream(self.h, self.torch.cuda.current_stream(self.device).cuda_stream)

    def set_vector_path(self, path: int):
        pong_set_vector_path(self.h, path)

    def close(self):
        if getattr(self, "h", None):
            pong_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        self._stream()
        if self.obs_mode == OBS_VECTOR:
            obs = self.torch.empty((self.n, 6), dtype=self.torch.float32, device=self.device)
            pong_reset(self.h, obs)
            return obs
        pong_reset(self.h, self.ring)
        return self.ring

    def _outputs(self, T, obs, reward, done, lead=True):
        t = self.torch
        shape = (T, self.n) if lead else (self.n,)
        if obs is None:
            obs = self.ring if self.obs_mode == OBS_PIXELS else \
                t.empty(shape + (6,), dtype=t.float32, device=self.device)
        if reward is None:
            reward = t.empty(shape, dtype=t.float32, device=self.device)
        if done is None:
            done = t.empty(shape, dtype=t.uint8, device=self.device)
        return obs, reward, done

    def step(self, actions, obs=None, reward=None, done=None):
        self._stream()
        obs, reward, done = self._outputs(1, obs, reward, done, lead=False)
        pong_step(self.h, actions, obs, reward, done)
        return obs, reward, done

    def rollout(self, T, action_mode=ACT_PHILOX, actions=None, obs=None, reward=None, done=None):
        self._stream()
        obs, reward, done = self._outputs(int(T), obs, reward, done)
        pong_rollout(self.h, T, action_mode, actions, obs, reward, done)
        return obs, reward, done

    def fill_actions(self, T, sticky=0, out=None):
        self._stream()
        if out is None:
            out = self.torch.empty((int(T), self.n), dtype=self.torch.uint8, device=self.device)
        pong_fill_actions(self.h, T, sticky, out)
        return out

    def fill_words(self, T, out=None):
        self._stream()
        if out is None:
            out = self.torch.empty((int(T), self.n), dtype=self.torch.int32, device=self.device)
        pong_fill_words(self.h, T, out)
        return out

    def sample_actions(self, logits, words, out=None):
        self._stream()
        if out is None:
            out = self.torch.empty((self.n,), dtype=self.torch.uint8, device=self.device)
        pong_sample_actions(self.h, logits, words, out)
        return out

    @property
    def t(self):
        return pong_get_step_counter(self.h)

    @t.setter
    def t(self, value):
        pong_set_step_counter(self.h, value)

    def episode_stats(self, clear=False):
        self._stream()
        return pong_episode_stats(self.h, clear)

    def get_state(self):
        self._stream()
        return pong_get_state(self.h)

    def set_state(self, soa, t):
        self._stream()
        pong_set_state(self.h, soa, t)

    @property
    def launches(self):
        return pong_launch_count(self.h)
