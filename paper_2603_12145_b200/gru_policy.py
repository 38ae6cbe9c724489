"""ctypes binding of libgru_policy_b200.so: the entry points of
include/gru_policy.h under their own names, plus a small wrapper that owns the
handle and allocates output tensors with torch.  Argument marshalling only; no
CPU path."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

from . import build as _build

EXPORTS = ("gru_policy_create", "gru_policy_destroy", "gru_policy_set_stream", "gru_policy_encode",
           "gru_policy_cell", "gru_policy_head", "gru_policy_workspace_bytes", "gru_policy_cell_head",
           "gru_policy_status", "gru_policy_hidden", "gru_policy_launch_count", "gru_policy_strerror")

PARAMETERS = ("enc_w", "enc_b", "w_ih", "w_hh", "b_ih", "b_hh", "head_w", "head_b")


class GruPolicyError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (code %d)" % (where, strerror(code), code))


_lib = None


def load(build_if_missing: bool = False):
    """Load libgru_policy_b200.so.  Raises if it is missing (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.GRU_POLICY_LIB
    if build_if_missing:
        _build.build_one("libgru_policy_b200.so")
    if not os.path.exists(path):
        raise ImportError("CUDA library %s is not built; run `python -m paper_2603_12145_b200.build`"
                          " (needs nvcc). There is no CPU fallback." % path)
    L = ctypes.CDLL(path)
    vp, i32 = ctypes.c_void_p, ctypes.c_int
    L.gru_policy_create.argtypes = [ctypes.POINTER(vp), i32, i32, i32] + [vp] * 8
    L.gru_policy_destroy.argtypes = [vp]
    L.gru_policy_set_stream.argtypes = [vp, vp]
    L.gru_policy_encode.argtypes = [vp, vp, vp, vp, vp, i32]
    L.gru_policy_cell.argtypes = [vp, vp, vp, vp, i32]
    L.gru_policy_head.argtypes = [vp, vp, vp, i32]
    L.gru_policy_workspace_bytes.argtypes = [vp, i32]
    L.gru_policy_workspace_bytes.restype = ctypes.c_size_t
    L.gru_policy_cell_head.argtypes = [vp, vp, vp, vp, vp, vp, i32]
    L.gru_policy_status.argtypes = [vp]
    L.gru_policy_hidden.argtypes = [vp]
    L.gru_policy_launch_count.argtypes = [vp]
    L.gru_policy_launch_count.restype = ctypes.c_int64
    L.gru_policy_strerror.argtypes = [i32]
    L.gru_policy_strerror.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("gru_policy_launch_count", "gru_policy_strerror", "gru_policy_workspace_bytes"):
            getattr(L, name).restype = i32
    _lib = L
    return L


def strerror(code: int) -> str:
    return load().gru_policy_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise GruPolicyError(code, where)


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


# ---- the C entry points under their own names ------------------------------------

def gru_policy_create(hidden: int, obs_dim: int, n_actions: int, params: dict) -> int:
    """params: the eight host float32 arrays of PARAMETERS."""
    arrays = [np.ascontiguousarray(params[k], dtype=np.float32) for k in PARAMETERS]
    h = ctypes.c_void_p()
    _check(load().gru_policy_create(ctypes.byref(h), int(hidden), int(obs_dim), int(n_actions),
                                    *[a.ctypes.data for a in arrays]), "gru_policy_create")
    return h.value


def gru_policy_destroy(h: int) -> None:
    _check(load().gru_policy_destroy(h), "gru_policy_destroy")


def gru_policy_set_stream(h: int, cuda_stream: int) -> None:
    _check(load().gru_policy_set_stream(h, cuda_stream), "gru_policy_set_stream")


def gru_policy_encode(h: int, obs, done, hidden_state, x_out, n: int) -> None:
    _check(load().gru_policy_encode(h, _ptr(obs), _ptr(done), _ptr(hidden_state), _ptr(x_out), int(n)),
           "gru_policy_encode")


def gru_policy_cell(h: int, x, h_in, h_out, n: int) -> None:
    _check(load().gru_policy_cell(h, _ptr(x), _ptr(h_in), _ptr(h_out), int(n)), "gru_policy_cell")


def gru_policy_head(h: int, hidden_state, logits, n: int) -> None:
    _check(load().gru_policy_head(h, _ptr(hidden_state), _ptr(logits), int(n)), "gru_policy_head")


def gru_policy_workspace_bytes(h: int, n: int) -> int:
    return int(load().gru_policy_workspace_bytes(h, int(n)))


def gru_policy_cell_head(h: int, x, h_in, h_out, logits, workspace, n: int) -> None:
    _check(load().gru_policy_cell_head(h, _ptr(x), _ptr(h_in), _ptr(h_out), _ptr(logits), _ptr(workspace),
                                       int(n)), "gru_policy_cell_head")


def gru_policy_status(h: int) -> None:
    _check(load().gru_policy_status(h), "gru_policy_status")


def gru_policy_hidden(h: int) -> int:
    return int(load().gru_policy_hidden(h))


def gru_policy_launch_count(h: int) -> int:
    return int(load().gru_policy_launch_count(h))


# ---- a small owner of the handle ----------------------------------------------------

class GruPolicy:
    """The policy's parameters on the device.  Tensors are torch CUDA tensors:
    obs float32 [n, obs_dim], x and h bfloat16 [n, hidden], logits float32
    [n, n_actions]."""

    def __init__(self, params: dict, device: str = "cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.hidden, self.obs_dim = (int(v) for v in np.asarray(params["enc_w"]).shape)
        self.n_actions = int(np.asarray(params["head_w"]).shape[0])
        with torch.cuda.device(self.device):
            self.h = gru_policy_create(self.hidden, self.obs_dim, self.n_actions, params)

    def close(self):
        if getattr(self, "h", None):
            with self.torch.cuda.device(self.device):
                gru_policy_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self):
        gru_policy_set_stream(self.h, self.torch.cuda.current_stream(self.device).cuda_stream)

    @property
    def launches(self) -> int:
        return gru_policy_launch_count(self.h)

    def encode(self, obs, x_out=None, done=None, hidden_state=None):
        t = self.torch
        n = obs.shape[0]
        if x_out is None:
            x_out = t.empty((n, self.hidden), dtype=t.bfloat16, device=self.device)
        self._stream()
        gru_policy_encode(self.h, obs, done, hidden_state, x_out, n)
        return x_out

    def cell(self, x, h_in, h_out=None):
        t = self.torch
        n = x.shape[0]
        if h_out is None:
            h_out = t.empty((n, self.hidden), dtype=t.bfloat16, device=self.device)
        self._stream()
        gru_policy_cell(self.h, x, h_in, h_out, n)
        return h_out

    def workspace(self, n: int):
        """Device scratch for cell_head at n envs."""
        t = self.torch
        return t.empty((gru_policy_workspace_bytes(self.h, n),), dtype=t.uint8, device=self.device)

    def cell_head(self, x, h_in, h_out=None, logits=None, workspace=None):
        """(h_out, logits): the cell and the head of its result in one pass."""
        t = self.torch
        n = x.shape[0]
        if h_out is None:
            h_out = t.empty((n, self.hidden), dtype=t.bfloat16, device=self.device)
        if logits is None:
            logits = t.empty((n, self.n_actions), dtype=t.float32, device=self.device)
        if workspace is None:
            workspace = self.workspace(n)
        self._stream()
        gru_policy_cell_head(self.h, x, h_in, h_out, logits, workspace, n)
        return h_out, logits

    def head(self, hidden_state, logits=None):
        t = self.torch
        n = hidden_state.shape[0]
        if logits is None:
            logits = t.empty((n, self.n_actions), dtype=t.float32, device=self.device)
        self._stream()
        gru_policy_head(self.h, hidden_state, logits, n)
        return logits

    def status(self) -> None:
        """Synchronises; raises if a kernel gave up a wait."""
        gru_policy_status(self.h)
