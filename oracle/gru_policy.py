"""ctypes wrapper of the GRU-policy CPU oracle -- TEST INFRASTRUCTURE (see the
header of gru_policy_oracle.c).  Only tests, the smoke check and the CPU-baseline
timing of the benchmark may import it."""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gru_policy_oracle.c")
_LIB = os.path.join(_HERE, "libgru_policy_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            vp, i32, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
            L.gp_oracle_bf16_round.argtypes = [f32]
            L.gp_oracle_bf16_round.restype = f32
            L.gp_oracle_bf16_round_f64.argtypes = [vp, vp, ctypes.c_size_t]
            L.gp_oracle_bf16_round_f64.restype = None
            L.gp_oracle_encode.argtypes = [vp, i32, i32, i32, vp, vp, vp]
            L.gp_oracle_encode.restype = None
            L.gp_oracle_cell.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp, vp, vp]
            L.gp_oracle_cell.restype = None
            L.gp_oracle_head.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
            L.gp_oracle_head.restype = None
            _lib = L
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def bf16_round(v: float) -> float:
    return float(lib().gp_oracle_bf16_round(float(np.float32(v))))


def bf16_round_f64(a) -> np.ndarray:
    """float32 array of the bfloat16 values nearest to the float64 array a."""
    a = np.ascontiguousarray(a, dtype=np.float64)
    out = np.empty(a.shape, dtype=np.float32)
    lib().gp_oracle_bf16_round_f64(a.ctypes.data, out.ctypes.data, a.size)
    return out


def encode(obs, enc_w, enc_b) -> np.ndarray:
    """float32 [n, H] holding bfloat16 values."""
    obs, enc_w, enc_b = _f32(obs), _f32(enc_w), _f32(enc_b)
    n, d = obs.shape
    H = enc_w.shape[0]
    assert enc_w.shape == (H, d) and enc_b.shape == (H,)
    out = np.empty((n, H), dtype=np.float32)
    lib().gp_oracle_encode(obs.ctypes.data, n, d, H, enc_w.ctypes.data, enc_b.ctypes.data,
                           out.ctypes.data)
    return out


def cell(x, h, w_ih, w_hh, b_ih, b_hh, with_abs_sum: bool = False):
    """float64 [n, H] new hidden state (not rounded); with_abs_sum also returns
    the per-output sum of |products| of the six dot products."""
    x, h, w_ih, w_hh, b_ih, b_hh = map(_f32, (x, h, w_ih, w_hh, b_ih, b_hh))
    n, H = x.shape
    assert h.shape == (n, H) and w_ih.shape == (3 * H, H) and w_hh.shape == (3 * H, H)
    assert b_ih.shape == (3 * H,) and b_hh.shape == (3 * H,)
    out = np.empty((n, H), dtype=np.float64)
    t = np.empty((n, H), dtype=np.float64) if with_abs_sum else None
    lib().gp_oracle_cell(x.ctypes.data, h.ctypes.data, n, H, w_ih.ctypes.data, w_hh.ctypes.data,
                         b_ih.ctypes.data, b_hh.ctypes.data, out.ctypes.data,
                         t.ctypes.data if with_abs_sum else None)
    return (out, t) if with_abs_sum else out


def head(h, head_w, head_b, with_abs_sum: bool = False):
    """float64 [n, A] logits W_o h + b_o; with_abs_sum also returns |b_o| + sum |h w| per logit."""
    h, head_w, head_b = _f32(h), _f32(head_w), _f32(head_b)
    n, H = h.shape
    A = head_w.shape[0]
    assert head_w.shape == (A, H) and head_b.shape == (A,)
    out = np.empty((n, A), dtype=np.float64)
    t = np.empty((n, A), dtype=np.float64) if with_abs_sum else None
    lib().gp_oracle_head(h.ctypes.data, n, H, A, head_w.ctypes.data, head_b.ctypes.data,
                         out.ctypes.data, t.ctypes.data if with_abs_sum else None)
    return (out, t) if with_abs_sum else out
