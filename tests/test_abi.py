"""The C-ABI library builds, loads and exports every symbol the header
declares (no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2603_12145_b200 import build, pong

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols(header="pong.h", prefix="pong"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(%s_[a-z_]+)\s*\(" % prefix, text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(pong.EXPORTS)


def test_strerror_and_null_handles_without_gpu():
    L = pong.load(build_if_missing=True)
    assert pong.strerror(0) == "ok"
    for code in range(-6, 0):
        assert pong.strerror(code) != "unknown error code"
    assert pong.strerror(-99) == "unknown error code"
    # NULL handle / NULL out-pointer are rejected before any CUDA call
    assert L.pong_reset(None, None) == -2
    assert L.pong_step(None, None, None, None, None) == -2
    assert L.pong_rollout(None, 1, 0, None, None, None, None) == -2
    assert L.pong_fill_actions(None, 1, 0, None) == -2
    assert L.pong_episode_stats(None, None, None, None, 0) == -2
    assert L.pong_get_state(None, None, None) == -2
    assert L.pong_set_state(None, None, 0) == -2
    assert L.pong_set_stream(None, None) == -2
    assert L.pong_destroy(None) == 0
    assert L.pong_create(None, 4, 0) == -2
    h = ctypes.c_void_p()
    assert L.pong_create(ctypes.byref(h), 0, 0) == -1
    cfg = pong._Config(2, 1, 0)
    assert L.pong_create_ex(ctypes.byref(h), 4, 0, ctypes.byref(cfg)) == -1
    cfg = pong._Config(0, 17, 0)
    assert L.pong_create_ex(ctypes.byref(h), 4, 0, ctypes.byref(cfg)) == -1
    cfg = pong._Config(0, 1, -1)
    assert L.pong_create_ex(ctypes.byref(h), 4, 0, ctypes.byref(cfg)) == -1


def test_no_cpu_fallback_without_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises((pong.PongError, RuntimeError)):
        pong.PongEnv(4, 0)
    with pytest.raises(pong.PongError) as ei:
        pong.pong_create(4, 0)
    assert ei.value.code == -4


def test_cartpole_library_exports_every_declared_symbol():
    from paper_2603_12145_b200 import cartpole
    lib = ctypes.CDLL(build.build_one("libcartpole_b200.so"))
    names = declared_symbols("cartpole.h", "cartpole")
    assert len(names) >= 13
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(cartpole.EXPORTS)
    L = cartpole.load(build_if_missing=True)
    assert cartpole.strerror(0) == "ok" and cartpole.strerror(-99) == "unknown error code"
    assert L.cartpole_reset(None, None) == -2 and L.cartpole_destroy(None) == 0
    h = ctypes.c_void_p()
    assert L.cartpole_create(ctypes.byref(h), 0, 0, 0) == -1
    assert L.cartpole_create(ctypes.byref(h), 4, 0, -1) == -1
    assert L.cartpole_create(None, 4, 0, 0) == -2


def test_gru_policy_library_exports_every_declared_symbol():
    from paper_2603_12145_b200 import gru_policy
    lib = ctypes.CDLL(build.build_one("libgru_policy_b200.so"))
    names = declared_symbols("gru_policy.h", "gru_policy")
    assert len(names) >= 10
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(gru_policy.EXPORTS)
    L = gru_policy.load(build_if_missing=True)
    assert gru_policy.strerror(0) == "ok" and gru_policy.strerror(-6).startswith("a kernel gave up")
    # argument checks that run before any CUDA call
    assert L.gru_policy_create(None, 64, 6, 3, *([None] * 8)) == -2
    h = ctypes.c_void_p()
    assert L.gru_policy_create(ctypes.byref(h), 64, 6, 3, *([None] * 8)) == -2
    assert L.gru_policy_destroy(None) == -2 and L.gru_policy_status(None) == -2
    assert L.gru_policy_cell(None, None, None, None, 1) == -2
