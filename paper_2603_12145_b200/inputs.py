"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the environment's arithmetic: it only draws numbers
(numpy's PCG64) that both the CUDA library and the CPU oracle are then fed.
"""
from __future__ import annotations

import numpy as np

# Field order of the unpacked state, as exchanged by get_state / set_state.
STATE_FIELDS = ("bx", "by", "vx", "vy", "apy", "opy", "score_a", "score_o",
                "ep_len", "episode", "prev_action")


def explicit_actions(T: int, n_envs: int, seed: int, repeat_fraction: float = 0.0,
                     odd_codes: bool = False) -> np.ndarray:
    """uint8 [T, n_envs] action bytes: uniform on {0,1,2}; a fraction carries
    bit 2 ("repeat the previous action"); with odd_codes some bytes use the
    spare code 3."""
    rng = np.random.Generator(np.random.PCG64(seed))
    a = rng.integers(0, 4 if odd_codes else 3, size=(T, n_envs), dtype=np.uint8)
    if repeat_fraction > 0.0:
        rep = rng.random((T, n_envs)) < repeat_fraction
        a = np.where(rep, a | np.uint8(4), a).astype(np.uint8)
    return a


def random_states(n_envs: int, seed: int, near_end: bool = False) -> np.ndarray:
    """int32 [11, n_envs] states drawn inside the legal ranges of every field
    (ball inside the court, paddles clamped, speeds within their caps).  With
    near_end the scores and frame counts sit close to the episode limits so
    that auto-resets happen within a few steps."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n = n_envs
    s = np.zeros((len(STATE_FIELDS), n), dtype=np.int32)
    s[0] = rng.integers(0, 40961, n)                       # bx
    s[1] = rng.integers(0, 48641, n)                       # by
    s[2] = rng.integers(512, 1025, n) * rng.choice([-1, 1], n)  # vx
    s[3] = rng.integers(-768, 769, n)                      # vy
    s[4] = rng.integers(0, 45057, n)                       # apy
    s[5] = rng.integers(0, 45057, n)                       # opy
    if near_end:
        s[6] = rng.integers(15, 21, n)
        s[7] = rng.integers(15, 21, n)
        s[8] = rng.integers(9950, 10000, n)
    else:
        s[6] = rng.integers(0, 21, n)
        s[7] = rng.integers(0, 21, n)
        s[8] = rng.integers(0, 10000, n)
    s[9] = rng.integers(0, 1000, n)                        # episode
    s[10] = rng.integers(0, 3, n)                          # prev_action
    return s


def policy_weights(hidden: int, seed: int, obs_dim: int = 6, n_actions: int = 3) -> dict:
    """float32 parameters of the GRU policy, rows = output units, gate blocks in
    the order r, z, n.  Every matrix entry is an integer / 2048 with at most
    seven significant bits, so it is exactly representable in bfloat16 and both
    the tensor-core path and the CPU oracle see the same numbers; the range
    matches the usual 1 / sqrt(hidden) initialisation at hidden = 576."""
    rng = np.random.Generator(np.random.PCG64(seed))
    H = hidden

    def m(*shape):
        return (rng.integers(-85, 86, size=shape).astype(np.float32) / np.float32(2048.0))

    return {
        "enc_w": (rng.integers(-96, 97, size=(H, obs_dim)).astype(np.float32) / np.float32(64.0)),
        "enc_b": m(H),
        "w_ih": m(3 * H, H), "w_hh": m(3 * H, H), "b_ih": m(3 * H), "b_hh": m(3 * H),
        "head_w": (rng.integers(-96, 97, size=(n_actions, H)).astype(np.float32)
                   / np.float32(512.0)),
        "head_b": m(n_actions),
    }


def policy_activations(n_envs: int, hidden: int, seed: int):
    """(x, h): float32 [n_envs, hidden] each, bfloat16-representable values; x is
    non-negative like an encoder output after its rectifier, h lies in (-1, 1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.integers(0, 128, size=(n_envs, hidden)).astype(np.float32) / np.float32(64.0)
    h = rng.integers(-127, 128, size=(n_envs, hidden)).astype(np.float32) / np.float32(128.0)
    return x, h


def bf16_values(shape, seed: int, min_exp: int = -6, max_exp: int = 0) -> np.ndarray:
    """float32 array of random bfloat16-representable values +-(1 + m/128) * 2^e,
    m uniform on 0..127 and e uniform on min_exp..max_exp, assembled from the bit
    fields (no rounding involved)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    sign = rng.integers(0, 2, size=shape, dtype=np.uint32) << np.uint32(31)
    expo = (rng.integers(min_exp, max_exp + 1, size=shape) + 127).astype(np.uint32) << np.uint32(23)
    mant = rng.integers(0, 128, size=shape, dtype=np.uint32) << np.uint32(16)
    return (sign | expo | mant).view(np.float32)
