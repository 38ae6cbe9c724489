"""Pins for the oracle's observations: vector scaling, rasteriser, frame skip
and the frame-stack ring."""
import os
import struct

import numpy as np

import oracle
from paper_2603_12145_b200.inputs import explicit_actions, random_states

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(f):
    return struct.unpack("<I", struct.pack("<f", float(f)))[0]


def test_scale_constant_and_golden_bit_patterns():
    with open(os.path.join(GOLDEN, "obs_scale_bits.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) >= 10
    for v, want in rows:
        e = oracle.Env(bx=int(v), by=0, vx=0, vy=0, apy=0, opy=0)
        assert bits(e.obs_vector()[0]) == int(want, 16), v


def test_reset_obs_bit_pattern_and_field_order():
    e = oracle.Env(bx=20224, by=24320, vx=512, vy=0, apy=22528, opy=22528)
    got = [bits(x) for x in e.obs_vector()]
    assert got == [0x3EFCCCCD, 0x3F180000, 0x3C4CCCCD, 0x00000000, 0x3F0CCCCD, 0x3F0CCCCD]
    e = oracle.Env(bx=1024, by=768, vx=-384, vy=512, apy=45056, opy=48640)
    got = [bits(x) for x in e.obs_vector()]
    assert got == [0x3CCCCCCD, 0x3C99999A, 0xBC19999A, 0x3C4CCCCD, 0x3F8CCCCD, 0x3F980000]


def test_scaling_exhaustive_against_double_precision():
    """v * C is exact in binary64 (24-bit times 24-bit significand), so one
    rounding of that product to binary32 is the correctly rounded result."""
    C = struct.unpack("<f", struct.pack("<I", 0x37CCCCCD))[0]
    vs = np.arange(-1024, 49153, dtype=np.int64)
    want = (vs.astype(np.float64) * np.float64(C)).astype(np.float32)
    got = np.zeros(len(vs), dtype=np.float32)
    e = oracle.Env()
    for k in range(0, len(vs), 6):
        chunk = [int(x) for x in vs[k:k + 6]] + [0] * 6
        e.c.bx, e.c.by, e.c.vx, e.c.vy, e.c.apy, e.c.opy = chunk[:6]
        got[k:k + 6] = e.obs_vector()[:len(vs[k:k + 6])]
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the multiply is not the division: the two differ on many integers
    div = (vs.astype(np.float64) / 40960.0).astype(np.float32)
    differ = int((div.view(np.uint32) != want.view(np.uint32)).sum())
    assert differ > 5000


def paint_then_sample(apy, opy, bx, by):
    """Independent form of the rasteriser: paint the 160x192 court, then pick
    source pixels by integer index maps."""
    court = np.zeros((192, 160), dtype=np.uint8)

    def rect(x, y, w, h):
        x0, x1 = max(x, 0), min(x + w, 160)
        y0, y1 = max(y, 0), min(y + h, 192)
        if x0 < x1 and y0 < y1:
            court[y0:y1, x0:x1] = 255

    rect(148, apy >> 8, 4, 16)
    rect(8, opy >> 8, 4, 16)
    rect(bx >> 8, by >> 8, 2, 2)
    rows = (np.arange(84) * 192) // 84
    cols = (np.arange(84) * 160) // 84
    return court[np.ix_(rows, cols)]


def test_rasteriser_against_paint_then_sample():
    rng = np.random.Generator(np.random.PCG64(5))
    cases = [(22528, 22528, 20224, 24320), (0, 45056, 0, 0), (45056, 0, 40960, 48640),
             (45056, 45056, 40959, 48640), (0, 0, 37888, 100), (100, 200, 2048, 300)]
    for _ in range(400):
        cases.append((int(rng.integers(0, 45057)), int(rng.integers(0, 45057)),
                      int(rng.integers(0, 40961)), int(rng.integers(0, 48641))))
    for apy, opy, bx, by in cases:
        e = oracle.Env(bx=bx, by=by, apy=apy, opy=opy)
        assert np.array_equal(e.render(), paint_then_sample(apy, opy, bx, by)), (apy, opy, bx, by)


def test_rasteriser_structure():
    """Facts that follow from the index maps: the agent's paddle lands in
    output columns 78-79, the opponent's in 5-6, a paddle covers exactly 7
    output rows, source rows are 2 or 3 apart and columns 1 or 2 apart."""
    rows = [(i * 192) // 84 for i in range(84)]
    cols = [(j * 160) // 84 for j in range(84)]
    assert {b - a for a, b in zip(rows, rows[1:])} == {2, 3}
    assert {b - a for a, b in zip(cols, cols[1:])} == {1, 2}
    assert [j for j, c in enumerate(cols) if 148 <= c < 152] == [78, 79]
    assert [j for j, c in enumerate(cols) if 8 <= c < 12] == [5, 6]
    for p in range(0, 177):
        e = oracle.Env(bx=20224, by=0, apy=p << 8, opy=(176 - p) << 8)
        f = e.render()
        assert int((f[:, 78] == 255).sum()) == 7 and int((f[:, 79] == 255).sum()) == 7
        assert int((f[:, 5] == 255).sum()) == 7 and int((f[:, 6] == 255).sum()) == 7
        assert set(np.unique(f)) <= {0, 255}
    # the ball can fall between sampled rows: invisible at some top rows
    invisible = 0
    for y in range(0, 191):
        f = oracle.Env(bx=80 << 8, by=y << 8, apy=0, opy=0).render()
        lit = f.copy()
        lit[:, [5, 6, 78, 79]] = 0
        invisible += int(lit.sum() == 0)
    assert invisible == 24
    # but never between sampled columns
    for x in range(12, 146):
        f = oracle.Env(bx=x << 8, by=96 << 8, apy=0, opy=0).render()
        f[:, [5, 6, 78, 79]] = 0
        assert f.sum() > 0


def test_frameskip_repeats_action_sums_rewards_and_stops_at_done():
    n, T, seed = 7, 500, 31
    acts = explicit_actions(T, n, seed=2)
    o = oracle.OraclePong(n, seed, frameskip=4)
    start, _ = o.get_state()
    near = random_states(n, seed=6, near_end=True)
    o.set_state(near, 0)
    obs, reward, done = o.rollout(T, 2, acts)
    assert done.sum() > 0
    for i in range(n):
        e = oracle.Env(**{k: int(near[j, i]) for j, k in enumerate(oracle.ENV_FIELDS)})
        for t in range(T):
            a = int(acts[t, i])
            rsum, ended = 0, 0
            for _ in range(4):
                r, d = e.frame(a, seed=seed, env_id=i)
                rsum += r
                if d:
                    ended = 1
                    break
            assert reward[t, i] == rsum and done[t, i] == ended
            assert np.array_equal(obs[t, i], e.obs_vector())


def test_ring_slots_and_reset_fill():
    n, seed = 3, 4
    o = oracle.OraclePong(n, seed, obs_mode=1, frameskip=4)
    ring = o.reset()
    first = oracle.Env().reset(seed, 1, 0).render()
    for s in range(4):
        assert np.array_equal(ring[1, s], first)
    snapshots = []
    for t in range(6):
        acts = np.full(n, t % 3, dtype=np.uint8)
        before = o.ring.copy()
        ring, reward, done = o.step(acts)
        assert done.sum() == 0
        for s in range(4):
            if s != t % 4:
                assert np.array_equal(ring[:, s], before[:, s])   # untouched slots
        state, _ = o.get_state()
        for i in range(n):
            e = oracle.Env(**{k: int(state[j, i]) for j, k in enumerate(oracle.ENV_FIELDS)})
            assert np.array_equal(ring[i, t % 4], e.render())
    # force an episode end: all four slots take the reset frame
    near = random_states(n, seed=1, near_end=True)
    near[8] = 9999
    o.set_state(near, 6)
    ring, reward, done = o.step(np.zeros(n, dtype=np.uint8))
    assert done.tolist() == [1, 1, 1]
    for i in range(n):
        f = oracle.Env().reset(seed, i, int(near[9, i]) + 1).render()
        for s in range(4):
            assert np.array_equal(ring[i, s], f)
