"""Pins for the oracle's game rules: hand-computed single frames, a closed-form
rally, per-step invariants and brute force over every short action sequence.
All expected values here are worked out by hand (or by a closed form) from the
rule set, never by running the oracle."""
import itertools

import numpy as np

import oracle
from paper_2603_12145_b200.inputs import explicit_actions, random_states

CENTRE = 22528


def env(**kw):
    base = dict(bx=20224, by=24320, vx=512, vy=0, apy=CENTRE, opy=CENTRE,
                score_a=0, score_o=0, ep_len=0, episode=0, prev_action=0)
    base.update(kw)
    return oracle.Env(**base)


# ---- hand-computed single frames ---------------------------------------------

def test_agent_paddle_moves_and_clamps():
    e = env(); e.frame(1); assert e.apy == CENTRE - 768      # up = towards y 0
    e = env(); e.frame(2); assert e.apy == CENTRE + 768
    e = env(); e.frame(0); assert e.apy == CENTRE
    e = env(apy=300); e.frame(1); assert e.apy == 0
    e = env(apy=44800); e.frame(2); assert e.apy == 45056


def test_opponent_tracks_ball_centre_by_at_most_two_pixels():
    e = env(by=30000); e.frame(0); assert e.opy == 23040     # d = 5680 -> +512
    e = env(by=10000); e.frame(0); assert e.opy == 22016     # d < -512 -> -512
    e = env(by=24420); e.frame(0); assert e.opy == CENTRE + 100  # d = 100
    # uses the ball as it was before it moved this frame
    e = env(by=24320, vy=300); e.frame(0); assert e.opy == CENTRE
    e = env(by=48640, opy=44900, vy=0); e.frame(0); assert e.opy == 45056
    e = env(by=0, opy=100, vy=0); e.frame(0); assert e.opy == 0


def test_wall_reflection_mirrors():
    e = env(by=100, vy=-384); e.frame(0); assert (e.by, e.vy) == (284, 384)
    e = env(by=48500, vy=300); e.frame(0); assert (e.by, e.vy) == (48480, -300)
    # touching the wall exactly is not a reflection
    e = env(by=384, vy=-384); e.frame(0); assert (e.by, e.vy) == (0, -384)
    e = env(by=48340, vy=300); e.frame(0); assert (e.by, e.vy) == (48640, 300)


def test_agent_paddle_hit_centre():
    e = env(bx=37000, vx=512, by=24320, vy=0)
    r, d = e.frame(0)
    assert (e.bx, e.vx, e.vy, r, d) == (37512, -528, 0, 0, 0)


def test_agent_paddle_hit_offset_adds_spin():
    e = env(bx=37000, vx=512, by=23040, vy=100)
    e.frame(0)
    # by = 23140; ball centre px = 91, paddle centre px = 96 -> vy = 100 - 80
    assert (e.by, e.vx, e.vy) == (23140, -528, 20)


def test_opponent_paddle_hit():
    # opponent paddle spans x in [2048, 3072); ball arrives from the right
    e = env(bx=3500, vx=-600, by=24320, vy=0)
    e.frame(0)
    assert (e.bx, e.vx, e.vy) == (2900, 616, 0)
    # spin from the opponent paddle: opy tracks first (22528 -> 23040 for a low
    # ball), then dpx = ((26000+256)>>8) - ((23040+2048)>>8) = 102 - 98 = 4
    e = env(bx=3500, vx=-600, by=26000, vy=0)
    e.frame(0)
    assert (e.opy, e.vx, e.vy) == (23040, 616, 64)


def test_no_hit_when_moving_away_or_outside_box():
    e = env(bx=37512, vx=-528); e.frame(0); assert e.vx == -528      # moving away
    e = env(bx=2900, vx=616); e.frame(0); assert e.vx == 616
    # ball just above the agent paddle: by + 512 == apy is not an overlap
    e = env(bx=37000, vx=512, by=CENTRE - 512, vy=0, opy=CENTRE); e.frame(0)
    assert e.vx == 512
    e = env(bx=37000, vx=512, by=CENTRE - 511, vy=0); e.frame(0)
    assert e.vx == -528
    # ball just below: by == apy + 4096 is not an overlap
    e = env(bx=37000, vx=512, by=CENTRE + 4096, vy=0); e.frame(0); assert e.vx == 512
    e = env(bx=37000, vx=512, by=CENTRE + 4095, vy=0); e.frame(0); assert e.vx == -528
    # x edges of the agent box: bx + 512 > 37888 and bx < 38912 after the move
    e = env(bx=37376 - 512, vx=512); e.frame(0); assert e.vx == 512   # bx = 37376
    e = env(bx=37377 - 512, vx=512); e.frame(0); assert e.vx == -528
    e = env(bx=38912 - 512, vx=512); e.frame(0); assert e.vx == 512   # bx = 38912
    e = env(bx=38911 - 512, vx=512); e.frame(0); assert e.vx == -528


def test_speed_cap_and_spin_clamp():
    e = env(bx=37000, vx=1020, by=24320, vy=0); e.frame(0); assert e.vx == -1024
    e = env(bx=37000, vx=1024, by=24320, vy=0); e.frame(0); assert e.vx == -1024
    # ball 9 px above paddle centre, vy already near the cap
    e = env(bx=37000, vx=512, by=22728, vy=-700); e.frame(0)
    # by = 22028 overlaps the paddle top (22540 > 22528); ball centre px =
    # (22284 >> 8) = 87, paddle centre px = 96 -> vy = -700 - 144, clamped
    assert (e.by, e.vx, e.vy) == (22028, -528, -768)
    e = env(bx=37000, vx=512, by=25000, vy=760); e.frame(0)
    # by = 25760, centre px = (26016 >> 8) = 101 -> vy = 760 + 80, clamped
    assert (e.by, e.vx, e.vy) == (25760, -528, 768)


def test_agent_action_affects_same_frame_collision():
    # paddle at 26624: ball at by = 25856 + 512 = 26368 <= apy, a miss unless
    # the paddle moves up by 768 in this very frame
    e = env(bx=37000, vx=512, by=25856, vy=0, apy=26624); e.frame(0); assert e.vx == 512
    e = env(bx=37000, vx=512, by=25856, vy=0, apy=26624); e.frame(1); assert e.vx == -528


def test_scoring_right_edge_rewards_plus_one_and_respawns():
    e = env(bx=40700, vx=512, by=1000, vy=0, apy=40000, episode=2)
    r, d = e.frame(0, seed=9, env_id=4)
    assert (r, d, e.score_a, e.score_o, e.ep_len) == (1, 0, 1, 0, 1)
    want = oracle.Env().spawn(9, 4, 2, 1)        # keyed by point = 1
    assert (e.bx, e.by, e.vx, e.vy) == (want.bx, want.by, want.vx, want.vy)
    assert (e.bx, e.by) == (20224, 24320)
    assert e.apy == 40000                        # paddles are not moved by a point


def test_scoring_left_edge_rewards_minus_one():
    e = env(bx=300, vx=-512, by=1000, vy=0, opy=40000)
    r, d = e.frame(0, seed=9, env_id=4)
    assert (r, d, e.score_a, e.score_o) == (-1, 0, 0, 1)
    # bx == 0 and bx == 40960 are still in play
    e = env(bx=512, vx=-512, by=1000, opy=40000); r, _ = e.frame(0); assert r == 0 and e.bx == 0
    e = env(bx=40448, vx=512, by=1000, apy=40000); r, _ = e.frame(0); assert r == 0 and e.bx == 40960


def test_done_on_21st_point_then_auto_reset():
    st = oracle.new_stats()
    e = env(bx=40700, vx=512, by=1000, apy=40000, score_a=20, score_o=7, ep_len=1234,
            episode=5, prev_action=2)
    r, d = e.frame(0, seed=3, env_id=8, stats=st)
    assert (r, d) == (1, 1)
    assert (st.episodes, st.sum_return, st.sum_length) == (1, 14, 1235)
    assert e.as_dict() == oracle.Env().reset(3, 8, 6).as_dict()
    # opponent's 21st point
    st = oracle.new_stats()
    e = env(bx=300, vx=-512, by=1000, opy=40000, score_a=2, score_o=20, ep_len=50, episode=0)
    r, d = e.frame(0, seed=3, env_id=8, stats=st)
    assert (r, d) == (-1, 1)
    assert (st.episodes, st.sum_return, st.sum_length) == (1, -19, 51)
    # 20 points is not the end
    e = env(bx=40700, vx=512, by=1000, apy=40000, score_a=19)
    assert e.frame(0) == (1, 0) and e.score_a == 20


def test_done_on_step_limit():
    st = oracle.new_stats()
    e = env(ep_len=9998, score_a=3, score_o=5, episode=1)
    assert e.frame(0, stats=st) == (0, 0) and e.ep_len == 9999
    assert e.frame(0, seed=1, env_id=2, stats=st) == (0, 1)
    assert (st.episodes, st.sum_return, st.sum_length) == (1, -2, 10000)
    assert e.as_dict() == oracle.Env().reset(1, 2, 2).as_dict()


# ---- closed-form rally ----------------------------------------------------------

def rally_hit_frames(limit):
    """Frames on which a vy = 0 ball that starts rightwards from the spawn
    point is hit, by solving each leg in closed form: the agent's box is
    entered by the first bx with bx + 512 > 37888, the opponent's by the first
    bx < 3072."""
    frames, speeds = [], []
    bx, speed, frame, right = 20224, 512, 0, True
    while True:
        if right:
            n = (37376 - bx) // speed + 1          # smallest n: bx + n*speed > 37376
            bx += n * speed
        else:
            n = (bx - 3072) // speed + 1           # smallest n: bx - n*speed < 3072
            bx -= n * speed
        frame += n
        if frame > limit:
            return frames, speeds
        speed = min(speed + 16, 1024)
        frames.append(frame)
        speeds.append(speed)
        right = not right


def test_closed_form_rally_until_step_limit():
    frames, speeds = rally_hit_frames(10000)
    assert frames[:2] == [34, 100] and speeds[:2] == [528, 544]
    hits = dict(zip(frames, speeds))
    st = oracle.new_stats()
    e = env(vx=512, vy=0)
    prev_vx = 512
    for f in range(1, 10000):
        r, d = e.frame(0, seed=0, env_id=0, stats=st)
        assert (r, d) == (0, 0)
        assert e.vy == 0 and e.by == 24320 and e.opy == CENTRE and e.apy == CENTRE
        if f in hits:
            assert abs(e.vx) == hits[f] and (e.vx > 0) != (prev_vx > 0), f
        else:
            assert e.vx == prev_vx, f
        prev_vx = e.vx
    assert abs(e.vx) == 1024
    r, d = e.frame(0, seed=0, env_id=0, stats=st)
    assert (r, d) == (0, 1)
    assert (st.episodes, st.sum_return, st.sum_length) == (1, 0, 10000)
    assert e.as_dict() == oracle.Env().reset(0, 0, 1).as_dict()


# ---- invariants over long random play -------------------------------------------

def check_invariants(before, after, r, d, seed, env_id):
    a = after
    assert 0 <= a["bx"] <= 40960 and 0 <= a["by"] <= 48640
    assert 0 <= a["apy"] <= 45056 and 0 <= a["opy"] <= 45056
    assert 512 <= abs(a["vx"]) <= 1024 and abs(a["vy"]) <= 768
    assert r in (-1, 0, 1) and d in (0, 1)
    if d:
        assert a == oracle.Env().reset(seed, env_id, before["episode"] + 1).as_dict()
        assert (r == 1 and before["score_a"] == 20) or (r == -1 and before["score_o"] == 20) \
            or before["ep_len"] == 9999
    else:
        assert a["episode"] == before["episode"]
        assert a["ep_len"] == before["ep_len"] + 1 and a["ep_len"] < 10000
        assert a["score_a"] == before["score_a"] + (r == 1) <= 20
        assert a["score_o"] == before["score_o"] + (r == -1) <= 20
        if r != 0:
            assert (a["bx"], a["by"]) == (20224, 24320) and abs(a["vx"]) == 512 \
                and abs(a["vy"]) <= 384
            assert abs(a["apy"] - before["apy"]) <= 768       # paddles keep their place
        else:
            assert abs(a["bx"] - before["bx"]) <= 1024
            if abs(a["vx"]) != abs(before["vx"]):            # a hit
                assert a["vx"] * before["vx"] < 0
                assert abs(a["vx"]) == min(abs(before["vx"]) + 16, 1024)
                pad_lo = 37376 if before["vx"] > 0 else 1536
                pad_hi = 38912 if before["vx"] > 0 else 3072
                assert pad_lo < a["bx"] < pad_hi


def test_invariants_random_play():
    seed = 12345
    acts = explicit_actions(6000, 6, seed=1)
    for env_id in range(6):
        e = oracle.Env().reset(seed, env_id, 0)
        ret, finished = 0, 0
        st = oracle.new_stats()
        for t in range(6000):
            before = e.as_dict()
            r, d = e.frame(int(acts[t, env_id]), seed=seed, env_id=env_id, stats=st)
            check_invariants(before, e.as_dict(), r, d, seed, env_id)
            ret += r
            if d:
                finished += 1
                assert st.episodes == finished
                assert st.sum_return == ret      # sum of rewards = score difference
        assert finished >= 1


def test_invariants_from_random_states_near_episode_end():
    s = random_states(400, seed=3, near_end=True)
    acts = explicit_actions(80, 400, seed=4)
    dones = 0
    for i in range(400):
        e = oracle.Env(**{k: int(s[j, i]) for j, k in enumerate(oracle.ENV_FIELDS)})
        for t in range(80):
            before = e.as_dict()
            r, d = e.frame(int(acts[t, i]), seed=77, env_id=i)
            check_invariants(before, e.as_dict(), r, d, 77, i)
            dones += d
    assert dones > 100


# ---- brute force over every action sequence --------------------------------------

def test_brute_force_all_sequences_from_reset():
    """From a reset, for T <= 8 no wall or paddle can be reached, so every
    quantity has a closed form in the action counts."""
    for seed, env_id in ((0, 0), (1, 5), (0xDEADBEEF, 63)):
        start = oracle.Env().reset(seed, env_id, 0).as_dict()
        for T in (1, 2, 5, 8):
            for seq in itertools.product((0, 1, 2), repeat=T):
                e = oracle.Env(**start)
                opy = CENTRE
                for t, a in enumerate(seq):
                    ball_c = start["by"] + t * start["vy"] + 256
                    opy += max(-512, min(512, ball_c - (opy + 2048)))
                    assert e.frame(a, seed=seed, env_id=env_id) == (0, 0)
                ups, downs = seq.count(1), seq.count(2)
                assert e.apy == CENTRE + 768 * (downs - ups)
                assert e.bx == 20224 + T * start["vx"]
                assert e.by == 24320 + T * start["vy"]
                assert (e.vx, e.vy) == (start["vx"], start["vy"])
                assert e.opy == opy and e.ep_len == T


def test_brute_force_near_agent_paddle():
    """Ball two frames from the agent's box, paddle edge near the ball: whether
    it is returned depends on the action sequence.  Checked against geometry
    worked out from the box definition, for all 3^6 sequences."""
    n_hit = n_miss = 0
    for seq in itertools.product((0, 1, 2), repeat=6):
        e = env(bx=36400, vx=512, by=20000, vy=0, apy=20000 + 512 + 768, opy=CENTRE)
        apy, hit_frame = e.apy, None
        for t, a in enumerate(seq):
            apy = max(0, min(45056, apy + (768 if a == 2 else -768 if a == 1 else 0)))
            bx = 36400 + 512 * (t + 1)
            inside_x = bx + 512 > 37888 and bx < 38912
            inside_y = 20000 + 512 > apy and 20000 < apy + 4096
            before = e.as_dict()
            r, d = e.frame(a)
            check_invariants(before, e.as_dict(), r, d, 0, 0)
            if hit_frame is None and inside_x and inside_y:
                hit_frame = t
                assert e.vx == -528
                break
            assert e.vx == 512
        if hit_frame is None:
            n_miss += 1
        else:
            n_hit += 1
    assert n_hit > 50 and n_miss > 50


def test_batch_rollout_equals_frame_by_frame():
    """The batch driver is the single-env frame applied to every env, with the
    outputs stacked over T."""
    n, T, seed = 5, 300, 21
    acts = explicit_actions(T, n, seed=8)
    o = oracle.OraclePong(n, seed)
    obs, reward, done = o.rollout(T, 2, acts)
    for i in range(n):
        e = oracle.Env().reset(seed, i, 0)
        for t in range(T):
            r, d = e.frame(int(acts[t, i]), seed=seed, env_id=i)
            assert reward[t, i] == r and done[t, i] == d
            assert np.array_equal(obs[t, i], e.obs_vector())


def test_opponent_box_y_edges_are_half_open():
    # the opponent first tracks by 512 (0 -> 512); box is [512, 4608)
    e = env(bx=3500, vx=-600, by=4608, vy=0, opy=0); e.frame(0)
    assert (e.opy, e.vx) == (512, -600)
    e = env(bx=3500, vx=-600, by=4607, vy=0, opy=0); e.frame(0)
    assert (e.opy, e.vx) == (512, 616)
    # tracking upwards 45056 -> 44544; the ball's bottom edge must pass 44544
    e = env(bx=3500, vx=-600, by=44544 - 512, vy=0, opy=45056); e.frame(0)
    assert (e.opy, e.vx) == (44544, -600)
    e = env(bx=3500, vx=-600, by=44544 - 511, vy=0, opy=45056); e.frame(0)
    assert (e.opy, e.vx) == (44544, 616)


def test_respawn_point_key_counts_both_scores():
    e = env(bx=40700, vx=512, by=1000, vy=0, apy=40000, score_a=3, score_o=4, episode=6)
    e.frame(0, seed=13, env_id=21)
    want = oracle.Env().spawn(13, 21, 6, 8)
    assert (e.vx, e.vy) == (want.vx, want.vy)
    e = env(bx=300, vx=-512, by=1000, vy=0, opy=40000, score_a=3, score_o=4, episode=6)
    e.frame(0, seed=13, env_id=21)
    assert (e.vx, e.vy) == (want.vx, want.vy)


def test_spin_uses_floored_whole_pixel_centres():
    # paddle top 22628 -> centre 24676 -> pixel 96 (floor); ball by = 25000 ->
    # centre 25256 -> pixel 98; vy = 0 + 16 * 2
    e = env(bx=37000, vx=512, by=25000, vy=0, apy=22628); e.frame(0)
    assert (e.vx, e.vy) == (-528, 32)
    # ball centre 24831 -> pixel 96 (floor, not round): no spin
    e = env(bx=37000, vx=512, by=24575, vy=0, apy=22528); e.frame(0)
    assert (e.vx, e.vy) == (-528, 0)
