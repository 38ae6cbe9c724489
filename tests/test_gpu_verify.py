"""The paper's Level-3 protocol run on the real pair of backends: the CUDA
library against the CPU oracle, matched seeds and actions, every step compared,
over more than 100 episodes; then the Level-4 style equivalence test on the
episode returns of the two."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import pong, verify
from paper_2603_12145_b200.inputs import explicit_actions

pytestmark = pytest.mark.gpu


def test_level3_rollout_comparison_gpu_against_oracle_100_episodes():
    import torch
    assert torch.cuda.is_available()
    n, seed = 48, 2024
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    schedule = [(128, 1)] * 40 + [(1, 2)] * 5 + [(37, 0), (512, 2), (8, 3), (128, 0)] * 3
    rep = verify.compare_rollouts(
        env, ora, schedule,
        actions_for=lambda ci, T: explicit_actions(T, n, seed=ci, repeat_fraction=0.1)
        if schedule[ci][1] == 2 else ci % 3)
    assert rep.equal, str(rep)
    assert rep.episodes_finished >= 100
    assert rep.steps_compared == sum(T for T, _ in schedule)


def test_level4_style_equivalence_of_returns():
    import torch
    n, seed = 64, 5
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    rg, cg, ro, co = [], None, [], None
    for _ in range(12):
        g = env.rollout(512, 0)
        o = ora.rollout(512, 0)
        a, cg = verify.episode_returns(g[1], g[2], cg)
        b, co = verify.episode_returns(o[1], o[2], co)
        rg.extend(a.tolist())
        ro.extend(b.tolist())
    assert len(rg) == len(ro) >= 100 and rg == ro
    r = verify.tost_equivalence(rg, ro, margin=1.0)     # the paper's margin for Pong
    assert r.equivalent and r.difference == 0.0
    # a backend whose returns are shifted by more than the margin is rejected
    assert not verify.tost_equivalence(rg, np.array(ro) + 3.0, margin=1.0).equivalent
