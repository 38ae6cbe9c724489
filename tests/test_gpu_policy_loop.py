"""Policy in the loop on the GPU: the sampling kernel and the word stream against
the oracle, and the captured loop against the eager loop and against the oracle
driven by the same logits."""
import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import pong, policy_loop

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t
    assert t.cuda.is_available()
    pong.load(build_if_missing=True)
    return t


def test_fill_words_and_sample_actions_match_the_oracle(torch):
    n, seed = 1000, 12
    env = pong.PongEnv(n, seed, env_id_base=7)
    ora = oracle.OraclePong(n, seed, env_id_base=7)
    env.rollout(5, 0); ora.rollout(5, 0)
    for T in (1, 3, 8, 130):
        w = env.fill_words(T).cpu().numpy().view(np.uint32)
        assert np.array_equal(w, ora.fill_words(T))
    rng = np.random.Generator(np.random.PCG64(0))
    n2 = 1 << 20
    env2 = pong.PongEnv(n2, 1)
    for scale in (0.1, 1.0, 5.0, 40.0):
        logits = (rng.normal(0, scale, (n2, 3))).astype(np.float32)
        words = rng.integers(0, 1 << 32, n2, dtype=np.uint64).astype(np.uint32)
        got = env2.sample_actions(torch.from_numpy(logits).cuda(),
                                  torch.from_numpy(words.view(np.int32)).cuda()).cpu().numpy()
        assert np.array_equal(got, oracle.sample_actions(logits, words)), scale
    # edge logits: ties, huge gaps, zeros
    logits = np.array([[0, 0, 0], [5, 5, -5], [-200, 0, -200], [100, -100, 100], [1e-8, 0, -1e-8]] * 200,
                      dtype=np.float32)
    words = rng.integers(0, 1 << 32, len(logits), dtype=np.uint64).astype(np.uint32)
    env3 = pong.PongEnv(len(logits), 2)
    got = env3.sample_actions(torch.from_numpy(logits).cuda(),
                              torch.from_numpy(words.view(np.int32)).cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.sample_actions(logits, words))


def test_captured_loop_equals_eager_loop_and_the_oracle_env(torch):
    n, seed, K = 512, 3, 8
    policy = policy_loop.make_policy(hidden=64, seed=1)
    a = policy_loop.PolicyLoop(pong.PongEnv(n, seed), policy, steps_per_graph=K)
    b = policy_loop.PolicyLoop(pong.PongEnv(n, seed), policy, steps_per_graph=K)
    ora = oracle.OraclePong(n, seed)
    ora.reset()
    b.capture()
    assert b.env.t == 0
    for rep in range(6):
        # eager loop, step by step, with the oracle env fed the GPU policy's logits
        a.env._stream()
        pong.pong_fill_words(a.env.h, K, a.words)
        words = ora.fill_words(K)
        assert np.array_equal(a.words.cpu().numpy().view(np.uint32), words)
        for i in range(K):
            a._step(i)
            acts = oracle.sample_actions(a.logits.cpu().numpy(), words[i])
            assert np.array_equal(a.actions.cpu().numpy(), acts)
            o, r, d = ora.step(acts)
            assert a.obs.cpu().numpy().tobytes() == o.tobytes()
            assert a.reward.cpu().numpy().tobytes() == r.tobytes()
            assert a.done.cpu().numpy().tobytes() == d.tobytes()
        b.replay()
        torch.cuda.synchronize()
        assert b.env.t == a.env.t == (rep + 1) * K
        assert b.obs.cpu().numpy().tobytes() == a.obs.cpu().numpy().tobytes()
        assert torch.equal(b.hidden, a.hidden) and torch.equal(b.actions, a.actions)
    sa, sb = a.env.get_state(), b.env.get_state()
    assert sa[0].tobytes() == sb[0].tobytes() == ora.get_state()[0].tobytes() and sa[1] == sb[1]
    assert float(a.reward_sum) == float(b.reward_sum)
