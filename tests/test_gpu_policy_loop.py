"""Policy in the loop on the GPU: the sampling kernel and the word stream against
the oracle, the action path on given hidden states (head within its rounding bound,
everything after it bit for bit), the captured loop against the eager loop, and the
whole loop against an independent CPU loop."""
import numpy as np
import pytest

import oracle
from oracle import gru_policy as ogp
from paper_2603_12145_b200 import gru_policy, pong, policy_loop
from paper_2603_12145_b200.inputs import bf16_values, policy_weights

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t
    assert t.cuda.is_available()
    pong.load(build_if_missing=True)
    gru_policy.load(build_if_missing=True)
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


def cdf_margin(logits64, words):
    """Distance of each draw u = (word >> 8) 2^-24 from the nearest boundary of the
    cumulative distribution of softmax(logits), in binary64."""
    p = np.exp(logits64 - logits64.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    u = (words >> np.uint32(8)).astype(np.float64) * 2.0 ** -24
    return np.abs(np.cumsum(p, axis=1)[:, :2] - u[:, None]).min(axis=1)


def test_action_path_on_given_hidden_states(torch):
    """head -> sample -> env step -> encoder of the next observation.  The head is a binary32
    sum in the kernel's order: within (H + H/32 + 1) 2^-24 (|b| + sum |h w|) of the oracle's
    binary64 logits.  Sampling, env step and encoder are fixed-order binary32 or integer: from
    the same logits both sides give the same bits.  An action drawn from the device's logits
    may differ from the one drawn from the oracle's own logits only where the oracle's draw
    lies within the head's bound of a boundary of the cumulative distribution."""
    n, seed, H = 3000, 5, 128
    w = policy_weights(H, 17)
    pol = gru_policy.GruPolicy(w)
    env = pong.PongEnv(n, seed)
    ora = oracle.OraclePong(n, seed)
    env.reset(); ora.reset()
    for rep in range(4):
        h = bf16_values((n, H), 100 + rep, -6, 0)
        hd = torch.from_numpy(h).cuda().to(torch.bfloat16)
        logits = pol.head(hd)
        g_logits = logits.cpu().numpy()
        want_logits, mag = ogp.head(h, w["head_w"], w["head_b"], with_abs_sum=True)
        bound = (H + H // 32 + 1) * 2.0 ** -24 * mag
        assert np.all(np.abs(g_logits.astype(np.float64) - want_logits) <= bound)
        words = ora.fill_words(1)
        assert np.array_equal(env.fill_words(1).cpu().numpy().view(np.uint32), words)
        acts = env.sample_actions(logits, torch.from_numpy(words[0].view(np.int32)).cuda())
        want_acts = oracle.sample_actions(g_logits, words[0])
        assert np.array_equal(acts.cpu().numpy(), want_acts)
        own_acts = oracle.sample_actions(want_logits.astype(np.float32), words[0])
        differ = own_acts != want_acts
        if differ.any():
            # a logit error e moves a boundary by at most 2e (softmax is 1/2-Lipschitz per logit
            # and both boundaries sum at most two probabilities); 1e-6 covers the draw's own arithmetic
            assert np.all(cdf_margin(want_logits[differ], words[0][differ])
                          <= 2 * bound[differ].max(axis=1) + 1e-6)
        assert differ.mean() <= 0.002
        obs, reward, done = env.step(acts)
        o, r, d = ora.step(want_acts)
        assert obs.cpu().numpy().tobytes() == o.tobytes() and done.cpu().numpy().tobytes() == d.tobytes()
        x = pol.encode(obs, done=done, hidden_state=hd)
        want_x = ogp.encode(o, w["enc_w"], w["enc_b"])
        assert np.array_equal(x.to(torch.float32).cpu().numpy().view(np.uint32), want_x.view(np.uint32))
        assert np.array_equal(hd.to(torch.float32).cpu().numpy(), np.where(d[:, None] != 0, np.float32(0), h))
    pol.status()


def test_captured_loop_equals_eager_loop(torch):
    n, seed, K, H = 1000, 3, 8, 128
    pol = gru_policy.GruPolicy(policy_weights(H, 1))
    a = policy_loop.PolicyLoop(pong.PongEnv(n, seed), pol, steps_per_graph=K)
    b = policy_loop.PolicyLoop(pong.PongEnv(n, seed), pol, steps_per_graph=K)
    b.capture()
    assert b.env.t == 0
    for rep in range(6):
        a.run_eager(K)
        b.replay()
        torch.cuda.synchronize()
        assert b.env.t == a.env.t == (rep + 1) * K
        assert torch.equal(b.obs, a.obs) and torch.equal(b.hidden, a.hidden)
        assert torch.equal(b.actions, a.actions) and torch.equal(b.done, a.done)
        assert torch.equal(b.logits, a.logits) and torch.equal(b.x, a.x)
    sa, sb = a.env.get_state(), b.env.get_state()
    assert sa[0].tobytes() == sb[0].tobytes() and sa[1] == sb[1]
    assert a.env.episode_stats() == b.env.episode_stats()
    pol.status()


def test_loop_against_an_independent_oracle_loop(torch):
    """The whole loop on the CPU, from the oracles alone (binary64 cell rounded once to
    bfloat16, binary64 head rounded once to binary32), against the GPU loop.  The cell's
    results differ in the last bfloat16 place now and then (tensor-core accumulation order,
    approximate exponentials) and the head's binary32 sum carries its own rounding, so
    the logits differ slightly and a draw that falls within that distance of a
    boundary of the cumulative distribution may pick the neighbouring action.  What
    must hold: until an env's first differing action everything it emits is bit-equal;
    at that step the oracle's draw was close to a boundary; few envs get there; the
    hidden states stay within a few bfloat16 places."""
    n, seed, K, H = 2048, 9, 12, 128
    w = policy_weights(H, 2)
    pol = gru_policy.GruPolicy(w)
    loop = policy_loop.PolicyLoop(pong.PongEnv(n, seed), pol, steps_per_graph=K)
    ora = oracle.OraclePong(n, seed)
    obs = ora.reset()
    h = np.zeros((n, H), np.float32)
    done = np.zeros(n, np.uint8)
    words = ora.fill_words(K)
    loop._streams()
    pong.pong_fill_words(loop.env.h, K, loop.words)
    same = np.ones(n, bool)          # envs whose actions have all agreed so far
    worst_margin, worst_h = 0.0, 0.0
    for i in range(K):
        h[done != 0] = 0.0
        x = ogp.encode(obs, w["enc_w"], w["enc_b"])
        h = ogp.bf16_round_f64(ogp.cell(x, h, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"]))
        logits = ogp.head(h, w["head_w"], w["head_b"]).astype(np.float32)   # rounded once
        acts = oracle.sample_actions(logits, words[i])
        obs, r, done = ora.step(acts)
        loop._step(i)
        g_h = loop.hidden.to(torch.float32).cpu().numpy()
        g_acts = loop.actions.cpu().numpy()
        worst_h = max(worst_h, float(np.abs(g_h[same] - h[same]).max()))
        differ = same & (g_acts != acts)
        if differ.any():
            p = np.exp(logits[differ].astype(np.float64))
            p /= p.sum(axis=1, keepdims=True)
            u = (words[i][differ] >> np.uint32(8)).astype(np.float64) * 2.0 ** -24
            cdf = np.cumsum(p, axis=1)[:, :2]
            worst_margin = max(worst_margin, float(np.abs(cdf - u[:, None]).min(axis=1).max()))
        same &= ~differ
        assert np.array_equal(loop.obs.cpu().numpy()[same].view(np.uint32), obs[same].view(np.uint32))
        assert np.array_equal(loop.reward.cpu().numpy()[same], r[same])
        assert np.array_equal(loop.done.cpu().numpy()[same], done[same])
    pol.status()
    assert worst_h <= 2.0 ** -7, worst_h          # observed: one place (2^-9 at |h| < 1/2); a few are allowed
    assert worst_margin <= 2e-3, worst_margin
    assert (~same).mean() <= 0.01, (~same).sum()  # observed: none


def test_pipelined_loop_equals_the_single_loop(torch):
    """Two slices on two streams in one graph: the union of their trajectories is the
    single loop's, bit for bit (global env ids; the cell's result for a row does not
    depend on where the row sits in a tile)."""
    n, seed, K, H = 1024, 4, 6, 128
    pol = gru_policy.GruPolicy(policy_weights(H, 3))
    one = policy_loop.PolicyLoop(pong.PongEnv(n, seed), pol, steps_per_graph=K)
    two = policy_loop.PipelinedPolicyLoop(n, seed, pol, steps_per_graph=K, parts=2)
    two.capture()
    for rep in range(4):
        one.run_eager(K)
        two.replay()
        torch.cuda.synchronize()
        for name in ("obs", "actions", "done", "logits", "reward"):
            whole = getattr(one, name)
            halves = torch.cat([getattr(p, name) for p in two.parts])
            assert torch.equal(whole, halves), name
        assert torch.equal(one.hidden, torch.cat([p.hidden for p in two.parts]))
    assert two.episode_stats() == tuple(int(v) for v in one.env.episode_stats())
    states = [p.env.get_state() for p in two.parts]
    assert np.array_equal(np.concatenate([s[0] for s in states], axis=1), one.env.get_state()[0])
    assert all(s[1] == one.env.get_state()[1] for s in states)
    pol.status()
