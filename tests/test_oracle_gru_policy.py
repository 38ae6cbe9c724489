"""Pins of the GRU-policy oracle against things other than itself: torch's
GRUCell in binary64 (a library routine with the same definition), closed forms,
one-hot weights that expose a transposed operand or a wrong gate block,
binary64 dot products (numpy, exact rationals) with their rounding bounds,
bfloat16 bit patterns."""
import numpy as np
import pytest

from oracle import gru_policy as gp
from paper_2603_12145_b200.inputs import policy_activations, policy_weights


def bits(v):
    return int(np.float32(v).view(np.uint32))


def test_bf16_rounding_bit_patterns_and_ties():
    assert gp.bf16_round(1.0) == 1.0
    # halfway between 1 and 1 + 2^-7: ties to the even significand (1.0)
    assert gp.bf16_round(1.0 + 2.0 ** -8) == 1.0
    # halfway between 1 + 2^-7 (odd) and 1 + 2^-6 (even)
    assert gp.bf16_round(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6
    assert gp.bf16_round(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert gp.bf16_round(-(1.0 + 2.0 ** -8 + 2.0 ** -20)) == -(1.0 + 2.0 ** -7)
    assert bits(gp.bf16_round(0.1)) == 0x3DCD0000          # 0.1f = 0x3DCCCCCD
    assert bits(gp.bf16_round(-384.0 / 40960.0)) == 0xBC1A0000
    assert gp.bf16_round(0.0) == 0.0 and np.isinf(gp.bf16_round(np.inf))
    assert np.isnan(gp.bf16_round(np.nan))
    # the largest finite binary32 rounds up to infinity
    assert np.isinf(gp.bf16_round(np.finfo(np.float32).max))


def test_bf16_rounding_against_torch():
    import torch
    rng = np.random.Generator(np.random.PCG64(5))
    v = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-3, 1000),
                        rng.normal(0, 1e4, 1000)]).astype(np.float32)
    want = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([gp.bf16_round(x) for x in v], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_bf16_rounding_of_float64_is_a_single_rounding():
    # 1 + 2^-8 is a tie (-> 1.0); the same plus 2^-40 lies above the tie, but rounding it to
    # binary32 first would land back on the tie: a double rounding would return 1.0
    v = np.array([1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 2.0 ** -8 - 2.0 ** -40,
                  -(1.0 + 3 * 2.0 ** -8 - 2.0 ** -40), 0.0, 1e-3, -2.5])
    want = np.array([1.0, 1.0 + 2.0 ** -7, 1.0, -(1.0 + 2.0 ** -7), 0.0,
                     gp.bf16_round(1e-3), -2.5], dtype=np.float32)
    assert np.array_equal(gp.bf16_round_f64(v), want)
    rng = np.random.Generator(np.random.PCG64(6))
    f = rng.normal(0, 1, 2000).astype(np.float32)
    assert np.array_equal(gp.bf16_round_f64(f.astype(np.float64)),
                          np.array([gp.bf16_round(x) for x in f], dtype=np.float32))


@pytest.mark.parametrize("H,n,seed", [(64, 5, 1), (192, 3, 2)])
def test_cell_against_torch_grucell_float64(H, n, seed):
    import torch
    w = policy_weights(H, seed)
    x, h = policy_activations(n, H, seed + 10)
    cell = torch.nn.GRUCell(H, H, dtype=torch.float64)
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(w["w_ih"].astype(np.float64)))
        cell.weight_hh.copy_(torch.from_numpy(w["w_hh"].astype(np.float64)))
        cell.bias_ih.copy_(torch.from_numpy(w["b_ih"].astype(np.float64)))
        cell.bias_hh.copy_(torch.from_numpy(w["b_hh"].astype(np.float64)))
        want = cell(torch.from_numpy(x.astype(np.float64)),
                    torch.from_numpy(h.astype(np.float64))).numpy()
    got = gp.cell(x, h, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"])
    assert np.max(np.abs(got - want)) < 1e-13


def zero_weights(H):
    z = np.zeros
    return dict(w_ih=z((3 * H, H), np.float32), w_hh=z((3 * H, H), np.float32),
                b_ih=z(3 * H, np.float32), b_hh=z(3 * H, np.float32))


def test_cell_closed_forms():
    H, n = 8, 4
    x, h = policy_activations(n, H, 3)
    w = zero_weights(H)
    # all zero: r = z = 1/2, n = tanh(0) = 0  ->  h' = h / 2
    assert np.allclose(gp.cell(x, h, **w), 0.5 * h, atol=1e-15)
    # update gate saturated open: h' = h
    w1 = zero_weights(H); w1["b_ih"][H:2 * H] = 40.0
    assert np.allclose(gp.cell(x, h, **w1), h, atol=1e-15)
    # update gate shut, candidate from the input-side bias, reset gate at 1/2 scales the hidden-side bias
    w2 = zero_weights(H); w2["b_hh"][H:2 * H] = -40.0
    w2["b_ih"][2 * H:] = 0.3; w2["b_hh"][2 * H:] = 0.8
    assert np.allclose(gp.cell(x, h, **w2), np.tanh(0.3 + 0.5 * 0.8), atol=1e-15)
    # reset gate shut: the hidden-side part of the candidate vanishes
    w3 = zero_weights(H); w3["b_hh"][H:2 * H] = -40.0; w3["b_ih"][:H] = -40.0
    w3["b_ih"][2 * H:] = 0.3; w3["b_hh"][2 * H:] = 0.8
    assert np.allclose(gp.cell(x, h, **w3), np.tanh(0.3), atol=1e-15)


def test_cell_one_hot_weights_expose_transposes_and_gate_blocks():
    H, n = 8, 3
    x, h = policy_activations(n, H, 4)
    j, k = 2, 5
    # candidate of unit j reads input k only; update gate shut; reset gate irrelevant (no hidden part)
    w = zero_weights(H); w["b_ih"][H:2 * H] = -40.0
    w["w_ih"][2 * H + j, k] = 1.0
    out = gp.cell(x, h, **w)
    assert np.allclose(out[:, j], np.tanh(x[:, k]), atol=1e-15)
    assert np.allclose(np.delete(out, j, axis=1), 0.0, atol=1e-15)
    # hidden-side candidate weight, reset gate saturated open
    w = zero_weights(H); w["b_ih"][H:2 * H] = -40.0; w["b_ih"][:H] = 40.0
    w["w_hh"][2 * H + j, k] = 1.0
    out = gp.cell(x, h, **w)
    assert np.allclose(out[:, j], np.tanh(h[:, k]), atol=1e-15)
    # update gate of unit j driven by hidden k: h'_j = z h_j with the candidate at 0
    w = zero_weights(H); w["w_hh"][H + j, k] = 4.0
    out = gp.cell(x, h, **w)
    z = 1.0 / (1.0 + np.exp(-4.0 * h[:, k].astype(np.float64)))
    assert np.allclose(out[:, j], z * h[:, j], atol=1e-15)
    # reset gate of unit j driven by input k scales the hidden-side candidate bias
    w = zero_weights(H); w["b_ih"][H:2 * H] = -40.0
    w["w_ih"][j, k] = 2.0; w["b_hh"][2 * H:] = 0.7
    out = gp.cell(x, h, **w)
    r = 1.0 / (1.0 + np.exp(-2.0 * x[:, k].astype(np.float64)))
    assert np.allclose(out[:, j], np.tanh(r * 0.7), atol=1e-15)
    other = np.delete(out, j, axis=1)
    assert np.allclose(other, np.tanh(0.5 * 0.7), atol=1e-15)


def test_cell_abs_sum_is_the_sum_of_absolute_products():
    H, n = 16, 3
    w = policy_weights(H, 7)
    x, h = policy_activations(n, H, 8)
    _, t = gp.cell(x, h, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"], with_abs_sum=True)
    ax, ah = np.abs(x.astype(np.float64)), np.abs(h.astype(np.float64))
    wi, wh = np.abs(w["w_ih"].astype(np.float64)), np.abs(w["w_hh"].astype(np.float64))
    want = sum(ax @ wi[g * H:(g + 1) * H].T + ah @ wh[g * H:(g + 1) * H].T for g in range(3))
    assert np.allclose(t, want, rtol=1e-14)


def test_encode_against_float64_and_exact_small_integers():
    H, n = 64, 200
    w = policy_weights(H, 9)
    rng = np.random.Generator(np.random.PCG64(10))
    obs = rng.uniform(-0.1, 1.2, (n, 6)).astype(np.float32)
    got = gp.encode(obs, w["enc_w"], w["enc_b"])
    pre = obs.astype(np.float64) @ w["enc_w"].astype(np.float64).T + w["enc_b"].astype(np.float64)
    want = np.maximum(pre, 0.0)
    mag = np.abs(obs.astype(np.float64)) @ np.abs(w["enc_w"].astype(np.float64)).T + 1.0
    # six fused steps of at most half an ulp each, then one bfloat16 rounding (unit roundoff 2^-8)
    assert np.all(np.abs(got - want) <= 6 * 2.0 ** -24 * mag + 2.0 ** -8 * np.abs(want) * 1.0001)
    assert np.all(got >= 0.0) and np.all((got.view(np.uint32) & 0xFFFF) == 0)
    assert np.any(pre < 0) and np.all(got[pre < -1e-6] == 0.0)
    # small integers: every step is exact, so the result is the exact value rounded once
    obs_i = rng.integers(-3, 4, (n, 6)).astype(np.float32)
    w_i = rng.integers(-3, 4, (H, 6)).astype(np.float32)
    b_i = rng.integers(-3, 4, H).astype(np.float32)
    got = gp.encode(obs_i, w_i, b_i)
    assert np.array_equal(got, np.maximum(obs_i @ w_i.T + b_i, 0.0))   # |values| <= 57: exact in bf16


def test_head_against_numpy_float64_and_exact_small_integers():
    H, n = 96, 50
    w = policy_weights(H, 11)
    _, h = policy_activations(n, H, 12)
    got, mag = gp.head(h, w["head_w"], w["head_b"], with_abs_sum=True)
    assert got.dtype == np.float64
    want = h.astype(np.float64) @ w["head_w"].astype(np.float64).T + w["head_b"].astype(np.float64)
    want_mag = (np.abs(h.astype(np.float64)) @ np.abs(w["head_w"].astype(np.float64)).T
                + np.abs(w["head_b"].astype(np.float64)))
    # numpy's product may add in another order: binary64 rounding only
    assert np.all(np.abs(got - want) <= H * 2.0 ** -52 * want_mag)
    assert np.allclose(mag, want_mag, rtol=1e-14)
    # general binary32 values (not only the generated short ones), against exact rationals
    from fractions import Fraction
    rng = np.random.Generator(np.random.PCG64(13))
    hg = rng.normal(0, 1, (3, 40)).astype(np.float32)
    wg = rng.normal(0, 1, (3, 40)).astype(np.float32)
    bg = rng.normal(0, 1, 3).astype(np.float32)
    out = gp.head(hg, wg, bg)
    for m in range(3):
        for a in range(3):
            exact = sum(Fraction(float(hg[m, k])) * Fraction(float(wg[a, k])) for k in range(40))
            exact += Fraction(float(bg[a]))
            assert abs(Fraction(float(out[m, a])) - exact) <= Fraction(41, 2 ** 52) * 60
    h_i = rng.integers(-4, 5, (n, H)).astype(np.float32)
    w_i = rng.integers(-4, 5, (3, H)).astype(np.float32)
    b_i = rng.integers(-4, 5, 3).astype(np.float32)
    assert np.array_equal(gp.head(h_i, w_i, b_i), (h_i @ w_i.T + b_i).astype(np.float64))
    # a single non-zero weight picks one column: exposes a transposed weight matrix
    w1 = np.zeros((3, H), np.float32); w1[1, 7] = 1.0
    out = gp.head(h, w1, np.zeros(3, np.float32))
    assert np.array_equal(out[:, 1], h[:, 7]) and not out[:, 0].any() and not out[:, 2].any()
    # the bias belongs to its own logit
    out = gp.head(np.zeros((2, H), np.float32), w1, np.array([0.25, -1.5, 3.0], np.float32))
    assert np.array_equal(out, np.array([[0.25, -1.5, 3.0]] * 2))


def test_head_keeps_what_a_binary32_sum_would_lose():
    # 2^24 from unit 0 plus 33 ones: exact in binary64 whatever the order, whereas a binary32
    # running sum would drop every 1 added to 2^24 (ties to even)
    H = 64
    h = np.zeros((1, H), np.float32); w = np.zeros((3, H), np.float32)
    h[0, 0] = 4096.0; w[0, 0] = 4096.0
    h[0, 31:] = 1.0; w[0, 31:] = 1.0
    out = gp.head(h, w, np.array([0.0, 0.0, 0.5], np.float32))
    assert out[0, 0] == 2.0 ** 24 + 33.0 and out[0, 1] == 0.0 and out[0, 2] == 0.5


def test_generated_parameters_are_bfloat16_representable():
    w = policy_weights(128, 14)
    x, h = policy_activations(7, 128, 15)
    for a in (w["w_ih"], w["w_hh"], x, h):
        assert np.all((np.ascontiguousarray(a).view(np.uint32) & 0xFFFF) == 0)
