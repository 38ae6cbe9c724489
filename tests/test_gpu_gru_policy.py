"""Parity of the GRU-policy kernels with the CPU oracle, through the C ABI.

The encoder is fixed-order binary32 and must match bit for bit.  The head is a
binary32 sum in the kernel's own order (documented in include/gru_policy.h) and
is compared with the oracle's binary64 evaluation of W_o h' + b_o within

    |logit_gpu - logit| <= (H + H/32 + 1) * 2^-24 * (|b| + sum |h w|)

(one binary32 rounding per fused multiply-add, one per partial sum added, one for
the bias: each at most 2^-24 of a running sum that never exceeds the sum of the
absolute terms); on operands whose every partial sum is a binary32 number the
two must agree exactly.  The cell
runs on the tensor cores, whose accumulation order is unspecified; its result
is compared with the oracle's binary64 evaluation within

    |h'_gpu - h'| <= 2^-8 |h'|  +  2e-5  +  c * 2H * 2^-23 * S

  - 2^-8 |h'|: the one bfloat16 rounding of the result (unit roundoff 2^-8);
  - 2e-5: the epilogue's exponentials and reciprocals (approximate to a few
    binary32 ulps) carried through two sigmoids, a tanh and the blend;
  - the last term bounds the binary32 accumulation of a 2H-term sum whose
    absolute products add up to at most S (the oracle returns S per output),
    each step losing at most 2^-23 of the running sum, carried into h' with
    sensitivity c = 2.5 + (S + 1) / 4  (|dh'| <= |d nx| + |d nh| + |d z| / 2 +
    |nh + b_hn| |d r| / 4).
The generated test operands are small multiples of powers of two, chosen so that
every partial sum is exactly representable in binary32: there the last term is
dropped and the bound is tight enough to see a dropped bias or a swapped gate.
"""
import numpy as np
import pytest

from oracle import gru_policy as ogp
from paper_2603_12145_b200 import gru_policy as gp
from paper_2603_12145_b200.inputs import bf16_values, policy_activations, policy_weights

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available()
    gp.load(build_if_missing=True)
    return torch


def to_dev_bf16(torch, a):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    b = t.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float32), t), "operand is not bfloat16-representable"
    return b


def from_dev_bf16(torch, t):
    return t.to(torch.float32).cpu().numpy()


def cell_tolerance(want, S=None, H=None):
    tol = 2.0 ** -8 * np.abs(want) + 2e-5
    if S is not None:
        tol = tol + (2.5 + 0.25 * (S + 1.0)) * (2 * H) * 2.0 ** -23 * S
    return tol


@pytest.mark.parametrize("H,n,seed", [(64, 1, 1), (64, 128, 2), (128, 129, 3), (192, 257, 4),
                                      (576, 300, 5), (576, 1024, 6), (1024, 130, 7)])
def test_cell_exact_accumulation_inputs(torch_cuda, H, n, seed):
    torch = torch_cuda
    w = policy_weights(H, seed)
    x, h = policy_activations(n, H, seed + 100)
    want, S = ogp.cell(x, h, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"], with_abs_sum=True)
    # every partial sum of an accumulator is a multiple of 2^-18 below 2^6: exact in binary32
    # in any order
    ax, ah = np.abs(x.astype(np.float64)), np.abs(h.astype(np.float64))
    for g in range(3):
        rows = slice(g * H, (g + 1) * H)
        assert (ax @ np.abs(w["w_ih"][rows]).T.astype(np.float64)
                + ah @ np.abs(w["w_hh"][rows]).T.astype(np.float64)).max() < 64.0
    pol = gp.GruPolicy(w)
    out = pol.cell(to_dev_bf16(torch, x), to_dev_bf16(torch, h))
    pol.status()
    got = from_dev_bf16(torch, out)
    err = np.abs(got - want)
    tol = cell_tolerance(want)
    bad = np.argwhere(err > tol)
    assert bad.size == 0, "first mismatch at %s: got %r want %r" % (
        bad[0], got[tuple(bad[0])], want[tuple(bad[0])])
    # the error must look like one rounding, not like a systematic offset
    assert np.mean(err) < 2.0 ** -9 * np.mean(np.abs(want)) + 1e-5
    pol.close()


@pytest.mark.parametrize("H,n,seed", [(128, 200, 11), (576, 384, 12)])
def test_cell_general_bfloat16_inputs(torch_cuda, H, n, seed):
    torch = torch_cuda
    w = policy_weights(H, seed)
    w["w_ih"] = bf16_values((3 * H, H), seed + 1, -9, -5)
    w["w_hh"] = bf16_values((3 * H, H), seed + 2, -9, -5)
    w["b_ih"] = bf16_values((3 * H,), seed + 3, -6, -2)
    w["b_hh"] = bf16_values((3 * H,), seed + 4, -6, -2)
    x = np.abs(bf16_values((n, H), seed + 5, -5, 1))
    h = bf16_values((n, H), seed + 6, -8, -1)
    want, S = ogp.cell(x, h, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"], with_abs_sum=True)
    pol = gp.GruPolicy(w)
    out = pol.cell(to_dev_bf16(torch, x), to_dev_bf16(torch, h))
    pol.status()
    got = from_dev_bf16(torch, out)
    err = np.abs(got - want)
    assert np.all(err <= cell_tolerance(want, S, H))
    # in practice the accumulation error is far below its worst-case bound
    assert np.quantile(err - 2.0 ** -8 * np.abs(want), 0.999) < 1e-4
    pol.close()


def test_cell_full_size_sampled_rows_and_determinism(torch_cuda):
    torch = torch_cuda
    H, n = 576, 65536
    w = policy_weights(H, 21)
    x, h = policy_activations(n, H, 22)
    pol = gp.GruPolicy(w)
    xd, hd = to_dev_bf16(torch, x), to_dev_bf16(torch, h)
    out1 = pol.cell(xd, hd)
    out2 = pol.cell(xd, hd)
    pol.status()
    assert torch.equal(out1, out2)
    rng = np.random.Generator(np.random.PCG64(23))
    rows = np.unique(np.concatenate([[0, 127, 128, n - 129, n - 128, n - 1],
                                     rng.integers(0, n, 250)]))
    want = ogp.cell(x[rows], h[rows], w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"])
    got = from_dev_bf16(torch, out1[torch.from_numpy(rows).cuda()])
    assert np.all(np.abs(got - want) <= cell_tolerance(want))
    assert pol.launches == 2
    pol.close()


@pytest.mark.parametrize("H,n", [(64, 1), (576, 1000), (128, 4097)])
def test_encode_bit_exact_and_done_mask(torch_cuda, H, n):
    torch = torch_cuda
    w = policy_weights(H, 31)
    rng = np.random.Generator(np.random.PCG64(32))
    obs = rng.uniform(-0.1, 1.2, (n, 6)).astype(np.float32)
    done = (rng.random(n) < 0.3).astype(np.uint8)
    _, h = policy_activations(n, H, 33)
    pol = gp.GruPolicy(w)
    hd = to_dev_bf16(torch, h)
    x = pol.encode(torch.from_numpy(obs).cuda(), done=torch.from_numpy(done).cuda(), hidden_state=hd)
    pol.status()
    want = ogp.encode(obs, w["enc_w"], w["enc_b"])
    got = from_dev_bf16(torch, x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    h_want = np.where(done[:, None] != 0, np.float32(0.0), h)
    assert np.array_equal(from_dev_bf16(torch, hd), h_want)
    # without a mask h is not touched
    hd2 = to_dev_bf16(torch, h)
    pol.encode(torch.from_numpy(obs).cuda())
    assert np.array_equal(from_dev_bf16(torch, hd2), h)
    pol.close()


def head_tolerance(mag, H):
    return (H + H // 32 + 1) * 2.0 ** -24 * mag


@pytest.mark.parametrize("H,n", [(64, 1), (576, 1000), (1024, 300)])
def test_head_within_rounding_bound(torch_cuda, H, n):
    torch = torch_cuda
    w = policy_weights(H, 41)
    h = bf16_values((n, H), 42, -8, 0)
    pol = gp.GruPolicy(w)
    logits = pol.head(to_dev_bf16(torch, h)).cpu().numpy().astype(np.float64)
    pol.status()
    want, mag = ogp.head(h, w["head_w"], w["head_b"], with_abs_sum=True)
    assert np.all(np.abs(logits - want) <= head_tolerance(mag, H))
    pol.close()


@pytest.mark.parametrize("H,n", [(64, 33), (576, 1000), (1024, 300)])
def test_head_exact_where_every_partial_sum_is_representable(torch_cuda, H, n):
    """h = k/128 and w = j/512 with |k| <= 127, |j| <= 96, bias = i/2048: every product is a
    multiple of 2^-16 and any partial sum stays below 2^24 such units, so a binary32 sum in any
    order is exact and must equal the binary64 value."""
    torch = torch_cuda
    w = policy_weights(H, 43)
    _, h = policy_activations(n, H, 44)
    pol = gp.GruPolicy(w)
    logits = pol.head(to_dev_bf16(torch, h)).cpu().numpy()
    pol.status()
    want = ogp.head(h, w["head_w"], w["head_b"])
    assert np.array_equal(want.astype(np.float32).astype(np.float64), want)
    assert np.array_equal(logits.astype(np.float64), want)
    pol.close()


@pytest.mark.parametrize("H,n", [(64, 1), (576, 700), (128, 513)])
def test_fused_head_against_the_oracle(torch_cuda, H, n):
    """The logits the cell kernel's epilogue forms, against W_o h' + b_o of the oracle on the
    hidden state the kernel stored."""
    torch = torch_cuda
    w = policy_weights(H, 63)
    x = np.abs(bf16_values((n, H), 64, -6, 0))
    h = bf16_values((n, H), 65, -7, -1)
    pol = gp.GruPolicy(w)
    h2, l2 = pol.cell_head(to_dev_bf16(torch, x), to_dev_bf16(torch, h))
    pol.status()
    want, mag = ogp.head(from_dev_bf16(torch, h2), w["head_w"], w["head_b"], with_abs_sum=True)
    assert np.all(np.abs(l2.cpu().numpy().astype(np.float64) - want) <= head_tolerance(mag, H))
    pol.close()


@pytest.mark.parametrize("H,n", [(64, 1), (576, 700), (128, 513)])
def test_self_consistency_fused_head_equals_standalone_head(torch_cuda, H, n):
    """Self-consistency of the two device paths, not a parity claim: the fused entry point
    gives the bits of the two separate calls (each is compared with the oracle above)."""
    torch = torch_cuda
    w = policy_weights(H, 61)
    x, h = policy_activations(n, H, 62)
    pol = gp.GruPolicy(w)
    xd, hd = to_dev_bf16(torch, x), to_dev_bf16(torch, h)
    h1 = pol.cell(xd, hd)
    l1 = pol.head(h1)
    h2, l2 = pol.cell_head(xd, hd)
    pol.status()
    assert torch.equal(h1, h2)
    assert torch.equal(l1, l2)
    assert gp.gru_policy_workspace_bytes(pol.h, n) == n * (H // 32) * 16
    pol.close()


def test_cell_rows_do_not_depend_on_the_batch(torch_cuda):
    """A row's result is the same bits whatever the batch it is launched in: task counts below,
    at and above the number of resident block pairs, ragged last tiles, both entry points."""
    torch = torch_cuda
    H, nmax = 576, 20000
    pol = gp.GruPolicy(policy_weights(H, 81))
    x, h = policy_activations(nmax, H, 82)
    xd, hd = to_dev_bf16(torch, x), to_dev_bf16(torch, h)
    ref_h = torch.empty_like(hd)
    ref_l = torch.empty((nmax, 3), device="cuda")
    for a in range(0, nmax, 1024):
        b = min(nmax, a + 1024)
        ref_h[a:b], ref_l[a:b] = pol.cell_head(xd[a:b], hd[a:b])
    for n in (1, 127, 129, 256, 257, 2047, 2105, 2106, 4211, 9472, 18944, 18945, nmax):
        out, logits = pol.cell_head(xd[:n], hd[:n])
        assert torch.equal(out, ref_h[:n]) and torch.equal(logits, ref_l[:n]), n
        assert torch.equal(pol.cell(xd[:n], hd[:n]), ref_h[:n]), n
    pol.status()
    pol.close()


def test_other_shapes_odd_obs_dim_and_eight_actions(torch_cuda):
    """obs_dim 5 takes the scalar-load path of the encoder, 8 actions the two-vector path of the head;
    hidden 896 is the largest the fused entry point takes, 960 must be refused by it."""
    torch = torch_cuda
    H, n = 192, 777
    w = policy_weights(H, 71, obs_dim=5, n_actions=8)
    rng = np.random.Generator(np.random.PCG64(72))
    obs = rng.uniform(-1.0, 1.0, (n, 5)).astype(np.float32)
    hvals = bf16_values((n, H), 73, -7, 0)
    pol = gp.GruPolicy(w)
    x = pol.encode(torch.from_numpy(obs).cuda())
    assert np.array_equal(from_dev_bf16(torch, x).view(np.uint32),
                          ogp.encode(obs, w["enc_w"], w["enc_b"]).view(np.uint32))
    logits = pol.head(to_dev_bf16(torch, hvals)).cpu().numpy().astype(np.float64)
    want_l, mag = ogp.head(hvals, w["head_w"], w["head_b"], with_abs_sum=True)
    assert np.all(np.abs(logits - want_l) <= head_tolerance(mag, H))
    with pytest.raises(gp.GruPolicyError) as e:      # more than 4 actions: not through the fused call
        pol.cell_head(x, to_dev_bf16(torch, hvals))
    assert e.value.code == -1
    pol.status(); pol.close()
    for H, fused in ((896, True), (960, False)):
        w = policy_weights(H, 74)
        xs, hs = policy_activations(130, H, 75)
        pol = gp.GruPolicy(w)
        xd, hd = to_dev_bf16(torch, xs), to_dev_bf16(torch, hs)
        h1 = pol.cell(xd, hd)
        want = ogp.cell(xs, hs, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"])
        assert np.all(np.abs(from_dev_bf16(torch, h1) - want) <= cell_tolerance(want))
        if fused:
            h2, l2 = pol.cell_head(xd, hd)
            assert torch.equal(h1, h2) and torch.equal(l2, pol.head(h1))
        else:
            with pytest.raises(gp.GruPolicyError) as e:
                pol.cell_head(xd, hd)
            assert e.value.code == -1
        pol.status(); pol.close()


def test_argument_errors(torch_cuda):
    torch = torch_cuda
    w = policy_weights(64, 51)
    with pytest.raises(gp.GruPolicyError) as e:
        gp.gru_policy_create(96, 6, 3, policy_weights(96, 1))
    assert e.value.code == -1
    pol = gp.GruPolicy(w)
    x = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    h = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((9, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gp.GruPolicyError) as e:
        gp.gru_policy_cell(pol.h, x, h, None, 8)
    assert e.value.code == -2
    with pytest.raises(gp.GruPolicyError) as e:
        gp.gru_policy_cell(pol.h, x, h, h, 8)
    assert e.value.code == -1
    with pytest.raises(gp.GruPolicyError) as e:
        gp.gru_policy_cell(pol.h, x, h, out.data_ptr() + 2, 8)
    assert e.value.code == -3
    with pytest.raises(gp.GruPolicyError) as e:
        gp.gru_policy_cell(pol.h, x, h, out, 0)
    assert e.value.code == -1
    logits = torch.zeros((8, 3), device="cuda")
    ws = pol.workspace(8)
    with pytest.raises(gp.GruPolicyError) as e:      # scratch must be 16-byte aligned
        gp.gru_policy_cell_head(pol.h, x, h, out, logits, ws.data_ptr() + 4, 8)
    assert e.value.code == -3
    with pytest.raises(gp.GruPolicyError) as e:
        gp.gru_policy_cell_head(pol.h, x, h, out, logits, None, 8)
    assert e.value.code == -2
    obs = torch.zeros((9, 6), device="cuda")
    with pytest.raises(gp.GruPolicyError) as e:      # obs rows are read in pairs: 8-byte alignment
        gp.gru_policy_encode(pol.h, obs.data_ptr() + 4, None, None, x, 8)
    assert e.value.code == -3
    pol.status()
    pol.close()


def test_two_policies_of_different_hidden_size_alive_together(torch_cuda):
    """The kernels' shared-memory limits belong to the kernel, not to a handle: creating a small
    policy after a large one must not take the large one's launch configuration away."""
    torch = torch_cuda
    big_w, small_w = policy_weights(1024, 91), policy_weights(64, 92)
    big = gp.GruPolicy(big_w)
    small = gp.GruPolicy(small_w)          # created second: would lower the limits if they were per handle
    rng = np.random.Generator(np.random.PCG64(93))
    for pol, w, H in ((big, big_w, 1024), (small, small_w, 64), (big, big_w, 1024)):
        x, h = policy_activations(130, H, 94)
        obs = rng.uniform(-0.1, 1.1, (130, 6)).astype(np.float32)
        xe = pol.encode(torch.from_numpy(obs).cuda())
        assert np.array_equal(from_dev_bf16(torch, xe).view(np.uint32),
                              ogp.encode(obs, w["enc_w"], w["enc_b"]).view(np.uint32))
        out = pol.cell(to_dev_bf16(torch, x), to_dev_bf16(torch, h))
        want = ogp.cell(x, h, w["w_ih"], w["w_hh"], w["b_ih"], w["b_hh"])
        assert np.all(np.abs(from_dev_bf16(torch, out) - want) <= cell_tolerance(want))
        logits = pol.head(to_dev_bf16(torch, h)).cpu().numpy().astype(np.float64)
        assert np.array_equal(logits, ogp.head(h, w["head_w"], w["head_b"]))
        pol.status()
    big.close(); small.close()
