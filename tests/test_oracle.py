"""Pins for the fp64 CPU oracle: closed forms, invariants and brute force (no GPU).

Each test fixes the oracle to something other than itself, so that a dropped term,
a wrong sign or index, or a transposed operand in it fails at least one of them.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_fractions(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([float(Fraction(v)) for v in vals])
    return out


def _rand(B, H, n, d, seed, scale=1.0, wscale=None):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((B, H, n, d)).astype(np.float32) * scale for _ in range(3))
    ws = (1.0 / (math.sqrt(d) * scale)) if wscale is None else wscale
    Wq, Wk = (rng.standard_normal((H, d, d // 2)).astype(np.float32) * ws for _ in range(2))
    return q, k, v, Wq.astype(np.float32), Wk.astype(np.float32)


# ---- hand-derived worked examples (tests/golden) -------------------------------------------

def test_closed_form_d4_n2():
    """Eq. 5 + Eq. 6 against fractions derived by hand (distinct W_q / W_k, decoy coordinates)."""
    g = _read_fractions("closed_form_d4_n2.txt")
    ln = math.log
    q = np.array([[ln(3), 7, 0, -2], [0, 1, ln(2), 5]], dtype=np.float32)[None, None]
    k = np.array([[9, ln(4), -1, 0], [3, 0, 3, 0]], dtype=np.float32)[None, None]
    v = np.array([[1, 0, -2, 4], [0, 10, 2, -4]], dtype=np.float32)[None, None]
    Wq = np.array([[1, 0], [0, 0], [0, 1], [0, 0]], dtype=np.float32)
    Wk = np.array([[0, 0], [1, 0], [0, 0], [0, 1]], dtype=np.float32)
    tol = 1e-6  # ln(.) is rounded to float32 on input
    np.testing.assert_allclose(oracle.phi(q[0, 0], Wq), np.stack([g["phi_q1"], g["phi_q2"]]), atol=tol)
    np.testing.assert_allclose(oracle.phi(k[0, 0], Wk), np.stack([g["phi_k1"], g["phi_k2"]]), atol=tol)
    want_o = np.stack([g["o_1"], g["o_2"]])
    want_S = np.stack([g["S_0"], g["S_1"], g["S_2"], g["S_3"]])
    o_lin, S, z = oracle.ref_linear(q, k, v, Wq, Wk, return_state=True)
    np.testing.assert_allclose(o_lin[0, 0], want_o, atol=tol)
    np.testing.assert_allclose(S[0, 0], want_S, atol=tol)
    np.testing.assert_allclose(z[0, 0], g["z"], atol=tol)
    np.testing.assert_allclose(oracle.ref_quadratic(q, k, v, Wq, Wk)[0, 0], want_o, atol=tol)
    # per-head weight layout [H, d, d/2] with H = 1 gives the same
    np.testing.assert_allclose(oracle.ref_linear(q, k, v, Wq[None], Wk[None])[0, 0], want_o, atol=tol)


def test_closed_form_phi_d6():
    g = _read_fractions("phi_d6.txt")
    W = np.zeros((6, 3), dtype=np.float32)
    W[0, 0] = 1.0
    W[2, 2] = 0.5
    x = np.array([[math.log(2), 5, math.log(16), 1, -3, 0]], dtype=np.float32)
    np.testing.assert_allclose(oracle.phi(x, W)[0], g["phi"], atol=1e-6)


# ---- Eq. 5: the two forms agree (brute force) ------------------------------------------------

@pytest.mark.parametrize("B,H,n,d", [(1, 2, 1024, 64), (2, 3, 37, 8), (1, 1, 129, 128), (1, 2, 5, 2)])
def test_linear_equals_quadratic(B, H, n, d):
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=n + d)
    a = oracle.ref_quadratic(q, k, v, Wq, Wk)
    b = oracle.ref_linear(q, k, v, Wq, Wk)
    assert np.abs(a - b).max() <= 1e-12 * max(1.0, np.abs(a).max())


def test_rows_subset_matches_full():
    q, k, v, Wq, Wk = _rand(1, 2, 200, 16, seed=3)
    rows = np.array([0, 199, 57, 57, 3])
    full = oracle.ref_linear(q, k, v, Wq, Wk)
    np.testing.assert_array_equal(oracle.ref_linear(q, k, v, Wq, Wk, rows=rows), full[:, :, rows])
    np.testing.assert_array_equal(oracle.ref_quadratic(q, k, v, Wq, Wk, rows=rows),
                                  oracle.ref_quadratic(q, k, v, Wq, Wk)[:, :, rows])


# ---- library routine with independent arithmetic --------------------------------------------

def test_against_torch_sdpa_fp64():
    """softmax(log A) is the row-normalised A, so torch's fp64 SDPA with q = 0 and additive mask
    log A evaluates the left form of Eq. 5 through a library routine."""
    B, H, n, d = 1, 2, 96, 16
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=11)
    tq, tk, tv = (torch.from_numpy(t).double() for t in (q, k, v))
    tWq, tWk = torch.from_numpy(Wq).double(), torch.from_numpy(Wk).double()

    def fmap(x, W):
        u = torch.einsum("bhnd,hdm->bhnm", x, W)
        return torch.cat([torch.softmax(u, -1), torch.softmax(-u, -1)], -1)

    A = torch.einsum("bhif,bhjf->bhij", fmap(tq, tWq), fmap(tk, tWk))
    want = torch.nn.functional.scaled_dot_product_attention(torch.zeros_like(tq), tk, tv, attn_mask=A.log())
    got = oracle.ref_linear(q, k, v, Wq, Wk)
    np.testing.assert_allclose(got, want.numpy(), rtol=0, atol=1e-12)


# ---- closed forms and invariants ---------------------------------------------------------------

def test_constant_feature_map_gives_mean_of_v():
    """W = 0 makes phi the constant 2/d, so every output row is the mean of V."""
    q, k, v, _, _ = _rand(2, 2, 77, 16, seed=5)
    W0 = np.zeros((2, 16, 8), dtype=np.float32)
    want = v.astype(np.float64).mean(axis=2, keepdims=True)
    for fn in (oracle.ref_linear, oracle.ref_quadratic):
        got = fn(q, k, v, W0, W0)
        np.testing.assert_allclose(got, np.broadcast_to(want, got.shape), atol=1e-13)


def test_d2_is_mean_of_v():
    """d = 2: each softmax is over one feature, phi = (1, 1) whatever W is."""
    q, k, v, Wq, Wk = _rand(1, 3, 40, 2, seed=6, wscale=3.0)
    want = v.astype(np.float64).mean(axis=2, keepdims=True)
    got = oracle.ref_linear(q, k, v, Wq, Wk)
    np.testing.assert_allclose(got, np.broadcast_to(want, got.shape), atol=1e-13)
    np.testing.assert_array_equal(oracle.phi(q[0, 0], Wq[0]), np.ones((40, 2)))


def test_single_token_returns_v():
    q, k, v, Wq, Wk = _rand(2, 2, 1, 32, seed=7)
    for fn in (oracle.ref_linear, oracle.ref_quadratic):
        np.testing.assert_allclose(fn(q, k, v, Wq, Wk), v.astype(np.float64), rtol=1e-14)


def test_phi_structure_and_state_sums():
    """Eq. 6: entries in (0, 1], each half sums to 1; hence sum(z) = 2 n and sum_f S[f, c] = 2 sum_j v_jc."""
    q, k, v, Wq, Wk = _rand(1, 2, 300, 64, seed=8, wscale=0.5)
    p = oracle.phi(k[0, 1], Wk[1])
    assert (p > 0).all() and (p <= 1).all()
    np.testing.assert_allclose(p[:, :32].sum(-1), 1.0, rtol=1e-14)
    np.testing.assert_allclose(p[:, 32:].sum(-1), 1.0, rtol=1e-14)
    # the second half is the first half's map applied to the negated input
    np.testing.assert_allclose(p[:, 32:], oracle.phi(-k[0, 1], Wk[1])[:, :32], rtol=1e-14)
    _, S, z = oracle.ref_linear(q, k, v, Wq, Wk, return_state=True)
    np.testing.assert_allclose(z.sum(-1), 2.0 * 300, rtol=1e-13)
    np.testing.assert_allclose(S.sum(-2), 2.0 * v.astype(np.float64).sum(2), atol=1e-11)
    # z and S restated from phi with numpy
    np.testing.assert_allclose(z[0, 1], p.sum(0), rtol=1e-13)
    np.testing.assert_allclose(S[0, 1], p.T @ v[0, 1].astype(np.float64), atol=1e-11)


def test_phi_is_shift_stable():
    """Large logits must not overflow: softmax is invariant to adding a constant to all logits."""
    W = np.zeros((4, 2), dtype=np.float32)
    W[0, 0] = 1.0
    W[1, 1] = 1.0
    x = np.array([[1000.0, 999.0, 0, 0], [-1000.0, -1001.0, 0, 0]], dtype=np.float32)
    e = math.e
    want = np.array([e / (1 + e), 1 / (1 + e), 1 / (1 + e), e / (1 + e)])
    got = oracle.phi(x, W)
    np.testing.assert_allclose(got[0], want, rtol=1e-14)
    np.testing.assert_allclose(got[1], want, rtol=1e-14)


def test_key_value_permutation_invariance_and_query_equivariance():
    q, k, v, Wq, Wk = _rand(1, 2, 150, 16, seed=9)
    base = oracle.ref_linear(q, k, v, Wq, Wk)
    perm = np.random.default_rng(1).permutation(150)
    np.testing.assert_allclose(oracle.ref_linear(q, k[:, :, perm], v[:, :, perm], Wq, Wk), base, atol=1e-13)
    np.testing.assert_allclose(oracle.ref_linear(q[:, :, perm], k, v, Wq, Wk), base[:, :, perm], atol=1e-15)
    # permuting only the keys (not the values) must change the result: k_j and v_j are paired
    assert np.abs(oracle.ref_linear(q, k[:, :, perm], v, Wq, Wk) - base).max() > 1e-3


def test_convex_combination_shift_and_linearity_in_v():
    q, k, v, Wq, Wk = _rand(1, 2, 120, 16, seed=10)
    o = oracle.ref_linear(q, k, v, Wq, Wk)
    v64 = v.astype(np.float64)
    assert (o <= v64.max(axis=2, keepdims=True) + 1e-12).all()
    assert (o >= v64.min(axis=2, keepdims=True) - 1e-12).all()
    shift = np.float32(2.0)  # exact in float32 for these magnitudes? compare against the shifted floats
    v2 = (v + shift).astype(np.float32)
    np.testing.assert_allclose(oracle.ref_linear(q, k, v2, Wq, Wk) - o,
                               (v2.astype(np.float64) - v64).mean() * np.ones_like(o), atol=1e-6)
    np.testing.assert_allclose(oracle.ref_linear(q, k, (2 * v).astype(np.float32), Wq, Wk), 2 * o, rtol=1e-14)


def test_duplicating_every_key_value_pair_changes_nothing():
    q, k, v, Wq, Wk = _rand(1, 2, 60, 16, seed=12)
    base = oracle.ref_linear(q, k, v, Wq, Wk)
    k2, v2 = np.repeat(k, 2, axis=2), np.repeat(v, 2, axis=2)
    q2 = np.concatenate([q, q], axis=2)
    o2, S2, z2 = oracle.ref_linear(q2, k2, v2, Wq, Wk, return_state=True)
    _, S, z = oracle.ref_linear(q, k, v, Wq, Wk, return_state=True)
    np.testing.assert_allclose(o2[:, :, :60], base, atol=1e-13)
    np.testing.assert_allclose(S2, 2 * S, atol=1e-12)
    np.testing.assert_allclose(z2, 2 * z, atol=1e-12)


def test_heads_and_batches_are_independent_and_use_their_own_weights():
    q, k, v, Wq, Wk = _rand(2, 3, 50, 8, seed=13)
    full = oracle.ref_linear(q, k, v, Wq, Wk)
    for b in range(2):
        for h in range(3):
            one = oracle.ref_linear(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1], v[b:b + 1, h:h + 1], Wq[h], Wk[h])
            np.testing.assert_array_equal(one[0, 0], full[b, h])
    # shared-weights mode equals per-head mode with the same matrix repeated
    shared = oracle.ref_linear(q, k, v, Wq[1], Wk[2])
    rep = oracle.ref_linear(q, k, v, np.repeat(Wq[1:2], 3, 0), np.repeat(Wk[2:3], 3, 0))
    np.testing.assert_array_equal(shared, rep)


def test_query_and_key_weights_are_not_interchangeable():
    q, k, v, Wq, Wk = _rand(1, 1, 64, 16, seed=14, wscale=1.0)
    a = oracle.ref_linear(q, k, v, Wq, Wk)
    b = oracle.ref_linear(q, k, v, Wk, Wq)
    assert np.abs(a - b).max() > 1e-3


def test_bad_arguments_are_rejected():
    q, k, v, Wq, Wk = _rand(1, 1, 4, 4, seed=15)
    with pytest.raises(AssertionError):
        oracle.ref_linear(q, k, v[:, :, :3], Wq, Wk)
    with pytest.raises(AssertionError):
        oracle.ref_linear(q, k, v, Wq, Wk, rows=np.array([4]))


# ---- Eq. 8: softmax-attention term and the blend ---------------------------------------------------

def test_mixed_attention_hand_example():
    gold = _read_fractions("mixed_n2_d2.txt")
    q = np.array([[[[1.0, 0.0], [0.0, 1.0]]]], dtype=np.float32)
    k = np.array([[[[math.log(3.0), math.log(4.0)], [0.0, 0.0]]]], dtype=np.float32)
    v = np.array([[[[4.0, 8.0], [0.0, -4.0]]]], dtype=np.float32)
    o = oracle.ref_softmax(q, k, v, scale=1.0)
    np.testing.assert_allclose(o[0, 0, 0], gold["softmax_o1"], rtol=0, atol=1e-6)
    np.testing.assert_allclose(o[0, 0, 1], gold["softmax_o2"], rtol=0, atol=1e-6)
    lin = np.ones_like(o)
    want = np.stack([gold["mix_o1"], gold["mix_o2"]])[None, None]
    np.testing.assert_allclose(oracle.ref_mix(o, lin, 0.25), want, rtol=0, atol=1e-6)
    np.testing.assert_array_equal(oracle.ref_mix(o, lin, 1.75), o)      # clipped to 1: the softmax term alone
    np.testing.assert_array_equal(oracle.ref_mix(o, lin, -0.5), lin)    # clipped to 0: the linear term alone


@pytest.mark.parametrize("scale", [1.0, 0.25, 1.0 / 8.0])
def test_softmax_term_matches_library_attention(scale):
    """torch's fp64 scaled_dot_product_attention is an independent implementation of the same definition."""
    rng = np.random.default_rng(5)
    q, k, v = (rng.standard_normal((2, 3, 37, 16)).astype(np.float32) for _ in range(3))
    got = oracle.ref_softmax(q, k, v, scale=scale)
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).double(), torch.from_numpy(k).double(), torch.from_numpy(v).double(), scale=scale).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)
    rows = np.array([0, 5, 36])
    np.testing.assert_allclose(oracle.ref_softmax(q, k, v, scale=scale, rows=rows), want[:, :, rows], rtol=1e-10, atol=1e-12)


def test_softmax_term_special_cases():
    rng = np.random.default_rng(6)
    q, k, v = (rng.standard_normal((1, 2, 50, 8)).astype(np.float32) for _ in range(3))
    # all keys equal -> uniform weights -> the mean of V, for every query
    kc = np.broadcast_to(k[:, :, :1], k.shape).copy()
    mean_v = v.astype(np.float64).mean(axis=2, keepdims=True)
    np.testing.assert_allclose(oracle.ref_softmax(q, kc, v, scale=0.7), np.broadcast_to(mean_v, v.shape), rtol=1e-12, atol=1e-12)
    # a very sharp softmax picks the value of the best-matching key
    o = oracle.ref_softmax(q, k, v, scale=1e4)
    best = np.einsum("bhid,bhjd->bhij", q.astype(np.float64), k.astype(np.float64)).argmax(-1)
    np.testing.assert_allclose(o, np.take_along_axis(v.astype(np.float64), best[..., None], axis=2), rtol=0, atol=1e-9)
    # logits of +-1e4 must not overflow
    assert np.isfinite(o).all()
    # joint permutation of (k, v) changes nothing
    perm = rng.permutation(50)
    np.testing.assert_allclose(oracle.ref_softmax(q, k[:, :, perm], v[:, :, perm], scale=0.3),
                               oracle.ref_softmax(q, k, v, scale=0.3), rtol=1e-12, atol=1e-13)


def test_mix_is_affine_in_the_clipped_score():
    rng = np.random.default_rng(7)
    a, b = rng.standard_normal((2, 3, 4, 5)), rng.standard_normal((2, 3, 4, 5))
    m0, m1 = oracle.ref_mix(a, b, 0.0), oracle.ref_mix(a, b, 1.0)
    np.testing.assert_array_equal(m0, b)
    np.testing.assert_array_equal(m1, a)
    for r in (0.1, 0.5, 0.9):
        np.testing.assert_allclose(oracle.ref_mix(a, b, r), m0 + r * (m1 - m0), rtol=1e-13, atol=1e-14)
    np.testing.assert_array_equal(oracle.ref_mix(a, b, 3.0), m1)
    np.testing.assert_array_equal(oracle.ref_mix(a, b, -3.0), m0)


# ---- gradients (what Eq. 14 back-propagates through the operator) ----------------------------------------

def _torch_forward(q, k, v, Wq, Wk):
    """The operator in plain torch fp64 (Eq. 5 left form, Eq. 6), written independently of the C oracle so that
    autograd gives a second opinion on its hand-derived chain rule."""
    def phi(x, W):
        u = torch.einsum("bhnd,hdm->bhnm", x, W)
        return torch.cat([torch.softmax(u, -1), torch.softmax(-u, -1)], -1)
    a = torch.einsum("bhif,bhjf->bhij", phi(q, Wq), phi(k, Wk))
    return torch.einsum("bhij,bhjd->bhid", a / a.sum(-1, keepdim=True), v)


@pytest.mark.parametrize("B,H,n,d", [(1, 1, 5, 4), (2, 2, 9, 8), (1, 3, 17, 16)])
def test_backward_matches_autograd_of_an_independent_forward(B, H, n, d):
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=50 + n)
    g = np.random.default_rng(51).standard_normal((B, H, n, d)).astype(np.float32)
    t = [torch.from_numpy(x).double().requires_grad_(True) for x in (q, k, v, Wq, Wk)]
    (_torch_forward(*t) * torch.from_numpy(g).double()).sum().backward()
    got = oracle.ref_backward(q, k, v, Wq, Wk, g)
    for name, a, b in zip(("dq", "dk", "dv", "dWq", "dWk"), got, t):
        np.testing.assert_allclose(a, b.grad.numpy(), rtol=1e-9, atol=1e-12, err_msg=name)


def test_backward_matches_central_differences_of_the_forward_oracle():
    """The forward oracle is pinned above; its central differences pin every gradient of the backward oracle."""
    B, H, n, d = 1, 2, 6, 4
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=60)
    g = np.random.default_rng(61).standard_normal((B, H, n, d))
    # inputs must be exactly representable in float32 after +-h: use a power of two
    h = 2.0 ** -10
    grads = oracle.ref_backward(q, k, v, Wq, Wk, g.astype(np.float32))
    g32 = g.astype(np.float32).astype(np.float64)
    args = [q, k, v, Wq, Wk]
    rng = np.random.default_rng(62)
    for a_i, (arr, grad) in enumerate(zip(args, grads)):
        for _ in range(6):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            plus, minus = [x.copy() for x in args], [x.copy() for x in args]
            plus[a_i][idx] += h
            minus[a_i][idx] -= h
            fd = ((oracle.ref_linear(*plus) - oracle.ref_linear(*minus)) * g32).sum() / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-5 * max(1.0, abs(grad[idx])), (a_i, idx, fd, grad[idx])


def test_backward_shared_weights_sum_over_heads_and_invariances():
    B, H, n, d = 2, 3, 7, 8
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=70)
    g = np.random.default_rng(71).standard_normal((B, H, n, d)).astype(np.float32)
    shared_q, shared_k = Wq[0].copy(), Wk[0].copy()
    rep = lambda W: np.broadcast_to(W, (H,) + W.shape).copy()
    per = oracle.ref_backward(q, k, v, rep(shared_q), rep(shared_k), g)
    sh = oracle.ref_backward(q, k, v, shared_q, shared_k, g)
    for a, b in zip(per[:3], sh[:3]):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(per[3].sum(0), sh[3], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(per[4].sum(0), sh[4], rtol=1e-11, atol=1e-13)
    # dO = 0 gives all-zero gradients
    zero = oracle.ref_backward(q, k, v, Wq, Wk, np.zeros_like(g))
    assert all(np.all(x == 0.0) for x in zero)
    # and the gradients are linear in dO
    two = oracle.ref_backward(q, k, v, Wq, Wk, 2.0 * g)
    one = oracle.ref_backward(q, k, v, Wq, Wk, g)
    for a, b in zip(two, one):
        np.testing.assert_allclose(a, 2.0 * b, rtol=1e-12, atol=1e-14)


# ---- the ReLU kernel function of the paper's kernel-function ablation ---------------------------------------

def _qkv(B, H, n, d, seed):
    rng = np.random.default_rng(seed)
    return tuple(rng.standard_normal((B, H, n, d)).astype(np.float32) for _ in range(3))


@pytest.mark.parametrize("B,H,n,d", [(1, 1, 7, 4), (2, 2, 33, 8), (1, 2, 300, 64)])
def test_relu_linear_form_equals_quadratic_form_and_a_library_computation(B, H, n, d):
    q, k, v = _qkv(B, H, n, d, seed=80 + n)
    lin, S, z = oracle.ref_relu_linear(q, k, v, return_state=True)
    quad = oracle.ref_relu_quadratic(q, k, v)
    np.testing.assert_allclose(lin, quad, rtol=1e-10, atol=1e-12)
    # the same through torch's matmuls in fp64: A = relu(Q) relu(K)^T, O = (A / rowsum) V
    tq, tk, tv = (torch.from_numpy(x).double() for x in (q, k, v))
    A = torch.relu(tq) @ torch.relu(tk).transpose(-1, -2)
    want = (A / A.sum(-1, keepdim=True)) @ tv
    np.testing.assert_allclose(quad, want.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(S, (torch.relu(tk).transpose(-1, -2) @ tv).numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(z, torch.relu(tk).sum(-2).numpy(), rtol=1e-12, atol=1e-12)


def test_relu_closed_forms():
    B, H, n, d = 1, 2, 40, 8
    q, k, v = _qkv(B, H, n, d, seed=90)
    base = oracle.ref_relu_linear(q, k, v)
    # positively homogeneous: scaling q or k by a positive (power-of-two) factor leaves o unchanged
    np.testing.assert_allclose(oracle.ref_relu_linear(4.0 * q, 0.25 * k, v), base, rtol=1e-12, atol=1e-14)
    # negative entries are ignored: replacing them by other negative values changes nothing
    q2 = np.where(q < 0, 3.0 * q, q).astype(np.float32)
    k2 = np.where(k < 0, -1.0, k).astype(np.float32)
    np.testing.assert_array_equal(oracle.ref_relu_linear(q2, k2, v), base)
    # keys that are all equal and positive: every weight is equal, o = mean of V
    kc = np.ones_like(k)
    np.testing.assert_allclose(oracle.ref_relu_linear(np.abs(q), kc, v), np.broadcast_to(v.astype(np.float64).mean(2, keepdims=True), v.shape),
                               rtol=1e-12, atol=1e-13)
    # one-hot queries and keys pick out the average of the values whose key shares the query's feature
    e = np.zeros((1, 1, 4, 4), dtype=np.float32)
    e[0, 0, np.arange(4), [0, 1, 0, 1]] = 1.0
    vv = np.arange(16, dtype=np.float32).reshape(1, 1, 4, 4)
    o = oracle.ref_relu_linear(e, e, vv)
    np.testing.assert_allclose(o[0, 0, 0], (vv[0, 0, 0] + vv[0, 0, 2]) / 2)
    np.testing.assert_allclose(o[0, 0, 1], (vv[0, 0, 1] + vv[0, 0, 3]) / 2)
    # rows subset
    rows = np.array([3, 17, 39])
    np.testing.assert_array_equal(oracle.ref_relu_linear(q, k, v, rows=rows), base[:, :, rows])
    np.testing.assert_allclose(oracle.ref_relu_quadratic(q, k, v, rows=rows), base[:, :, rows], rtol=1e-10, atol=1e-12)


def test_backward_closed_forms():
    """Cases where the gradients are known without any computation.
    d = 2: one logit per half, so phi = [1, 1] whatever q, k, W are: o_i is the mean of V, dq = dk = dW = 0 and every
    dv_j is the mean of dO over the queries.  n = 1: o_1 = v_1, so dv = dO and the rest vanishes."""
    rng = np.random.default_rng(95)
    B, H, n, d = 2, 2, 6, 2
    q, k, v = (rng.standard_normal((B, H, n, d)).astype(np.float32) for _ in range(3))
    Wq, Wk = (rng.standard_normal((H, d, 1)).astype(np.float32) for _ in range(2))
    g = rng.standard_normal((B, H, n, d)).astype(np.float32)
    dq, dk, dv, dWq, dWk = oracle.ref_backward(q, k, v, Wq, Wk, g)
    for z in (dq, dk, dWq, dWk):
        assert np.abs(z).max() <= 1e-15
    np.testing.assert_allclose(dv, np.broadcast_to(g.astype(np.float64).mean(2, keepdims=True), g.shape), rtol=1e-13, atol=1e-15)
    B, H, n, d = 1, 3, 1, 8
    q, k, v = (rng.standard_normal((B, H, n, d)).astype(np.float32) for _ in range(3))
    Wq, Wk = (rng.standard_normal((H, d, d // 2)).astype(np.float32) for _ in range(2))
    g = rng.standard_normal((B, H, n, d)).astype(np.float32)
    dq, dk, dv, dWq, dWk = oracle.ref_backward(q, k, v, Wq, Wk, g)
    for z in (dq, dk, dWq, dWk):
        assert np.abs(z).max() <= 1e-12
    np.testing.assert_allclose(dv, g.astype(np.float64), rtol=1e-13, atol=1e-15)


# ---- gradients through Eq. 8 (mixed attention) and with the ReLU kernel function ------------------------------

@pytest.mark.parametrize("r", [0.3, 0.0, 1.0, -0.2, 1.4])
def test_mixed_backward_matches_autograd_of_an_independent_forward(r):
    """torch fp64 autograd through clamp(r) * a + (1 - clamp(r)) * [Eq. 5, left form]: every gradient, the one of the
    softmax branch's output and the one of r included.  torch's clamp passes the gradient on the closed interval
    [0, 1] (ends included) and blocks it outside, which is the reading the oracle states."""
    B, H, n, d = 2, 2, 7, 8
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=80)
    rng = np.random.default_rng(81)
    g = rng.standard_normal((B, H, n, d)).astype(np.float32)
    a = rng.standard_normal((B, H, n, d)).astype(np.float32)
    t = [torch.from_numpy(x).double().requires_grad_(True) for x in (q, k, v, Wq, Wk, a)]
    rt = torch.tensor(r, dtype=torch.float64, requires_grad=True)
    rc = torch.clamp(rt, 0.0, 1.0)
    out = rc * t[5] + (1.0 - rc) * _torch_forward(*t[:5])
    (out * torch.from_numpy(g).double()).sum().backward()
    got = oracle.ref_backward_mixed(q, k, v, Wq, Wk, a, r, g)
    for name, x, y in zip(("dq", "dk", "dv", "dWq", "dWk", "da"), got[:6], t):
        np.testing.assert_allclose(x, y.grad.numpy(), rtol=1e-9, atol=1e-12, err_msg=name)
    np.testing.assert_allclose(got[6], rt.grad.item(), rtol=1e-9, atol=1e-12)
    if r < 0.0 or r > 1.0:
        assert got[6] == 0.0


def test_mixed_backward_special_cases_and_central_difference_in_r():
    B, H, n, d = 1, 2, 6, 4
    q, k, v, Wq, Wk = _rand(B, H, n, d, seed=82)
    rng = np.random.default_rng(83)
    g = rng.standard_normal((B, H, n, d)).astype(np.float32)
    a = rng.standard_normal((B, H, n, d)).astype(np.float32)
    # r = 0: the layer IS the linear branch
    plain = oracle.ref_backward(q, k, v, Wq, Wk, g)
    at0 = oracle.ref_backward_mixed(q, k, v, Wq, Wk, a, 0.0, g)
    for x, y in zip(plain, at0[:5]):
        np.testing.assert_array_equal(x, y)
    assert np.abs(at0[5]).max() == 0.0
    # r = 1: nothing reaches the linear branch, the softmax branch gets dout unchanged
    at1 = oracle.ref_backward_mixed(q, k, v, Wq, Wk, a, 1.0, g)
    for x in at1[:5]:
        assert np.abs(x).max() == 0.0
    np.testing.assert_array_equal(at1[5], g.astype(np.float64))
    # dr against a central difference of the pinned forward (ref_mix of ref_linear); the blend is affine in r^
    lin = oracle.ref_linear(q, k, v, Wq, Wk)
    h = 2.0 ** -12
    fd = ((oracle.ref_mix(a, lin, 0.4 + h) - oracle.ref_mix(a, lin, 0.4 - h)) * g.astype(np.float64)).sum() / (2 * h)
    dr = oracle.ref_backward_mixed(q, k, v, Wq, Wk, a, 0.4, g)[6]
    assert abs(fd - dr) <= 1e-8 * max(1.0, abs(dr))
    # and linear in (1 - r^) for everything that passes through the linear branch
    half = oracle.ref_backward_mixed(q, k, v, Wq, Wk, a, 0.5, g)
    for x, y in zip(plain, half[:5]):
        np.testing.assert_allclose(0.5 * x, y, rtol=1e-13, atol=1e-15)


def _torch_relu_forward(q, k, v):
    a = torch.einsum("bhif,bhjf->bhij", torch.relu(q), torch.relu(k))
    return torch.einsum("bhij,bhjd->bhid", a / a.sum(-1, keepdim=True), v)


@pytest.mark.parametrize("B,H,n,d", [(1, 1, 5, 4), (2, 3, 11, 8)])
def test_relu_backward_matches_autograd_and_central_differences(B, H, n, d):
    q, k, v = _qkv(B, H, n, d, seed=90 + n)
    g = np.random.default_rng(91).standard_normal((B, H, n, d)).astype(np.float32)
    t = [torch.from_numpy(x).double().requires_grad_(True) for x in (q, k, v)]
    (_torch_relu_forward(*t) * torch.from_numpy(g).double()).sum().backward()
    got = oracle.ref_relu_backward(q, k, v, g)
    for name, x, y in zip(("dq", "dk", "dv"), got, t):
        np.testing.assert_allclose(x, y.grad.numpy(), rtol=1e-9, atol=1e-12, err_msg=name)
    # central differences of the pinned ReLU forward oracle (away from the kink: |x| > 2h for the sampled entries)
    h = 2.0 ** -10
    rng = np.random.default_rng(92)
    args = [q, k, v]
    for a_i, (arr, grad) in enumerate(zip(args, got)):
        done = 0
        while done < 5:
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            if abs(arr[idx]) <= 4 * h:
                continue
            plus, minus = [x.copy() for x in args], [x.copy() for x in args]
            plus[a_i][idx] += h
            minus[a_i][idx] -= h
            fd = ((oracle.ref_relu_linear(*plus) - oracle.ref_relu_linear(*minus)) * g.astype(np.float64)).sum() / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-5 * max(1.0, abs(grad[idx])), (a_i, idx, fd, grad[idx])
            done += 1


def test_relu_backward_closed_forms():
    """Negative entries of q and k get no gradient; n = 1 returns v, so dv = dO and dq = dk = 0."""
    rng = np.random.default_rng(93)
    q, k, v = (rng.standard_normal((1, 2, 9, 8)).astype(np.float32) for _ in range(3))
    g = rng.standard_normal((1, 2, 9, 8)).astype(np.float32)
    dq, dk, dv = oracle.ref_relu_backward(q, k, v, g)
    assert np.abs(dq[q <= 0]).max() == 0.0 and np.abs(dk[k <= 0]).max() == 0.0
    assert np.abs(dq[q > 0]).min() > 0.0
    q1, k1, v1, g1 = (x[:, :, :1].copy() for x in (np.abs(q) + 0.1, np.abs(k) + 0.1, v, g))
    dq, dk, dv = oracle.ref_relu_backward(q1, k1, v1, g1)
    assert np.abs(dq).max() <= 1e-12 and np.abs(dk).max() <= 1e-12
    np.testing.assert_allclose(dv, g1.astype(np.float64), rtol=1e-13, atol=1e-15)
