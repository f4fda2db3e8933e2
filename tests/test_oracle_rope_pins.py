"""Pins for the oracle's tensorized positional encoding (Section 3.2: the position of a token is
its coordinate vector and RoPE encodes it; reading: hop i rotates queries and keys by the
coordinate along dimension i, Llama pairing c <-> c + D/2, angle p * base^(-2c/D)).

Each check compares the C route (which rotates vectors) with something that does not share its
formula: the dense route (relative-phase form on complex features, no rotation anywhere), a
block-matrix implementation for one dimension, closed-form sin / cos scores, invariants."""
import math

import numpy as np
import pytest

import oracle

BASE = 10000.0


def rotation_matrix(p, D, base):
    """D x D orthogonal matrix of RoPE at position p (pairs c, c + D/2), built entry by entry."""
    r = np.zeros((D, D))
    half = D // 2
    for c in range(half):
        a = p * base ** (-2.0 * c / D)
        r[c, c] = math.cos(a)
        r[c, c + half] = -math.sin(a)
        r[c + half, c] = math.sin(a)
        r[c + half, c + half] = math.cos(a)
    return r


def rope_attention_one_dim(q, k, v, causal, base):
    from scipy.special import softmax
    n, d = q.shape
    qr = np.stack([rotation_matrix(t, d, base) @ q[t] for t in range(n)])
    kr = np.stack([rotation_matrix(t, d, base) @ k[t] for t in range(n)])
    s = qr @ kr.T / math.sqrt(d)
    if causal:
        s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
    return softmax(s, axis=1) @ v


@pytest.mark.parametrize("causal", [False, True])
def test_one_dim_is_textbook_rope_attention(causal):
    rng = np.random.default_rng(21)
    q, k, v = (rng.standard_normal((1, 2, 19, 8)) for _ in range(3))
    out = oracle.forward(q, k, v, [19], causal, rope_base=BASE)
    for h in range(2):
        ref = rope_attention_one_dim(q[0, h], k[0, h], v[0, h], causal, BASE)
        np.testing.assert_allclose(out[0, h], ref, rtol=0, atol=1e-12)
    assert np.abs(out - oracle.forward(q, k, v, [19], causal)).max() > 1e-2   # it does something


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dims", [[3, 4, 2], [5, 3], [2, 2, 2, 3], [6, 1, 4]])
def test_rotating_route_matches_relative_phase_dense_route(dims, causal):
    rng = np.random.default_rng(22)
    N = math.prod(dims)
    q = rng.standard_normal((1, 4, N, 6))
    k, v = rng.standard_normal((1, 2, N, 6)), rng.standard_normal((1, 2, N, 6))
    a = oracle.forward(q, k, v, dims, causal, rope_base=500.0)
    b = oracle.forward_dense(q, k, v, dims, causal, rope_base=500.0)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_closed_form_scores_fix_pairing_sign_and_frequencies():
    """Unit-vector inputs make the hop matrix a closed form of the relative position:
    q = e_0, k = e_{D/2}  ->  score = sin((t-u) theta_0) * scale   (zero for interleaved pairing)
    q = e_{D/2+c}, k = e_c ->  score = -sin((t-u) theta_c) * scale
    q = k = e_1           ->  score = cos((t-u) theta_1) * scale,  theta_1 = base^(-2/D)."""
    from scipy.special import softmax
    n, D, scale = 8, 8, 0.8                        # n == D so that V = I returns the weights
    v = np.eye(n)[None, None, :, :]                # out = the attention matrix itself
    t = np.arange(n)
    rel = t[:, None] - t[None, :]
    for qi, ki, fn, theta in ((0, 4, np.sin, 1.0), (1, 1, np.cos, BASE ** (-2.0 / D)),
                              (4, 0, lambda x: -np.sin(x), 1.0), (7, 3, lambda x: -np.sin(x), BASE ** (-6.0 / D))):
        q = np.zeros((1, 1, n, D)); q[..., qi] = 1.0
        k = np.zeros((1, 1, n, D)); k[..., ki] = 1.0
        out = oracle.forward(q, k, v, [n], False, scale=scale, rope_base=BASE)
        np.testing.assert_allclose(out[0, 0], softmax(fn(rel * theta) * scale, axis=1), atol=1e-13)


def test_position_is_the_coordinate_along_the_hop_dimension():
    """With dims = [a, b] the last hop must see positions j mod b (not the flat index): a head
    whose first hop is switched off (a single visible key under the causal mask at t = 0 ...)
    is awkward, so use dims [1, n] vs [n] and [n, 1] vs [n]: unit dimensions change nothing,
    and [2, n] non-causal equals two independent length-n problems on positions 0..n-1."""
    rng = np.random.default_rng(23)
    n, D = 6, 4
    q, k, v = (rng.standard_normal((1, 1, 2 * n, D)) for _ in range(3))
    full = oracle.forward(q, k, v, [2, n], False, rope_base=BASE, return_xs=True)[1][0]
    # undo nothing: take X after hop 0 as the value input of the per-row problems
    x1 = full[1]
    for row in range(2):
        sl = slice(row * n, (row + 1) * n)
        ref = rope_attention_one_dim(q[0, 0, sl], k[0, 0, sl], x1[sl], False, BASE)
        np.testing.assert_allclose(full[2][sl], ref, atol=1e-12)
    a = oracle.forward(q, k, v, [2 * n], True, rope_base=BASE)
    np.testing.assert_allclose(oracle.forward(q, k, v, [1, 2 * n, 1], True, rope_base=BASE), a, atol=1e-13)


def test_rope_keeps_invariants():
    rng = np.random.default_rng(24)
    dims = [3, 4, 2]
    N = 24
    q, k = rng.standard_normal((1, 2, N, 8)), rng.standard_normal((1, 2, N, 8))
    v = np.broadcast_to(rng.standard_normal((1, 2, 1, 8)), (1, 2, N, 8)).copy()
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, True, rope_base=BASE), v, atol=1e-13)
    # q = 0: scores vanish with or without rotation
    v = rng.standard_normal((1, 2, N, 8))
    np.testing.assert_allclose(oracle.forward(0 * q, k, v, dims, True, rope_base=BASE),
                               oracle.forward(0 * q, k, v, dims, True), atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_with_rope_finite_differences(causal):
    rng = np.random.default_rng(25)
    dims, D, H, Hkv = [3, 2, 4], 4, 2, 1
    N = math.prod(dims)
    q = rng.standard_normal((1, H, N, D))
    k, v = rng.standard_normal((1, Hkv, N, D)), rng.standard_normal((1, Hkv, N, D))
    dout = rng.standard_normal((1, H, N, D))
    dq, dk, dv = oracle.backward(dout, q, k, v, dims, causal, rope_base=100.0)

    def loss(q_, k_, v_):
        return float((oracle.forward(q_, k_, v_, dims, causal, rope_base=100.0) * dout).sum())

    eps = 1e-6
    for name, arr, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(10):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss(q, k, v)
            arr[idx] = old - eps
            lm = loss(q, k, v)
            arr[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[idx]) < 2e-7 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])
