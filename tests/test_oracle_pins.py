"""Pins for the CPU oracle: every check here compares it with something that is NOT the
oracle's own formula -- a textbook routine, a closed form, an invariant, brute force, or a
fact the paper states (tests/golden/paper_facts.txt)."""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")
RNG = np.random.default_rng(1234)


def rand_qkv(B, H, Hkv, N, D, rng=RNG):
    return (rng.standard_normal((B, H, N, D)), rng.standard_normal((B, Hkv, N, D)),
            rng.standard_normal((B, Hkv, N, D)))


def textbook_attention(q, k, v, causal):
    """Eq. 1: softmax(q k^T / sqrt(d)) v for one head, written with scipy's softmax."""
    from scipy.special import softmax
    n, d = q.shape
    s = q @ k.T / math.sqrt(d)
    if causal:
        s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
    return softmax(s, axis=1) @ v


def paper_facts():
    facts = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                facts.append(line.split())
    return facts


# 1. one dimension = ordinary attention (Eq. 1; "Tens-1" in Appendix D)
@pytest.mark.parametrize("causal", [False, True])
def test_one_dim_is_textbook_attention(causal):
    q, k, v = rand_qkv(2, 3, 3, 37, 16)
    out = oracle.forward(q, k, v, [37], causal)
    for b in range(2):
        for h in range(3):
            ref = textbook_attention(q[b, h], k[b, h], v[b, h], causal)
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-13)


# 2. size-1 dimensions are no-op hops
@pytest.mark.parametrize("causal", [False, True])
def test_unit_dims_are_noops(causal):
    q, k, v = rand_qkv(1, 2, 2, 24, 8)
    a = oracle.forward(q, k, v, [3, 8], causal)
    np.testing.assert_allclose(oracle.forward(q, k, v, [3, 1, 8], causal), a, atol=1e-14)
    np.testing.assert_allclose(oracle.forward(q, k, v, [1, 3, 8, 1], causal), a, atol=1e-14)
    full = oracle.forward(q, k, v, [24], causal)
    np.testing.assert_allclose(oracle.forward(q, k, v, [24, 1], causal), full, atol=1e-14)
    np.testing.assert_allclose(oracle.forward(q, k, v, [1, 24], causal), full, atol=1e-14)


# 3. Algorithm 1 == product of dense per-hop N x N matrices (brute force, tiny N)
@pytest.mark.parametrize("dims", [[3, 4, 2], [4, 4], [2, 3, 2, 2], [5, 3], [2, 2, 2, 2, 2]])
@pytest.mark.parametrize("causal", [False, True])
def test_matches_dense_bruteforce(dims, causal):
    N = math.prod(dims)
    q, k, v = rand_qkv(1, 4, 2, N, 8)
    a = oracle.forward(q, k, v, dims, causal)
    b = oracle.forward_dense(q, k, v, dims, causal)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_dense_hop_rows_are_stochastic_and_sparse():
    dims = [3, 4, 2]
    q, k, _ = rand_qkv(1, 1, 1, 24, 8)
    for i, n in enumerate(dims):
        a = oracle.dense_hop_matrix(q[0, 0], k[0, 0], dims, i, False)
        np.testing.assert_allclose(a.sum(1), 1.0, atol=1e-14)
        assert ((a > 0).sum(1) == n).all()


# 4. separable q,k: A_i does not depend on the batch coordinates, the result is the
#    Kronecker product of per-dimension attention matrices, the hop order is irrelevant, and
#    (non-causal) it equals ordinary full attention over all N tokens.
def _separable(dims, dsub, rng):
    m, N = len(dims), math.prod(dims)
    D = m * dsub
    a = [rng.standard_normal((n, dsub)) for n in dims]
    b = [rng.standard_normal((n, dsub)) for n in dims]
    coords = np.stack(np.unravel_index(np.arange(N), tuple(dims)), axis=1)
    q = np.concatenate([a[l][coords[:, l]] for l in range(m)], axis=1)
    k = np.concatenate([b[l][coords[:, l]] for l in range(m)], axis=1)
    return a, b, q, k, D


@pytest.mark.parametrize("causal", [False, True])
def test_kronecker_closed_form(causal):
    from scipy.special import softmax
    rng = np.random.default_rng(7)
    dims, dsub = [3, 4, 2], 4
    a, b, q, k, D = _separable(dims, dsub, rng)
    N = math.prod(dims)
    v = rng.standard_normal((N, 5 + D))[:, :D]
    us = []
    for l, n in enumerate(dims):
        s = a[l] @ b[l].T / math.sqrt(D)
        if causal:
            s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
        us.append(softmax(s, axis=1))
    kron = us[0]
    for u in us[1:]:
        kron = np.kron(kron, u)
    out = oracle.forward(q[None, None], k[None, None], v[None, None], dims, causal)[0, 0]
    np.testing.assert_allclose(out, kron @ v, rtol=0, atol=1e-13)
    if not causal:
        np.testing.assert_allclose(out, textbook_attention(q, k, v, False), atol=1e-13)
    # hop order irrelevant in the separable case: permute the tensor axes and compare
    perm = [2, 0, 1]
    pdims = [dims[p] for p in perm]

    def permute(x):
        return x.reshape(*dims, -1).transpose(*perm, 3).reshape(N, -1)

    outp = oracle.forward(permute(q)[None, None], permute(k)[None, None],
                          permute(v)[None, None], pdims, causal)[0, 0]
    np.testing.assert_allclose(outp, permute(out), rtol=0, atol=1e-13)


def test_hop_order_matters_in_general():
    # the general (non-separable) case depends on the order, so the oracle must run
    # dims[0] first as Algorithm 1 does; a reversed loop would not pass the dense pin.
    q, k, v = rand_qkv(1, 1, 1, 24, 8)
    dims = [3, 4, 2]
    a0 = oracle.dense_hop_matrix(q[0, 0], k[0, 0], dims, 0, False)
    a1 = oracle.dense_hop_matrix(q[0, 0], k[0, 0], dims, 1, False)
    a2 = oracle.dense_hop_matrix(q[0, 0], k[0, 0], dims, 2, False)
    fwd = a2 @ a1 @ a0 @ v[0, 0]
    rev = a0 @ a1 @ a2 @ v[0, 0]
    assert np.abs(fwd - rev).max() > 1e-3
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, False)[0, 0], fwd, atol=1e-13)


# 5. row-stochastic invariants
@pytest.mark.parametrize("causal", [False, True])
def test_constant_v_is_fixed_point_and_range(causal):
    q, k, v = rand_qkv(1, 2, 1, 36, 8)
    vc = np.broadcast_to(np.arange(8.0), v.shape).copy()
    np.testing.assert_allclose(oracle.forward(q, k, vc, [3, 3, 4], causal),
                               np.broadcast_to(np.arange(8.0), q.shape), atol=1e-13)
    out = oracle.forward(q, k, v, [3, 3, 4], causal)
    assert (out <= v.max(axis=2, keepdims=True).repeat(2, 1) + 1e-12).all()
    assert (out >= v.min(axis=2, keepdims=True).repeat(2, 1) - 1e-12).all()


# 6. Q = 0: uniform weights -> (prefix-)box means of V
@pytest.mark.parametrize("causal", [False, True])
def test_zero_q_gives_box_means(causal):
    dims = [3, 4, 2]
    N = 24
    _, k, v = rand_qkv(1, 1, 1, N, 8)
    q = np.zeros((1, 1, N, 8))
    out = oracle.forward(q, k, v, dims, causal)[0, 0]
    vt = v[0, 0].reshape(*dims, 8)
    if not causal:
        np.testing.assert_allclose(out, np.broadcast_to(vt.mean((0, 1, 2)), (N, 8)), atol=1e-13)
    else:
        ref = np.empty_like(vt)
        for j0 in range(3):
            for j1 in range(4):
                for j2 in range(2):
                    ref[j0, j1, j2] = vt[:j0 + 1, :j1 + 1, :j2 + 1].mean((0, 1, 2))
        np.testing.assert_allclose(out, ref.reshape(N, 8), atol=1e-13)


# 7. causality probe: token k influences exactly the rows j with j_l >= k_l for every l
def test_causal_influence_set():
    dims = [3, 4, 2]
    N = 24
    q, k, v = rand_qkv(1, 1, 1, N, 8)
    base = oracle.forward(q, k, v, dims, True)[0, 0]
    tok = np.ravel_multi_index((1, 2, 0), dims)
    for which in range(3):
        q2, k2, v2 = q.copy(), k.copy(), v.copy()
        [q2, k2, v2][which][0, 0, tok] += 1.0
        pert = oracle.forward(q2, k2, v2, dims, True)[0, 0]
        changed = set(np.nonzero(np.abs(pert - base).max(1) > 0)[0].tolist())
        coords = np.stack(np.unravel_index(np.arange(N), dims), 1)
        reach = set(np.nonzero((coords >= np.array([1, 2, 0])).all(1))[0].tolist())
        assert changed <= reach
        if which == 2:          # V enters linearly with strictly positive weights
            assert changed == reach


# 8. row-major reshape as the paper states it, and the shapes the paper uses
def test_reshape_pin_from_paper():
    facts = paper_facts()
    step = [f for f in facts if f[0] == "first_dim_step"][0]
    dims = [int(x) for x in step[1].split("=")[1].split(",")]
    tokens = int(step[2].split("=")[1])
    # shrink the feature width, keep the paper's tensor shape: perturb V at one token and
    # look where hop 0 alone (the other two hops disabled by Q=0... not needed) spreads it.
    N, D = math.prod(dims), 2
    rng = np.random.default_rng(5)
    q = rng.standard_normal((1, 1, N, D))
    k = rng.standard_normal((1, 1, N, D))
    v = np.zeros((1, 1, N, D))
    c = 777                                 # a token with first coordinate 0
    v[0, 0, c] = 1.0
    xs = oracle.forward(q, k, v, dims, False, return_xs=True)[1][0]
    hit = np.nonzero(np.abs(xs[1]).max(1) > 0)[0]          # support after hop 0 only
    assert hit.tolist() == [c + tokens * t for t in range(dims[0])]
    hit2 = np.nonzero(np.abs(xs[2]).max(1) > 0)[0]         # after hop 1: stride n_3
    assert set(hit2.tolist()) == {(c % dims[2]) + dims[2] * u + tokens * t
                                  for t in range(dims[0]) for u in range(dims[1])}
    for f in facts:
        if f[0] == "shape":
            assert math.prod(int(x) for x in f[2].split(",")) == int(f[1])


def test_paper_shapes_run_and_match_dense_where_small():
    # 12 x 12 attention <-> order-3 tensor example of Appendix C
    q, k, v = rand_qkv(1, 1, 1, 12, 4)
    np.testing.assert_allclose(oracle.forward(q, k, v, [2, 3, 2], True),
                               oracle.forward_dense(q, k, v, [2, 3, 2], True), atol=1e-13)


# 9. GQA == explicit repetition of KV heads
@pytest.mark.parametrize("causal", [False, True])
def test_gqa_equals_repeated_kv(causal):
    q, k, v = rand_qkv(2, 6, 2, 24, 8)
    a = oracle.forward(q, k, v, [4, 6], causal)
    b = oracle.forward(q, np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1), [4, 6], causal)
    np.testing.assert_allclose(a, b, rtol=0, atol=0)
    # and the grouping is contiguous: head 1 uses KV head 0, head 3 uses KV head 1
    ref = textbook_attention(q[0, 3], k[0, 1], v[0, 1], causal)
    np.testing.assert_allclose(oracle.forward(q, k, v, [24], causal)[0, 3], ref, atol=1e-13)


# scale: default is 1/sqrt(D) in every hop (Eq. 4); an explicit scale is honoured
def test_scale_argument():
    q, k, v = rand_qkv(1, 1, 1, 12, 4)
    a = oracle.forward(q, k, v, [3, 4], False)
    b = oracle.forward(q * 2.0, k, v, [3, 4], False, scale=0.25)
    np.testing.assert_allclose(a, b, atol=1e-13)


# 10. backward: finite differences, and dV = A_eff^T dout
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dims", [[3, 4, 2], [12], [4, 3]])
def test_backward_finite_differences(dims, causal):
    rng = np.random.default_rng(11)
    N, D, H, Hkv = math.prod(dims), 4, 4, 2
    q, k, v = rand_qkv(1, H, Hkv, N, D, rng)
    dout = rng.standard_normal((1, H, N, D))
    dq, dk, dv = oracle.backward(dout, q, k, v, dims, causal)

    def loss(q_, k_, v_):
        return float((oracle.forward(q_, k_, v_, dims, causal) * dout).sum())

    eps = 1e-6
    for name, arr, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        idxs = [tuple(rng.integers(0, s) for s in arr.shape) for _ in range(12)]
        for idx in idxs:
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss(q, k, v)
            arr[idx] = old - eps
            lm = loss(q, k, v)
            arr[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[idx]) < 2e-7 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


@pytest.mark.parametrize("causal", [False, True])
def test_backward_dv_is_transposed_effective_matrix(causal):
    rng = np.random.default_rng(12)
    dims, D, H, Hkv = [3, 2, 4], 4, 4, 2
    N = math.prod(dims)
    q, k, v = rand_qkv(1, H, Hkv, N, D, rng)
    dout = rng.standard_normal((1, H, N, D))
    _, _, dv = oracle.backward(dout, q, k, v, dims, causal)
    ref = np.zeros_like(dv)
    for h in range(H):
        a = oracle.dense_effective_matrix(q[0, h], k[0, h // 2], dims, causal)
        ref[0, h // 2] += a.T @ dout[0, h]
    np.testing.assert_allclose(dv, ref, rtol=0, atol=1e-13)


def test_bad_shapes_rejected():
    q, k, v = rand_qkv(1, 2, 2, 12, 4)
    with pytest.raises(ValueError):
        oracle.forward(q, k, v, [3, 5], False)
    with pytest.raises(ValueError):
        oracle.forward(q, k[:, :1].repeat(3, 1), v[:, :1].repeat(3, 1), [12], False)
