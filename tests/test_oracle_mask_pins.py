"""Pins for the oracle's per-hop sliding-window masks (the paper allows any sparsity mask M_i in
Eq. 3; here: in hop i a key is visible iff it lies within w_i positions of the query along
dimension i, and not after it when causal).  Each check compares the C route with something
that does not share its loops: the dense brute-force route (a boolean N x N mask built from
coordinates), closed forms, and special cases that reduce to the unmasked operator."""
import math

import numpy as np
import pytest

import oracle


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dims,window", [([3, 4, 2], [2, 3, 1]), ([12], [5]), ([5, 4], [0, 2]), ([2, 9], [1, 4])])
def test_windowed_route_matches_dense_mask_route(dims, window, causal):
    N = math.prod(dims)
    q, k, v = rnd((1, 4, N, 6), 31), rnd((1, 2, N, 6), 32), rnd((1, 2, N, 6), 33)
    a = oracle.forward(q, k, v, dims, causal, window=window)
    b = oracle.forward_dense(q, k, v, dims, causal, window=window)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_wide_or_zero_window_is_no_window(causal):
    dims = [3, 5, 4]
    q, k, v = rnd((1, 2, 60, 4), 34), rnd((1, 2, 60, 4), 35), rnd((1, 2, 60, 4), 36)
    plain = oracle.forward(q, k, v, dims, causal)
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, causal, window=[0, 0, 0]), plain, atol=0)
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, causal, window=[3, 5, 4]), plain, atol=1e-15)
    assert np.abs(oracle.forward(q, k, v, dims, causal, window=[3, 2, 4]) - plain).max() > 1e-3


def test_window_of_one_makes_the_hop_an_identity():
    dims = [4, 6]
    q, k, v = rnd((1, 2, 24, 4), 37), rnd((1, 2, 24, 4), 38), rnd((1, 2, 24, 4), 39)
    for causal in (False, True):
        a = oracle.forward(q, k, v, dims, causal, window=[1, 0])
        # hop 0 sees only the query's own position: the value tensor passes through unchanged,
        # and what is left is hop 1 alone = independent attentions over the rows of length 6
        ref = np.concatenate([oracle.forward(q[:, :, r * 6:(r + 1) * 6], k[:, :, r * 6:(r + 1) * 6],
                                             v[:, :, r * 6:(r + 1) * 6], [6], causal) for r in range(4)], axis=2)
        np.testing.assert_allclose(a, ref, atol=1e-14)


def test_zero_queries_average_the_window():
    """q = 0: uniform weights over the visible keys -> a moving average (closed form)."""
    n, w = 9, 3
    v = rnd((1, 1, n, 2), 40)
    k = rnd((1, 1, n, 2), 41)
    q = np.zeros((1, 1, n, 2))
    got = oracle.forward(q, k, v, [n], True, window=[w])[0, 0]
    for t in range(n):
        np.testing.assert_allclose(got[t], v[0, 0, max(0, t - w + 1):t + 1].mean(axis=0), atol=1e-14)
    got = oracle.forward(q, k, v, [n], False, window=[w])[0, 0]
    for t in range(n):
        np.testing.assert_allclose(got[t], v[0, 0, max(0, t - w + 1):min(n, t + w)].mean(axis=0), atol=1e-14)


def test_influence_set_is_the_window_box():
    """Perturbing one token changes exactly the tokens within the windows along every dimension."""
    dims, window = [3, 5], [2, 3]
    q, k, v = rnd((1, 1, 15, 4), 42), rnd((1, 1, 15, 4), 43), rnd((1, 1, 15, 4), 44)
    base = oracle.forward(q, k, v, dims, True, window=window)
    src = (1, 1)
    v2 = v.copy()
    v2[0, 0, src[0] * 5 + src[1]] += 1.0
    diff = np.abs(oracle.forward(q, k, v2, dims, True, window=window) - base).max(axis=-1)[0, 0].reshape(3, 5)
    for j0 in range(3):
        for j1 in range(5):
            reach = 0 <= j0 - src[0] < window[0] and 0 <= j1 - src[1] < window[1]
            assert (diff[j0, j1] > 1e-9) == reach, (j0, j1, diff[j0, j1])


@pytest.mark.parametrize("causal", [False, True])
def test_backward_with_window_finite_differences(causal):
    rng = np.random.default_rng(45)
    dims, window, D, H, Hkv = [3, 2, 4], [2, 0, 3], 4, 2, 1
    N = math.prod(dims)
    q = rng.standard_normal((1, H, N, D))
    k, v = rng.standard_normal((1, Hkv, N, D)), rng.standard_normal((1, Hkv, N, D))
    dout = rng.standard_normal((1, H, N, D))
    dq, dk, dv = oracle.backward(dout, q, k, v, dims, causal, window=window, rope_base=50.0)

    def loss(q_, k_, v_):
        return float((oracle.forward(q_, k_, v_, dims, causal, window=window, rope_base=50.0) * dout).sum())

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


# ---------------------------------------------------------------- explicit per-hop masks M_i
def random_mask(n, rng, keep_diag=True):
    m = rng.random((n, n)) < 0.5
    if keep_diag:
        m |= np.eye(n, dtype=bool)          # every row keeps its own position
    return m


@pytest.mark.parametrize("causal", [False, True])
def test_explicit_masks_match_dense_route(causal):
    rng = np.random.default_rng(51)
    dims = [3, 4, 5]
    N = 60
    masks = [random_mask(3, rng), None, random_mask(5, rng)]
    q, k, v = rnd((1, 4, N, 6), 52), rnd((1, 2, N, 6), 53), rnd((1, 2, N, 6), 54)
    a = oracle.forward(q, k, v, dims, causal, masks=masks, window=[0, 3, 0])
    b = oracle.forward_dense(q, k, v, dims, causal, masks=masks, window=[0, 3, 0])
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_mask_expresses_the_causal_flag_and_the_window():
    """Three features that must agree: an explicit lower-triangular mask is the causal flag, and an
    explicit band mask is the window parameter."""
    dims = [4, 6]
    q, k, v = rnd((1, 2, 24, 4), 55), rnd((1, 2, 24, 4), 56), rnd((1, 2, 24, 4), 57)
    tril = [np.tril(np.ones((n, n), dtype=bool)) for n in dims]
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, False, masks=tril),
                               oracle.forward(q, k, v, dims, True), atol=1e-15)
    band = [np.abs(np.subtract.outer(np.arange(n), np.arange(n))) < w for n, w in zip(dims, (2, 3))]
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, True, masks=band),
                               oracle.forward(q, k, v, dims, True, window=[2, 3]), atol=1e-15)
    ones = [np.ones((n, n)) for n in dims]
    np.testing.assert_allclose(oracle.forward(q, k, v, dims, True, masks=ones),
                               oracle.forward(q, k, v, dims, True), atol=0)


def test_zero_queries_average_the_masked_set():
    rng = np.random.default_rng(58)
    n = 7
    m = random_mask(n, rng)
    v = rnd((1, 1, n, 3), 59)
    got = oracle.forward(np.zeros((1, 1, n, 3)), rnd((1, 1, n, 3), 60), v, [n], False, masks=[m])[0, 0]
    for t in range(n):
        np.testing.assert_allclose(got[t], v[0, 0, m[t]].mean(axis=0), atol=1e-14)


def block_sparse_mask(n, bs, rng, density=0.4):
    """A block-sparse layout: visibility decided per bs x bs block, diagonal blocks kept."""
    nb = (n + bs - 1) // bs
    blocks = rng.random((nb, nb)) < density
    blocks |= np.eye(nb, dtype=bool)
    return np.kron(blocks, np.ones((bs, bs), dtype=bool))[:n, :n]


def lambda_mask(n, sinks, local):
    """The "Lambda" shape: the first `sinks` keys are always visible, plus the last `local` ones."""
    t, u = np.arange(n)[:, None], np.arange(n)[None, :]
    return (u < sinks) | ((u <= t) & (u > t - local))


@pytest.mark.parametrize("causal", [False, True])
def test_block_sparse_and_lambda_masks_match_dense_route(causal):
    """Structured masks of the kinds the paper names (block-sparse, global + local): the C route
    against the dense route, which builds its N x N boolean mask from coordinates."""
    rng = np.random.default_rng(70)
    dims = [6, 10]
    N = 60
    masks = [block_sparse_mask(6, 2, rng), lambda_mask(10, 2, 3)]
    q, k, v = rnd((1, 2, N, 5), 71), rnd((1, 1, N, 5), 72), rnd((1, 1, N, 5), 73)
    a = oracle.forward(q, k, v, dims, causal, masks=masks)
    b = oracle.forward_dense(q, k, v, dims, causal, masks=masks)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)
    assert np.abs(a - oracle.forward(q, k, v, dims, causal)).max() > 1e-2


def test_lambda_mask_with_zero_queries_is_a_closed_form():
    """q = 0 under the Lambda mask: row t is the mean of the sink keys and its local band."""
    n, sinks, local = 12, 2, 3
    v = rnd((1, 1, n, 3), 74)
    got = oracle.forward(np.zeros((1, 1, n, 3)), rnd((1, 1, n, 3), 75), v, [n], True,
                         masks=[lambda_mask(n, sinks, local)])[0, 0]
    for t in range(n):
        keys = sorted(set(range(min(sinks, t + 1))) | set(range(max(0, t - local + 1), t + 1)))
        np.testing.assert_allclose(got[t], v[0, 0, keys].mean(axis=0), atol=1e-14)


def test_block_diagonal_mask_splits_the_dimension():
    """A block-diagonal mask over one dimension = independent attentions over its blocks."""
    n, bs = 12, 4
    q, k, v = rnd((1, 2, n, 4), 76), rnd((1, 2, n, 4), 77), rnd((1, 2, n, 4), 78)
    m = np.kron(np.eye(n // bs, dtype=bool), np.ones((bs, bs), dtype=bool))
    got = oracle.forward(q, k, v, [n], False, masks=[m])
    ref = np.concatenate([oracle.forward(q[:, :, i:i + bs], k[:, :, i:i + bs], v[:, :, i:i + bs], [bs], False)
                          for i in range(0, n, bs)], axis=2)
    np.testing.assert_allclose(got, ref, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_per_head_masks(causal):
    """An H x n x n entry gives every query head its own matrix: the C route against the dense
    route, against one-head runs with that head's matrix, and -- all heads alike -- against the
    shared-matrix form; gradients of a GQA group sum heads that saw different masks."""
    rng = np.random.default_rng(80)
    dims, H, Hkv = [4, 6], 4, 2
    N = 24
    m0 = np.stack([random_mask(4, rng) for _ in range(H)])
    m1 = np.stack([random_mask(6, rng) for _ in range(H)])
    q, k, v = rnd((1, H, N, 5), 81), rnd((1, Hkv, N, 5), 82), rnd((1, Hkv, N, 5), 83)
    a = oracle.forward(q, k, v, dims, causal, masks=[m0, m1])
    np.testing.assert_allclose(a, oracle.forward_dense(q, k, v, dims, causal, masks=[m0, m1]), rtol=0, atol=1e-13)
    for h in range(H):
        one = oracle.forward(q[:, h:h + 1], k[:, h // 2:h // 2 + 1], v[:, h // 2:h // 2 + 1], dims, causal,
                             masks=[m0[h], m1[h]])
        np.testing.assert_allclose(a[:, h], one[:, 0], atol=1e-15)
    same = oracle.forward(q, k, v, dims, causal, masks=[np.stack([m0[1]] * H), None])
    np.testing.assert_allclose(same, oracle.forward(q, k, v, dims, causal, masks=[m0[1], None]), atol=0)
    assert np.abs(a[:, 0] - oracle.forward(q, k, v, dims, causal, masks=[m0[1], m1[1]])[:, 0]).max() > 1e-3
    # backward: a group's dk, dv are the sums of one-head gradients taken with each head's own masks
    dout = rnd((1, H, N, 5), 84)
    dq, dk, dv = oracle.backward(dout, q, k, v, dims, causal, masks=[m0, m1])
    for kv in range(Hkv):
        sk, sv = 0.0, 0.0
        for h in (2 * kv, 2 * kv + 1):
            gq, gk, gv = oracle.backward(dout[:, h:h + 1], q[:, h:h + 1], k[:, kv:kv + 1], v[:, kv:kv + 1], dims, causal,
                                         masks=[m0[h], m1[h]])
            np.testing.assert_allclose(dq[:, h], gq[:, 0], atol=1e-14)
            sk, sv = sk + gk[:, 0], sv + gv[:, 0]
        np.testing.assert_allclose(dk[:, kv], sk, atol=1e-13)
        np.testing.assert_allclose(dv[:, kv], sv, atol=1e-13)


def test_mask_with_an_empty_row_is_rejected():
    m = np.ones((4, 4), dtype=bool)
    m[2] = False
    q = rnd((1, 1, 4, 2), 61)
    with pytest.raises(RuntimeError):
        oracle.forward(q, q, q, [4], False, masks=[m])


def test_backward_with_explicit_mask_finite_differences():
    rng = np.random.default_rng(62)
    dims, D = [3, 4], 4
    masks = [random_mask(3, rng), random_mask(4, rng)]
    q, k, v = rng.standard_normal((1, 2, 12, D)), rng.standard_normal((1, 1, 12, D)), rng.standard_normal((1, 1, 12, D))
    dout = rng.standard_normal((1, 2, 12, D))
    dq, dk, dv = oracle.backward(dout, q, k, v, dims, False, masks=masks)

    def loss(q_, k_, v_):
        return float((oracle.forward(q_, k_, v_, dims, False, masks=masks) * dout).sum())

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
