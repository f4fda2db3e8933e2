"""Pins for the oracle's valid length (padding): tokens with flat index >= len are never visible
as keys, and a padding query gets an all-zero output row.  This is a segment-dependent mask M_i
(Eq. 3 of the paper lets M_i depend on every coordinate).  Each check compares the C route with
something that does not share its loops: the dense brute-force route (boolean N x N masks over
flat indices), the unpadded operator on truncated inputs, textbook attention, a closed form, and
finite differences for the backward."""
import math

import numpy as np
import pytest

import oracle


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dims,lens", [([3, 4, 2], [17, 24]), ([12], [5, 0]), ([5, 4], [1, 19]), ([2, 3, 3], [10, 9])])
def test_length_route_matches_dense_mask_route(dims, lens, causal):
    N = math.prod(dims)
    q, k, v = rnd((2, 4, N, 6), 51), rnd((2, 2, N, 6), 52), rnd((2, 2, N, 6), 53)
    a = oracle.forward(q, k, v, dims, causal, seq_lens=lens)
    b = oracle.forward_dense(q, k, v, dims, causal, seq_lens=lens)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)
    for bi, L in enumerate(lens):
        assert (a[bi, :, L:] == 0).all()


@pytest.mark.parametrize("causal", [False, True])
def test_whole_outer_slabs_equal_the_operator_on_the_truncated_input(causal):
    """len = r * (n_1 n_2): the padding removes whole slabs of the first dimension, and what is
    left is the unpadded operator with dims [r, n_1, n_2] on the first len tokens."""
    dims, r = [5, 3, 4], 3
    N, L = 60, 36
    q, k, v = rnd((1, 2, N, 4), 54), rnd((1, 1, N, 4), 55), rnd((1, 1, N, 4), 56)
    got = oracle.forward(q, k, v, dims, causal, seq_lens=[L])
    ref = oracle.forward(q[:, :, :L], k[:, :, :L], v[:, :, :L], [r, 3, 4], causal)
    np.testing.assert_allclose(got[:, :, :L], ref, atol=1e-14)
    assert (got[:, :, L:] == 0).all()


def test_one_dimension_is_textbook_attention_over_the_valid_prefix():
    N, L, D = 11, 7, 5
    q, k, v = rnd((1, 1, N, D), 57), rnd((1, 1, N, D), 58), rnd((1, 1, N, D), 59)
    for causal in (False, True):
        got = oracle.forward(q, k, v, [N], causal, seq_lens=[L])[0, 0]
        s = q[0, 0, :L] @ k[0, 0, :L].T / math.sqrt(D)
        if causal:
            s = np.where(np.tril(np.ones((L, L), bool)), s, -np.inf)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(got[:L], p @ v[0, 0, :L], atol=1e-14)
        assert (got[L:] == 0).all()


def test_causal_rows_below_the_length_do_not_depend_on_it():
    """Causal hops only read tokens with a smaller flat index, so a valid row is what the
    unpadded run gives; and the full length is no padding at all."""
    dims = [3, 4, 5]
    q, k, v = rnd((1, 2, 60, 4), 60), rnd((1, 2, 60, 4), 61), rnd((1, 2, 60, 4), 62)
    plain = oracle.forward(q, k, v, dims, True)
    for L in (1, 23, 47):
        got = oracle.forward(q, k, v, dims, True, seq_lens=[L])
        np.testing.assert_allclose(got[:, :, :L], plain[:, :, :L], atol=1e-15)
    for causal in (False, True):
        np.testing.assert_allclose(oracle.forward(q, k, v, dims, causal, seq_lens=[60]),
                                   oracle.forward(q, k, v, dims, causal), atol=0)
    # without the causal flag the padding does change valid rows
    assert np.abs(oracle.forward(q, k, v, dims, False, seq_lens=[23])[:, :, :23]
                  - oracle.forward(q, k, v, dims, False)[:, :, :23]).max() > 1e-3


def test_zero_queries_average_over_the_valid_part_of_each_fibre():
    """q = 0, two dimensions [a, b], len in the middle of row r: hop 0 averages each column over
    the rows that exist in it, hop 1 averages each row over the columns that exist in it."""
    a, b, L = 4, 5, 13                      # rows 0, 1 complete, row 2 has columns 0..2
    v = rnd((1, 1, a * b, 3), 63)
    k = rnd((1, 1, a * b, 3), 64)
    q = np.zeros((1, 1, a * b, 3))
    got = oracle.forward(q, k, v, [a, b], False, seq_lens=[L])[0, 0].reshape(a, b, 3)
    V = v[0, 0].reshape(a, b, 3)
    exists = (np.arange(a * b) < L).reshape(a, b)
    x1 = np.zeros_like(V)
    for c in range(b):
        rows = exists[:, c]
        x1[rows, c] = V[rows, c].mean(axis=0)
    ref = np.zeros_like(V)
    for r in range(a):
        cols = exists[r]
        if cols.any():
            ref[r, cols] = x1[r, cols].mean(axis=0)
    np.testing.assert_allclose(got, ref, atol=1e-14)


def test_padding_inputs_are_never_read():
    dims, L = [3, 4, 2], 15
    q, k, v = rnd((1, 2, 24, 4), 65), rnd((1, 1, 24, 4), 66), rnd((1, 1, 24, 4), 67)
    a = oracle.forward(q, k, v, dims, False, seq_lens=[L])
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, L:], k2[:, :, L:], v2[:, :, L:] = 1e6, -1e6, 1e6
    np.testing.assert_array_equal(a, oracle.forward(q2, k2, v2, dims, False, seq_lens=[L]))


@pytest.mark.parametrize("causal", [False, True])
def test_backward_with_length_matches_finite_differences(causal):
    dims, L = [3, 2, 3], 11
    N, D = 18, 3
    q, k, v = rnd((1, 2, N, D), 68), rnd((1, 1, N, D), 69), rnd((1, 1, N, D), 70)
    dout = rnd((1, 2, N, D), 71)
    dq, dk, dv = oracle.backward(dout, q, k, v, dims, causal, seq_lens=[L])

    def loss(q_, k_, v_):
        return float((oracle.forward(q_, k_, v_, dims, causal, seq_lens=[L]) * dout).sum())

    h = 1e-6
    rng = np.random.default_rng(72)
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            args_p = {"q": q, "k": k, "v": v, name: xp}
            args_m = {"q": q, "k": k, "v": v, name: xm}
            fd = (loss(args_p["q"], args_p["k"], args_p["v"]) - loss(args_m["q"], args_m["k"], args_m["v"])) / (2 * h)
            assert abs(fd - g[idx]) <= 1e-7 * max(1.0, abs(fd)), (name, idx, fd, g[idx])
        assert (g[:, :, L:] == 0).all()
    # the padding rows of dout are ignored, whatever they hold
    d2 = dout.copy()
    d2[:, :, L:] = np.nan
    for a_, b_ in zip((dq, dk, dv), oracle.backward(d2, q, k, v, dims, causal, seq_lens=[L])):
        np.testing.assert_array_equal(a_, b_)


def test_backward_whole_slabs_equal_the_truncated_problem():
    dims, r, L = [4, 3, 2], 2, 12
    q, k, v = rnd((1, 2, 24, 3), 73), rnd((1, 2, 24, 3), 74), rnd((1, 2, 24, 3), 75)
    dout = rnd((1, 2, 24, 3), 76)
    got = oracle.backward(dout, q, k, v, dims, False, seq_lens=[L])
    ref = oracle.backward(dout[:, :, :L], q[:, :, :L], k[:, :, :L], v[:, :, :L], [r, 3, 2], False)
    for g_, r_ in zip(got, ref):
        np.testing.assert_allclose(g_[:, :, :L], r_, atol=1e-14)


def test_bad_lengths_are_rejected():
    q = rnd((2, 1, 6, 2), 77)
    for lens in ([7, 1], [-1, 2], [3]):
        with pytest.raises(ValueError):
            oracle.forward(q, q, q, [2, 3], False, seq_lens=lens)
