"""Tensorized-attention oracle: Python face of the fp64 C implementation of Algorithm 1,
plus a brute-force dense (N x N) construction used to pin it.

TEST INFRASTRUCTURE ONLY -- never imported by the CUDA package.

Two independent routes to the same result live here:

* ``forward`` / ``backward`` call ``ta_oracle.c`` (Algorithm 1, hop by hop, one head at a
  time in fp64; backward = chain rule through that recurrence).
* ``dense_hop_matrix`` / ``forward_dense`` write every hop as one N x N row-stochastic
  matrix over all tokens (Eq. 3 unfolded: token j attends token k in hop i only if all their
  tensor coordinates except the i-th agree) and multiply them out with numpy.  It is only
  usable for tiny N and exists so that the C code is checked against something that does not
  share its indexing.

Parity pins (tests/test_oracle_pins.py): ndims=1 equals textbook attention (Eq. 1); size-1
dimensions are no-ops; C route == dense route; separable (Kronecker) inputs give
(U_1 (x) ... (x) U_m) V and, non-causal, ordinary full attention; constant V is a fixed point;
Q=0 gives (prefix-)box means; causality probe; the row-major reshape pin of Section 4.4
(one step on the first dimension of {32,32,32} is 1024 tokens); GQA equals explicit KV
repetition; backward equals central finite differences and dV = A_eff^T dout.

Tensorized positional encoding (``rope_base``): in hop i queries and keys are rotated (RoPE,
Llama pairing c <-> c + D/2) by the token's coordinate along dimension i.  The C route
rotates the vectors; the dense route never rotates anything -- it writes the score in the
relative form Re sum_c zq_c conj(zk_c) exp(i (p_j - p_k) theta_c) with complex features
z_c = x_c + i x_{c+D/2} -- so the two share neither code nor formula.  Extra pins: a third,
matrix-form implementation for one dimension; closed-form scores sin / cos of the relative
position for unit-vector inputs (fixes pairing, sign and the frequency ladder).
"""
from __future__ import annotations

import ctypes
import math
import os

import numpy as np

from . import build as _build

_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        path = _build.build()
        lib = ctypes.CDLL(path)
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        lib.ta_oracle_forward_head.restype = ctypes.c_int
        lib.ta_oracle_forward_head.argtypes = [dp, dp, dp, dp, ctypes.c_long, ctypes.c_int, ip,
                                               ctypes.c_int, ctypes.c_int, ctypes.c_double, dp]
        lib.ta_oracle_backward_head.restype = ctypes.c_int
        lib.ta_oracle_backward_head.argtypes = [dp, dp, dp, dp, dp, dp, dp, ctypes.c_long,
                                                ctypes.c_int, ip, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_double]
        lib.ta_oracle_forward_head_rope.restype = ctypes.c_int
        lib.ta_oracle_forward_head_rope.argtypes = [dp, dp, dp, dp, ctypes.c_long, ctypes.c_int, ip,
                                                    ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                                    ctypes.c_double, dp]
        lib.ta_oracle_backward_head_rope.restype = ctypes.c_int
        lib.ta_oracle_backward_head_rope.argtypes = [dp, dp, dp, dp, dp, dp, dp, ctypes.c_long,
                                                     ctypes.c_int, ip, ctypes.c_int, ctypes.c_int,
                                                     ctypes.c_double, ctypes.c_double]
        lib.ta_oracle_forward_head_ex.restype = ctypes.c_int
        lib.ta_oracle_forward_head_ex.argtypes = [dp, dp, dp, dp, ctypes.c_long, ctypes.c_int, ip,
                                                  ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                                  ctypes.c_double, ip, ctypes.POINTER(ctypes.c_void_p), dp]
        lib.ta_oracle_backward_head_ex.restype = ctypes.c_int
        lib.ta_oracle_backward_head_ex.argtypes = [dp, dp, dp, dp, dp, dp, dp, ctypes.c_long,
                                                   ctypes.c_int, ip, ctypes.c_int, ctypes.c_int,
                                                   ctypes.c_double, ctypes.c_double, ip,
                                                   ctypes.POINTER(ctypes.c_void_p)]
        lib.ta_oracle_forward_head_len.restype = ctypes.c_int
        lib.ta_oracle_forward_head_len.argtypes = [dp, dp, dp, dp, ctypes.c_long, ctypes.c_int, ip,
                                                   ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                                   ctypes.c_double, ip, ctypes.POINTER(ctypes.c_void_p),
                                                   ctypes.c_long, dp]
        lib.ta_oracle_backward_head_len.restype = ctypes.c_int
        lib.ta_oracle_backward_head_len.argtypes = [dp, dp, dp, dp, dp, dp, dp, ctypes.c_long,
                                                    ctypes.c_int, ip, ctypes.c_int, ctypes.c_int,
                                                    ctypes.c_double, ctypes.c_double, ip,
                                                    ctypes.POINTER(ctypes.c_void_p), ctypes.c_long]
        lib.ta_oracle_num_threads.restype = ctypes.c_int
        _LIB = lib
    return _LIB


def num_threads() -> int:
    """Threads the OpenMP loops of the C oracle actually use."""
    return int(_lib().ta_oracle_num_threads())


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _check(q, k, v, dims):
    q = np.asarray(q)
    k = np.asarray(k)
    v = np.asarray(v)
    if q.ndim != 4 or k.ndim != 4 or v.shape != k.shape:
        raise ValueError("q:[B,H,N,D], k,v:[B,H_kv,N,D] expected")
    B, H, N, D = q.shape
    Hkv = k.shape[1]
    if k.shape != (B, Hkv, N, D) or H % Hkv:
        raise ValueError("inconsistent q/k/v shapes")
    dims = [int(x) for x in dims]
    if len(dims) < 1 or any(x < 1 for x in dims) or math.prod(dims) != N:
        raise ValueError("prod(dims) must equal N")
    return B, H, Hkv, N, D, dims


def _cwindow(window, m):
    if window is None:
        return None
    w = [int(x) for x in window]
    if len(w) != m or any(x < 0 for x in w):
        raise ValueError("window: one non-negative int per dimension")
    return (ctypes.c_int * m)(*w)


def _cmasks(masks, dims, head=None, heads=None):
    """Per-dimension masks as a C array of byte-matrix pointers; returns (array or None, keep-alive).
    An entry may be n x n (every head) or H x n x n (one matrix per query head: `head` picks it)."""
    if masks is None:
        return None, None
    if len(masks) != len(dims):
        raise ValueError("masks: one entry (or None) per dimension")
    keep, ptrs = [], []
    for mk, n in zip(masks, dims):
        if mk is None:
            ptrs.append(None)
            continue
        a = np.asarray(mk) != 0
        if a.ndim == 3:
            if heads is not None and a.shape[0] != heads:
                raise ValueError("a per-head mask needs one n x n matrix per query head")
            a = a[0 if head is None else head]
        a = np.ascontiguousarray(a, dtype=np.uint8)
        if a.shape != (n, n):
            raise ValueError("mask of a dimension of extent n must be n x n")
        keep.append(a)
        ptrs.append(a.ctypes.data)
    return (ctypes.c_void_p * len(dims))(*ptrs), keep


def _per_head(masks) -> bool:
    return masks is not None and any(mk is not None and np.asarray(mk).ndim == 3 for mk in masks)


def _clens(seq_lens, B, N):
    if seq_lens is None:
        return None
    lens = [int(x) for x in seq_lens]
    if len(lens) != B or any(x < 0 or x > N for x in lens):
        raise ValueError("seq_lens: one length in [0, N] per batch entry")
    return lens


def _fwd_head(lib, qh, kh, vh, out, N, D, cdims, m, causal, scale, rope_base, xs, cwin=None, cmask=None,
              length=None):
    if length is not None:
        return lib.ta_oracle_forward_head_len(_dptr(qh), _dptr(kh), _dptr(vh), _dptr(out), N, D, cdims, m,
                                              int(bool(causal)), scale, float(rope_base or 0.0), cwin, cmask,
                                              int(length), _dptr(xs) if xs is not None else None)
    if cwin is not None or cmask is not None:
        return lib.ta_oracle_forward_head_ex(_dptr(qh), _dptr(kh), _dptr(vh), _dptr(out), N, D, cdims, m,
                                             int(bool(causal)), scale, float(rope_base or 0.0), cwin, cmask,
                                             _dptr(xs) if xs is not None else None)
    if rope_base:
        return lib.ta_oracle_forward_head_rope(_dptr(qh), _dptr(kh), _dptr(vh), _dptr(out), N, D,
                                               cdims, m, int(bool(causal)), scale,
                                               float(rope_base), _dptr(xs) if xs is not None else None)
    return lib.ta_oracle_forward_head(_dptr(qh), _dptr(kh), _dptr(vh), _dptr(out), N, D, cdims, m,
                                      int(bool(causal)), scale, _dptr(xs) if xs is not None else None)


def forward(q, k, v, dims, causal: bool, scale: float | None = None, heads=None,
            return_xs: bool = False, rope_base: float | None = None, window=None, masks=None,
            seq_lens=None):
    """Algorithm 1 for every (or the listed) head, fp64.

    q: [B,H,N,D]; k, v: [B,H_kv,N,D] (any float dtype; converted head by head to fp64).
    Query head h uses KV head h // (H/H_kv).  scale defaults to 1/sqrt(D) (Eq. 4).
    heads: optional list of (b, h) pairs; then the result is [len(heads), N, D].
    rope_base: None / 0 for no positional encoding, else the RoPE base (Llama: 10000) of the
    tensorized positional encoding (hop i rotates q, k by the coordinate along dimension i).
    window: None, or one int per dimension: w_i > 0 keeps, in hop i, only keys within w_i
    positions of the query along dimension i (|t - u| < w_i); 0 = no window.
    masks: None, or one entry per dimension: None or an n_i x n_i array (row = query position,
    column = key position, non-zero = visible) applied on top of `causal` and `window`; an
    H x n_i x n_i array gives every query head a matrix of its own.
    seq_lens: None, or one valid length per batch entry: tokens with flat index >= seq_lens[b]
    are padding (never visible as keys; their output rows are 0).
    Returns out [B,H,N,D] fp64 (and, with return_xs, the list of per-head [m+1,N,D]
    value tensors X_0=V ... X_m=out keyed like the output).
    """
    B, H, Hkv, N, D, dims = _check(q, k, v, dims)
    g = H // Hkv
    scale = 1.0 / math.sqrt(D) if scale is None else float(scale)
    cdims = (ctypes.c_int * len(dims))(*dims)
    cwin = _cwindow(window, len(dims))
    cmask, _keep = _cmasks(masks, dims, heads=H)
    per_head = _per_head(masks)
    lens = _clens(seq_lens, B, N)
    pairs = [(b, h) for b in range(B) for h in range(H)] if heads is None else list(heads)
    out = np.empty((len(pairs), N, D), dtype=np.float64)
    xs_all = []
    lib = _lib()
    for idx, (b, h) in enumerate(pairs):
        qh, kh, vh = _f64(q[b, h]), _f64(k[b, h // g]), _f64(v[b, h // g])
        xs = np.empty((len(dims) + 1, N, D), dtype=np.float64) if return_xs else None
        if per_head:
            cmask, _keep = _cmasks(masks, dims, head=h, heads=H)
        rc = _fwd_head(lib, qh, kh, vh, out[idx], N, D, cdims, len(dims), causal, scale,
                       rope_base, xs, cwin, cmask, None if lens is None else lens[b])
        if rc != 0:
            raise RuntimeError("ta_oracle_forward_head failed")
        if return_xs:
            xs_all.append(xs)
    if heads is None:
        out = out.reshape(B, H, N, D)
    return (out, xs_all) if return_xs else out


def backward(dout, q, k, v, dims, causal: bool, scale: float | None = None, groups=None,
             rope_base: float | None = None, window=None, masks=None, seq_lens=None):
    """Gradients of sum(out * dout) w.r.t. q, k, v (fp64), GQA groups summed into dk, dv.
    With seq_lens the rows of padding tokens are 0 in all three and their rows of dout are ignored.

    groups: optional list of (b, kv_head) pairs; then only those KV heads and their query
    heads are computed and the result is (dq [len, g, N, D], dk [len, N, D], dv [len, N, D]).
    """
    B, H, Hkv, N, D, dims = _check(q, k, v, dims)
    g = H // Hkv
    scale = 1.0 / math.sqrt(D) if scale is None else float(scale)
    cdims = (ctypes.c_int * len(dims))(*dims)
    cwin = _cwindow(window, len(dims))
    cmask, _keep = _cmasks(masks, dims, heads=H)
    per_head = _per_head(masks)
    lens = _clens(seq_lens, B, N)
    sel = [(b, kv) for b in range(B) for kv in range(Hkv)] if groups is None else list(groups)
    dq = np.zeros((len(sel), g, N, D))
    dk = np.zeros((len(sel), N, D))
    dv = np.zeros((len(sel), N, D))
    lib = _lib()
    for idx, (b, kv) in enumerate(sel):
        kh, vh = _f64(k[b, kv]), _f64(v[b, kv])
        for j in range(g):
            h = kv * g + j
            qh = _f64(q[b, h])
            if per_head:
                cmask, _keep = _cmasks(masks, dims, head=h, heads=H)
            o = np.empty((N, D))
            xs = np.empty((len(dims) + 1, N, D))
            rc = _fwd_head(lib, qh, kh, vh, o, N, D, cdims, len(dims), causal, scale, rope_base, xs, cwin, cmask,
                           None if lens is None else lens[b])
            if rc != 0:
                raise RuntimeError("ta_oracle_forward_head failed")
            dqh, dkh, dvh = np.empty((N, D)), np.empty((N, D)), np.empty((N, D))
            if lens is not None:
                rc = lib.ta_oracle_backward_head_len(_dptr(qh), _dptr(kh), _dptr(xs),
                                                     _dptr(_f64(dout[b, h])), _dptr(dqh), _dptr(dkh),
                                                     _dptr(dvh), N, D, cdims, len(dims),
                                                     int(bool(causal)), scale, float(rope_base or 0.0), cwin,
                                                     cmask, int(lens[b]))
            elif cwin is not None or cmask is not None:
                rc = lib.ta_oracle_backward_head_ex(_dptr(qh), _dptr(kh), _dptr(xs),
                                                    _dptr(_f64(dout[b, h])), _dptr(dqh), _dptr(dkh),
                                                    _dptr(dvh), N, D, cdims, len(dims),
                                                    int(bool(causal)), scale, float(rope_base or 0.0), cwin,
                                                    cmask)
            elif rope_base:
                rc = lib.ta_oracle_backward_head_rope(_dptr(qh), _dptr(kh), _dptr(xs),
                                                      _dptr(_f64(dout[b, h])), _dptr(dqh),
                                                      _dptr(dkh), _dptr(dvh), N, D, cdims,
                                                      len(dims), int(bool(causal)), scale,
                                                      float(rope_base))
            else:
                rc = lib.ta_oracle_backward_head(_dptr(qh), _dptr(kh), _dptr(xs),
                                                 _dptr(_f64(dout[b, h])), _dptr(dqh), _dptr(dkh),
                                                 _dptr(dvh), N, D, cdims, len(dims),
                                                 int(bool(causal)), scale)
            if rc != 0:
                raise RuntimeError("ta_oracle_backward_head failed")
            dq[idx, j] = dqh
            dk[idx] += dkh
            dv[idx] += dvh
    if groups is None:
        return dq.reshape(B, H, N, D), dk.reshape(B, Hkv, N, D), dv.reshape(B, Hkv, N, D)
    return dq, dk, dv


# --------------------------------------------------------------------------------------
# Brute force: every hop as a dense N x N matrix (tiny N only).  Independent of the C code.
# --------------------------------------------------------------------------------------

def dense_hop_matrix(qh, kh, dims, i: int, causal: bool, scale: float | None = None,
                     rope_base: float | None = None, window=None, masks=None, length=None):
    """The N x N matrix of hop i for one head (Eq. 3 written over flat token indices).

    Entry [j, k] is the softmax weight of key token k for query token j; it is non-zero only
    if j and k agree in every tensor coordinate except the i-th (and, causal, k_i <= j_i).
    """
    qh = np.asarray(qh, dtype=np.float64)
    kh = np.asarray(kh, dtype=np.float64)
    N, D = qh.shape
    scale = 1.0 / math.sqrt(D) if scale is None else float(scale)
    coords = np.stack(np.unravel_index(np.arange(N), tuple(dims)), axis=1)   # row-major
    allowed = np.ones((N, N), dtype=bool)
    for l in range(len(dims)):
        cj, ck = coords[:, l][:, None], coords[:, l][None, :]
        if l != i:
            allowed &= cj == ck
        else:
            if causal:
                allowed &= ck <= cj
            if window is not None and window[i] > 0:
                allowed &= np.abs(cj - ck) < window[i]
            if masks is not None and masks[i] is not None:
                allowed &= np.asarray(masks[i])[cj, ck] != 0        # looked up by the two coordinates
    if rope_base:
        # relative form of the rotary score: features c and c + D/2 form one complex number
        half = D // 2
        zq = qh[:, :half] + 1j * qh[:, half:2 * half]
        zk = kh[:, :half] + 1j * kh[:, half:2 * half]
        theta = float(rope_base) ** (-2.0 * np.arange(half) / D)
        rel = (coords[:, i][:, None] - coords[:, i][None, :]).astype(np.float64)   # p_j - p_k
        s = np.zeros((N, N))
        for c in range(half):
            s += np.real(np.outer(zq[:, c], np.conj(zk[:, c])) * np.exp(1j * rel * theta[c]))
        if D % 2:
            s += np.outer(qh[:, -1], kh[:, -1])
        s = s * scale
    else:
        s = (qh @ kh.T) * scale
    if length is not None:
        # padding tokens (flat index >= length): no column, and an all-zero row
        exists = np.arange(N) < int(length)
        allowed &= exists[None, :]
        s = np.where(allowed, s, -np.inf)
        a = np.zeros((N, N))
        live = s[exists]
        e = np.exp(live - live.max(axis=1, keepdims=True))
        a[exists] = e / e.sum(axis=1, keepdims=True)
        return a
    s = np.where(allowed, s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=1, keepdims=True)


def dense_effective_matrix(qh, kh, dims, causal: bool, scale: float | None = None,
                           rope_base: float | None = None, window=None, masks=None, length=None):
    """A_eff = A^_{m-1} ... A^_1 A^_0, the N x N map from V to the output of one head."""
    N = np.asarray(qh).shape[0]
    a = np.eye(N)
    for i in range(len(dims)):
        a = dense_hop_matrix(qh, kh, dims, i, causal, scale, rope_base, window, masks, length) @ a
    return a


def forward_dense(q, k, v, dims, causal: bool, scale: float | None = None,
                  rope_base: float | None = None, window=None, masks=None, seq_lens=None):
    """Brute-force forward for all heads via dense_effective_matrix (tiny N only)."""
    B, H, Hkv, N, D, dims = _check(q, k, v, dims)
    g = H // Hkv
    out = np.empty((B, H, N, D))
    for b in range(B):
        for h in range(H):
            masks_h = masks if masks is None else [mk if mk is None or np.asarray(mk).ndim == 2 else np.asarray(mk)[h]
                                                   for mk in masks]          # a head's own matrix, if per head
            a = dense_effective_matrix(q[b, h], k[b, h // g], dims, causal, scale, rope_base, window, masks_h,
                                       None if seq_lens is None else seq_lens[b])
            out[b, h] = a @ np.asarray(v[b, h // g], dtype=np.float64)
    return out
