"""GPU parity of explicit per-hop masks M_i (Eq. 3 of the paper allows any sparsity mask in a
hop; here hop i takes an n_i x n_i matrix of visible (query position, key position) pairs, the
same for every segment, batch and head) against the fp64 oracle: forward on the tensor-core and
generic kernels, with the causal flag, a window and the positional encoding on top, the backward,
and the argument checks.  Tolerances as for the unmasked operator."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward
from test_gpu_backward import assert_grad_close, gpu_backward

pytestmark = pytest.mark.gpu


def random_masks(dims, seed, density=0.5, skip=()):
    """One random 0/1 matrix per dimension with the diagonal set (so that no row is empty, with or
    without the causal flag); dimensions listed in `skip` get no mask."""
    rng = np.random.default_rng(seed)
    out = []
    for i, n in enumerate(dims):
        if i in skip:
            out.append(None)
            continue
        m = (rng.random((n, n)) < density).astype(np.uint8)
        m[np.arange(n), np.arange(n)] = 1
        out.append(m)
    return out


def run(B, H, Hkv, D, dims, masks, causal, dtype, seed, flags=0, expect=None, **kw):
    N = math.prod(dims)
    if expect is not None:
        # masked calls are planned without hop fusion
        assert expect in ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal,
                                             ta.TA_DTYPE_BF16 if dtype == "bf16" else ta.TA_DTYPE_F32,
                                             flags | ta.TA_FLAG_NO_HOP_FUSION)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, dtype, seed)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, dtype, flags, hop_masks=masks, **kw)
    okw = {"window": kw.get("window"), "rope_base": kw.get("rope_base") or None}
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, masks=masks, **okw)
    assert_close(got, ref, dtype)
    plain = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, **okw)
    assert np.abs(ref - plain).max() > 0.05          # the masks change the result visibly
    return got


@pytest.mark.parametrize("dims,D,causal,skip", [
    ([4, 64], 128, True, ()),
    ([64, 64], 128, False, (0,)),
    ([32, 8, 32], 128, True, (1,)),
    ([5, 24, 7], 64, False, ()),           # several segments per tile, ragged tiles
    ([128], 128, False, ()),
    ([3, 100], 64, True, ()),
    ([8, 8, 8], 64, False, ()),            # would be fused without masks
])
def test_masks_tensor_core_kernel(dims, D, causal, skip):
    run(2, 4, 2, D, dims, random_masks(dims, 11, skip=skip), causal, "bf16", 701, expect="tc")


def test_masks_with_window_and_positional_encoding():
    dims = [8, 64]
    run(1, 4, 2, 128, dims, random_masks(dims, 12), True, "bf16", 702, window=[3, 20])
    run(1, 4, 2, 128, dims, random_masks(dims, 13), True, "bf16", 703, rope_base=10000.0)
    run(1, 4, 2, 64, dims, random_masks(dims, 14), False, "bf16", 704, rope_base=10000.0, window=[0, 40])


def test_masks_generic_kernel():
    run(2, 4, 2, 40, [3, 5, 7], random_masks([3, 5, 7], 15), True, "f32", 705)
    run(1, 4, 2, 64, [6, 100], random_masks([6, 100], 16), False, "f32", 706)
    run(1, 2, 1, 64, [16, 16], random_masks([16, 16], 17), True, "bf16", 707, flags=ta.TA_FLAG_NO_TENSOR_CORE)


def test_triangular_and_band_masks_reproduce_the_flag_and_the_window():
    """A lower-triangular matrix is the causal flag, a band matrix is the window: the masked
    kernels must then give what the unmasked ones give (same products, same sums)."""
    B, H, Hkv, D, dims = 1, 4, 2, 128, [16, 64]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 708)
    tri = [np.tril(np.ones((n, n), np.uint8)) for n in dims]
    a = gpu_forward(inp, B, H, Hkv, N, D, dims, False, "bf16", ta.TA_FLAG_NO_HOP_FUSION, hop_masks=tri)
    b = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", ta.TA_FLAG_NO_HOP_FUSION)
    np.testing.assert_array_equal(a, b)
    w = [5, 9]
    band = [(np.abs(np.subtract.outer(np.arange(n), np.arange(n))) < wi).astype(np.uint8) for n, wi in zip(dims, w)]
    a = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", ta.TA_FLAG_NO_HOP_FUSION, hop_masks=band)
    b = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", ta.TA_FLAG_NO_HOP_FUSION, window=w)
    np.testing.assert_array_equal(a, b)


def test_mask_argument_checks():
    import torch
    x = torch.zeros(1, 2, 64, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(x)
    empty_row = np.ones((8, 8), np.uint8)
    empty_row[3, :] = 0
    rc = ta.ta_forward_ex(x, x, x, out, 1, 2, 2, 64, 64, [8, 8], False, hop_masks=[None, empty_row], check=False)
    assert rc == ta.TA_ERR_INVALID_ARG
    # a row whose only visible keys lie after the query is empty once the causal flag is applied
    upper = np.triu(np.ones((8, 8), np.uint8), 1)
    upper[7, 7] = 1
    rc = ta.ta_forward_ex(x, x, x, out, 1, 2, 2, 64, 64, [8, 8], True, hop_masks=[upper, None], check=False)
    assert rc == ta.TA_ERR_INVALID_ARG
    rc = ta.ta_forward_ex(x, x, x, out, 1, 2, 2, 64, 64, [8, 8], False, hop_masks=[upper, None], check=False)
    assert rc == ta.TA_OK
    # longer dimensions take masks too; an empty row is caught on the host there as well
    y = torch.zeros(1, 2, 256, 64, dtype=torch.bfloat16, device="cuda")
    o = torch.empty((1, 2, 256, 64), dtype=torch.bfloat16, device="cuda")
    rc = ta.ta_forward_ex(y, y, y, o, 1, 2, 2, 256, 64, [256], True,
                          hop_masks=[np.tril(np.ones((256, 256), np.uint8))], check=False)
    assert rc == ta.TA_OK
    bad = np.ones((256, 256), np.uint8)
    bad[200, :] = 0
    rc = ta.ta_forward_ex(y, y, y, o, 1, 2, 2, 256, 64, [256], True, hop_masks=[bad], check=False)
    assert rc == ta.TA_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        ta.ta_forward_ex(x, x, x, out, 1, 2, 2, 64, 64, [8, 8], False, hop_masks=[np.ones((4, 4))])


@pytest.mark.parametrize("dims,D,causal,skip,rope", [
    ([8, 16, 32], 128, True, (1,), 0.0),
    ([16, 16], 64, False, (), 0.0),
    ([128], 128, True, (), 0.0),
    ([5, 24], 64, False, (), 0.0),
    ([8, 64], 128, True, (), 10000.0),
])
def test_backward_with_masks(dims, D, causal, skip, rope):
    B, H, Hkv = 1, 4, 2
    N = math.prod(dims)
    masks = random_masks(dims, 18, skip=skip)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 709, with_dout=True)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, True, hop_masks=masks, rope_base=rope)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, masks=masks,
                          rope_base=rope or None)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, sum(1 for n in dims if n > 1), rope=bool(rope))


def block_sparse_mask(n, bs, rng, density=0.4):
    nb = (n + bs - 1) // bs
    blocks = rng.random((nb, nb)) < density
    blocks |= np.eye(nb, dtype=bool)
    return np.kron(blocks, np.ones((bs, bs), dtype=np.uint8))[:n, :n].astype(np.uint8)


def lambda_mask(n, sinks, local):
    t, u = np.arange(n)[:, None], np.arange(n)[None, :]
    return ((u < sinks) | ((u <= t) & (u > t - local))).astype(np.uint8)


@pytest.mark.parametrize("dims,D,causal,kind", [
    ([200], 64, True, "random"),              # one ragged second key block
    ([200], 128, False, "lambda"),
    ([1024], 128, True, "lambda"),            # sink keys + local band: the middle key blocks are empty
    ([1024], 64, False, "block"),             # block-sparse layout of 64 x 64 blocks
    ([1024], 128, True, "band"),              # banded: leading key blocks of a query block are skipped
    ([3, 200], 128, True, "random"),          # short (kernel-parameter mask) and long (bit matrix) hop
    ([260, 2], 64, False, "block"),           # long hop over a strided dimension
    ([1280], 64, True, "block"),              # pairs of query tiles (n > 1 024)
    ([1100], 64, False, "lambda"),
])
def test_masks_on_long_segments(dims, D, causal, kind):
    """Explicit masks on dimensions longer than 128: bit matrix in device memory, tensor-core forward."""
    B, H, Hkv = 2, 4, 2
    N = math.prod(dims)
    rng = np.random.default_rng(19)
    masks = []
    for n in dims:
        if kind == "random":
            m = (rng.random((n, n)) < 0.5).astype(np.uint8)
            m[np.arange(n), np.arange(n)] = 1
        elif kind == "lambda":
            m = lambda_mask(n, 4, 48)
        elif kind == "block":
            m = block_sparse_mask(n, 64 if n > 128 else 1, rng)
        else:
            t, u = np.arange(n)[:, None], np.arange(n)[None, :]
            m = (np.abs(t - u) < 150).astype(np.uint8)
        masks.append(m)
    assert "tc-long" in ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, 0)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 711)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", hop_masks=masks)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, masks=masks)
    assert_close(got, ref, "bf16")
    assert np.abs(ref - oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)).max() > 0.05
    # the generic kernel reads the same bit matrix
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", ta.TA_FLAG_NO_TENSOR_CORE, hop_masks=masks)
    assert_close(got, ref, "bf16")


@pytest.mark.parametrize("dims,D,causal,kind", [
    ([200], 64, True, "random"),
    ([1024], 128, True, "lambda"),
    ([3, 200], 128, False, "random"),
])
def test_backward_with_masks_on_long_segments(dims, D, causal, kind):
    B, H, Hkv = 1, 4, 2
    N = math.prod(dims)
    rng = np.random.default_rng(20)
    masks = []
    for n in dims:
        if kind == "lambda":
            m = lambda_mask(n, 4, 48)
        else:
            m = (rng.random((n, n)) < 0.5).astype(np.uint8)
            m[np.arange(n), np.arange(n)] = 1
        masks.append(m)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 712, with_dout=True)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, masks=masks)
    for grad_f32 in (True, False):
        got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32, hop_masks=masks)
        for name, g, r in zip(("dq", "dk", "dv"), got, ref):
            assert_grad_close(g, r, name, grad_f32, sum(1 for n in dims if n > 1))


@pytest.mark.parametrize("dims,D,causal,flags", [
    ([8, 16, 32], 128, True, 0),                         # tensor-core hops, four segments per tile
    ([5, 24], 64, False, 0),
    ([3, 200], 128, True, 0),                            # short hop and long hop
    ([6, 20], 40, True, 0),                              # generic kernels (head dim 40)
    ([4, 64], 128, True, ta.TA_FLAG_NO_TENSOR_CORE),
])
def test_masks_that_differ_per_head(dims, D, causal, flags):
    """masks_per_head: every query head has its own n_i x n_i matrix per hop (heads of one GQA group
    see different keys); forward and backward against the oracle, which takes H x n x n arrays."""
    B, H, Hkv = 2, 4, 2
    N = math.prod(dims)
    rng = np.random.default_rng(21)
    masks = []
    for n in dims:
        m = (rng.random((H, n, n)) < 0.5).astype(np.uint8)
        m[:, np.arange(n), np.arange(n)] = 1
        masks.append(m)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 713, with_dout=True)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", flags, hop_masks=masks)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, masks=masks)
    assert_close(got, ref, "bf16")
    shared = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, masks=[m[0] for m in masks])
    assert np.abs(ref[:, 1:] - shared[:, 1:]).max() > 0.05        # the other heads' masks matter
    if flags:
        return
    refs = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, masks=masks)
    for grad_f32 in (True, False):
        grads = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32, hop_masks=masks)
        for name, g, r in zip(("dq", "dk", "dv"), grads, refs):
            assert_grad_close(g, r, name, grad_f32, sum(1 for n in dims if n > 1))


def test_per_head_masks_with_equal_matrices_reproduce_the_shared_mask():
    B, H, Hkv, D, dims = 1, 4, 2, 128, [4, 64]
    N = math.prod(dims)
    masks = random_masks(dims, 22)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 714)
    a = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", hop_masks=masks)
    b = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", hop_masks=[np.stack([m] * H) for m in masks])
    np.testing.assert_array_equal(a, b)
    with pytest.raises(ValueError):       # either every mask is per head or none
        import torch
        x = torch.zeros(1, 4, 256, 64, dtype=torch.bfloat16, device="cuda")
        ta.ta_forward_ex(x, x[:, :2], x[:, :2], torch.empty_like(x), 1, 4, 2, 256, 64, [4, 64], True,
                         hop_masks=[np.ones((4, 4)), np.ones((4, 64, 64))])


def test_masks_llama_shape_sampled_heads():
    """32 768 tokens as 32x32x32, H=32, H_kv=8, D=128, causal, with a random mask on every hop."""
    c = ta_inputs.CONFIGS[3]
    masks = random_masks(list(c.dims), 19)
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_forward(inp, c.B, c.H, c.H_kv, c.N, c.D, list(c.dims), True, "bf16", hop_masks=masks)
    heads = [(0, 5), (0, 30)]
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], list(c.dims), True, masks=masks, heads=heads)
    assert_close(np.stack([got[b, h] for b, h in heads]), ref, "bf16")
