"""GPU parity of valid lengths (padding to prod(dims), batches of different lengths: tokens with
flat index >= seq_lens[b] are never keys and their output / gradient rows are 0) against the fp64
oracle: forward on the short-segment tensor-core kernel and on the generic kernel (which also
takes the segments longer than 128), with masks, windows and the positional encoding on top, and
the backward.  Tolerances as for the unmasked operator."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward
from test_gpu_backward import assert_grad_close, gpu_backward

pytestmark = pytest.mark.gpu


def dev_lens(lens):
    import torch
    return torch.tensor(lens, dtype=torch.int32, device="cuda")


def poison_padding(inp, lens, names=("q", "k", "v")):
    """Large finite values in the padding rows: they must not reach any valid output."""
    for name in names:
        x = inp[name]
        for b, L in enumerate(lens):
            x[b, :, L:] = 240.0 if name != "k" else -240.0
        if name + "_bits" in inp:
            inp[name + "_bits"] = ta_inputs.bf16_bits(x)
    return inp


def run(B, H, Hkv, D, dims, lens, causal, dtype, seed, flags=0, expect=None, **kw):
    N = math.prod(dims)
    inp = poison_padding(ta_inputs.make_inputs(B, H, Hkv, N, D, dtype, seed), lens)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, dtype, flags, seq_lens=dev_lens(lens), **kw)
    okw = {"window": kw.get("window"), "rope_base": kw.get("rope_base") or None, "masks": kw.get("hop_masks")}
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, seq_lens=lens, **okw)
    assert_close(got, ref, dtype)
    for b, L in enumerate(lens):
        assert (got[b, :, L:] == 0).all()
    return got


@pytest.mark.parametrize("dims,D,causal,lens", [
    ([4, 64], 128, False, [200, 256]),
    ([64, 64], 128, True, [4095, 1]),
    ([32, 8, 32], 128, False, [5000, 8192]),
    ([5, 24, 7], 64, False, [839, 400]),         # several segments per tile, ragged tiles
    ([128], 128, False, [77, 0]),                # an empty batch entry
    ([3, 100], 64, True, [150, 299]),
    ([8, 8, 8], 64, False, [100, 511]),          # would be fused without lengths
])
def test_lengths_tensor_core_kernel(dims, D, causal, lens):
    run(2, 4, 2, D, dims, lens, causal, "bf16", 801)


def test_lengths_with_masks_windows_and_positional_encoding():
    dims = [8, 64]
    rng = np.random.default_rng(5)
    masks = []
    for n in dims:
        m = (rng.random((n, n)) < 0.5).astype(np.uint8)
        m[np.arange(n), np.arange(n)] = 1
        masks.append(m)
    run(2, 4, 2, 128, dims, [300, 511], False, "bf16", 802, hop_masks=masks)
    run(2, 4, 2, 128, dims, [300, 511], True, "bf16", 803, window=[3, 20])
    run(2, 4, 2, 128, dims, [129, 512], False, "bf16", 804, rope_base=10000.0)
    run(2, 4, 2, 64, dims, [129, 40], True, "bf16", 805, rope_base=10000.0, hop_masks=masks, window=[0, 50])


def test_lengths_generic_kernel_and_long_segments():
    run(2, 4, 2, 40, [3, 5, 7], [100, 13], False, "f32", 806)
    run(2, 4, 2, 64, [6, 100], [599, 250], True, "f32", 807)
    run(1, 2, 1, 64, [16, 16], [77], False, "bf16", 808, flags=ta.TA_FLAG_NO_TENSOR_CORE)


@pytest.mark.parametrize("dims,D,causal,lens", [
    ([2, 300], 64, False, [450, 299]),            # second row of the tensor cut short / missing
    ([700], 128, True, [257, 700]),               # ordinary attention, batch entries of different lengths
    ([700], 64, False, [1, 0]),                   # one token; an empty batch entry
    ([3, 260], 128, False, [400, 780]),
    ([1024], 128, True, [1000, 130]),
    ([1400], 64, True, [1399, 200]),              # pairs of query tiles (n > 1 024)
    ([1150], 128, False, [640, 1150]),
])
def test_lengths_long_segments_tensor_core(dims, D, causal, lens):
    B, H, Hkv = 2, 4, 2
    assert "tc-long" in ta.ta_plan_describe(B, H, Hkv, math.prod(dims), D, dims, causal, ta.TA_DTYPE_BF16, 0)
    run(B, H, Hkv, D, dims, lens, causal, "bf16", 809)


def test_lengths_long_segments_with_window_and_generic_kernel():
    run(2, 4, 2, 64, [600], [599, 123], True, "bf16", 813, window=[100])
    run(1, 2, 1, 64, [2, 300], [450], False, "bf16", 814, flags=ta.TA_FLAG_NO_TENSOR_CORE)


def test_full_length_is_no_padding_and_causal_rows_do_not_depend_on_the_length():
    B, H, Hkv, D, dims = 1, 4, 2, 128, [16, 64]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 810)
    plain = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", ta.TA_FLAG_NO_HOP_FUSION)
    full = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", seq_lens=dev_lens([N]))
    np.testing.assert_array_equal(full, plain)
    part = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", seq_lens=dev_lens([700]))
    np.testing.assert_array_equal(part[:, :, :700], plain[:, :, :700])
    assert (part[:, :, 700:] == 0).all()


def test_all_unit_dims_with_lengths():
    import torch
    B, H, Hkv, D = 3, 4, 2, 64
    inp = ta_inputs.make_inputs(B, H, Hkv, 1, D, "bf16", 811)
    got = gpu_forward(inp, B, H, Hkv, 1, D, [1, 1], False, "bf16", seq_lens=dev_lens([1, 0, 1]))
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], [1, 1], False, seq_lens=[1, 0, 1])
    np.testing.assert_array_equal(got, ref.astype(np.float32))


@pytest.mark.parametrize("dims,D,causal,lens,rope", [
    ([8, 16, 32], 128, True, [3000, 4096], 0.0),
    ([16, 16], 64, False, [100, 255], 0.0),
    ([128], 128, False, [90, 128], 0.0),
    ([5, 24], 64, False, [119, 61], 0.0),
    ([8, 64], 128, False, [500, 65], 10000.0),
])
def test_backward_with_lengths(dims, D, causal, lens, rope):
    B, H, Hkv = 2, 4, 2
    N = math.prod(dims)
    inp = poison_padding(ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 812, with_dout=True), lens,
                         names=("q", "k", "v", "dout"))
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, True, seq_lens=dev_lens(lens), rope_base=rope)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, seq_lens=lens,
                          rope_base=rope or None)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, sum(1 for n in dims if n > 1), rope=bool(rope))
        for b, L in enumerate(lens):
            assert (g[b, :, L:] == 0).all(), name


def test_lengths_llama_shape_sampled_heads():
    """32 768 tokens as 32x32x32, H=32, H_kv=8, D=128, non-causal, 20 001 valid tokens."""
    c = ta_inputs.CONFIGS[3]
    L = 20001
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_forward(inp, c.B, c.H, c.H_kv, c.N, c.D, list(c.dims), False, "bf16", seq_lens=dev_lens([L]))
    heads = [(0, 5), (0, 30)]
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], list(c.dims), False, heads=heads, seq_lens=[L])
    assert_close(np.stack([got[b, h] for b, h in heads]), ref, "bf16")
    assert (got[:, :, L:] == 0).all()
