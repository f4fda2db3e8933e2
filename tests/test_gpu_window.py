"""GPU parity of the per-hop sliding-window masks (window[i] = w keeps the keys within w
positions of the query along dimension i) against the fp64 oracle, on every kernel: short
segments, fused trailing hops, long segments (key blocks outside the window are skipped), the
generic fp32 kernel, and the backward.  Tolerances as for the unmasked operator."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward
from test_gpu_backward import assert_grad_close, gpu_backward

pytestmark = pytest.mark.gpu


def run(B, H, Hkv, D, dims, window, causal, dtype, seed, flags=0, rope_base=0.0, expect=None):
    N = math.prod(dims)
    if expect is not None:
        assert expect in ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal,
                                             ta.TA_DTYPE_BF16 if dtype == "bf16" else ta.TA_DTYPE_F32, flags)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, dtype, seed)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, dtype, flags, window=window, rope_base=rope_base)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, window=window, rope_base=rope_base or None)
    assert_close(got, ref, dtype)
    plain = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, rope_base=rope_base or None)
    assert np.abs(ref - plain).max() > 0.05          # the window changes the result visibly


@pytest.mark.parametrize("dims,window,D,causal", [
    ([4, 64], [2, 16], 128, True),
    ([64, 64], [0, 8], 128, False),
    ([32, 8, 32], [4, 0, 5], 128, True),
    ([5, 24, 7], [3, 7, 2], 64, False),
    ([128], [33], 128, True),
    ([3, 100], [0, 40], 64, False),
])
def test_window_short_segments(dims, window, D, causal):
    run(1, 4, 2, D, dims, window, causal, "bf16", 601, flags=ta.TA_FLAG_NO_HOP_FUSION)


@pytest.mark.parametrize("dims,window,D,causal", [
    ([8, 8, 8], [3, 2, 5], 64, False),
    ([4, 8, 16], [0, 3, 4], 128, True),
    ([16, 4, 4, 4], [5, 2, 0, 3], 64, True),
])
def test_window_fused_hops(dims, window, D, causal):
    run(2, 4, 2, D, dims, window, causal, "bf16", 602, expect="tc-fused")


@pytest.mark.parametrize("dims,window,D,causal", [
    ([1000], [100], 64, True),          # most key blocks are skipped
    ([600], [200], 128, False),         # two-sided window
    ([2, 384], [0, 130], 128, True),
    ([300], [5], 64, True),             # rows that see nothing in the first block they visit
    ([130, 3], [129, 2], 64, False),
    ([1300], [150], 64, True),          # pairs of query tiles (n > 1 024): blocks before the window skipped
    ([1200], [300], 128, False),
])
def test_window_long_segments(dims, window, D, causal):
    run(2, 4, 2, D, dims, window, causal, "bf16", 603, expect="tc-long")


def test_window_generic_kernel_and_with_positional_encoding():
    run(2, 4, 2, 40, [3, 5, 7], [2, 3, 4], True, "f32", 604)
    run(1, 4, 2, 64, [200], [37], False, "f32", 605)
    run(1, 4, 2, 128, [8, 64], [3, 20], True, "bf16", 606, rope_base=10000.0)
    run(1, 2, 1, 64, [300], [64], True, "bf16", 607, rope_base=10000.0)    # long + rope: rotated copies, long-segment kernel


def test_window_rejects_negative_entries():
    import torch
    x = torch.zeros(1, 2, 64, 64, dtype=torch.bfloat16, device="cuda")
    rc = ta.ta_forward_ex(x, x, x, torch.empty_like(x), 1, 2, 2, 64, 64, [8, 8], True, window=[2, -1], check=False)
    assert rc == ta.TA_ERR_INVALID_ARG


@pytest.mark.parametrize("dims,window,D,causal", [
    ([8, 16, 32], [3, 0, 9], 128, True),
    ([16, 16], [5, 4], 64, False),
    ([128], [20], 128, True),
])
def test_backward_with_window(dims, window, D, causal):
    B, H, Hkv = 1, 4, 2
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 608, with_dout=True)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, True, window=window)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, window=window)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, sum(1 for n in dims if n > 1))


def test_window_llama_shape_sampled_heads():
    """Config 3's shape (32 768 tokens as 32x32x32, H=32, H_kv=8, D=128) with windows 8, 16, 4."""
    c = ta_inputs.CONFIGS[3]
    window = [8, 16, 4]
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_forward(inp, c.B, c.H, c.H_kv, c.N, c.D, list(c.dims), True, "bf16", window=window)
    heads = [(0, 2), (0, 29)]
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], list(c.dims), True, window=window, heads=heads)
    assert_close(np.stack([got[b, h] for b, h in heads]), ref, "bf16")
