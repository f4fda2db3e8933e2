"""GPU parity of the tensorized positional encoding (per-hop RoPE fused into the kernels)
against the fp64 oracle, same tolerances as the plain forward: bf16 max abs <= 2e-2 and mean
abs <= 2e-3; fp32 path max abs <= 1e-4."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward

pytestmark = pytest.mark.gpu
BASE = 10000.0


def run(B, H, Hkv, D, dims, causal, dtype, seed, flags=0, base=BASE, heads=None):
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, dtype, seed)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, dtype, flags, rope_base=base)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, rope_base=base, heads=heads)
    if heads is not None:
        got = np.stack([got[b, h] for b, h in heads])
    assert_close(got, ref, dtype)
    plain = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, heads=heads)
    assert np.abs(ref - plain).max() > 0.05          # the encoding changes the result visibly


@pytest.mark.parametrize("dims,D,causal", [
    ([4, 64], 128, True), ([64, 64], 128, False), ([32, 8, 32], 128, True), ([16, 16], 64, True),
    ([128, 3], 128, True), ([2, 4, 12], 64, True), ([5, 24, 7], 128, False), ([3, 100], 64, True),
    ([128], 128, True), ([2, 48], 128, True), ([6, 40], 64, False),
])
def test_rope_tensor_core(dims, D, causal):
    run(1, 4, 2, D, dims, causal, "bf16", seed=401)


def test_rope_batch_gqa_and_other_base():
    run(2, 8, 2, 128, [8, 64], True, "bf16", seed=402, base=500000.0)


@pytest.mark.parametrize("dims,D,causal", [([3, 5, 7], 40, True), ([200], 64, False), ([16, 16], 64, False)])
def test_rope_generic_f32(dims, D, causal):
    run(2, 4, 2, D, dims, causal, "f32", seed=403)


def test_rope_generic_bf16_and_mixed_paths():
    run(1, 4, 2, 64, [6, 20], True, "bf16", seed=404, flags=ta.TA_FLAG_NO_TENSOR_CORE)
    run(1, 2, 1, 64, [4, 160], True, "bf16", seed=405)      # hop 1 (n = 160): long-segment kernel on rotated copies


def test_rope_rejects_odd_head_dim_and_negative_base():
    import torch
    x = torch.zeros(1, 2, 16, 33, dtype=torch.float32, device="cuda")
    rc = ta.ta_forward_ex(x, x, x, torch.empty_like(x), 1, 2, 2, 16, 33, [16], True,
                          dtype=ta.TA_DTYPE_F32, rope_base=100.0, check=False)
    assert rc == ta.TA_ERR_UNSUPPORTED
    y = torch.zeros(1, 2, 16, 32, dtype=torch.float32, device="cuda")
    rc = ta.ta_forward_ex(y, y, y, torch.empty_like(y), 1, 2, 2, 16, 32, [16], True,
                          dtype=ta.TA_DTYPE_F32, rope_base=-1.0, check=False)
    assert rc == ta.TA_ERR_INVALID_ARG


def test_rope_llama_shape_sampled_heads():
    """Config 3 (32 768 tokens as 32x32x32, H=32, H_kv=8, D=128) with the positional encoding."""
    c = ta_inputs.CONFIGS[3]
    run(c.B, c.H, c.H_kv, c.D, list(c.dims), True, "bf16", seed=c.seed, heads=[(0, 5), (0, 30)])


@pytest.mark.parametrize("dims,D,causal", [
    ([2048], 128, True),            # ordinary attention with RoPE, positions up to 2047
    ([4, 1000], 64, False),
    ([3, 300, 2], 128, True),       # short, long, short: only the long hop works on rotated copies
])
def test_rope_long_segments_tensor_core(dims, D, causal):
    """Segments longer than 128 with the positional encoding: Q and K are rotated once per hop into
    library-owned copies and the long-segment tensor-core kernel runs on those."""
    B, H, Hkv = 1, 4, 2
    N = math.prod(dims)
    assert "tc-long" in ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, 0)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 410)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", rope_base=10000.0)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, rope_base=10000.0)
    assert_close(got, ref, "bf16")
    plain = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)
    assert np.abs(ref - plain).max() > 0.05
