"""Hop fusion on the GPU: when the trailing dimensions span at most one 128-row tile their hops
run as one pass (Q, K, value tile read once).  Checked against the fp64 oracle (bf16 tolerance:
max abs <= 2e-2, mean abs <= 2e-3) and against the same library run hop by hop
(TA_FLAG_NO_HOP_FUSION).  The fused pass rounds the value tensor to fp16 between hops exactly
as the unfused tensor-core passes do; only the order of the fp32 sums over a row's keys differs
(the keys of a mode-i vector are interleaved with other columns of the tile), so the two runs
agree to about one bf16 unit in the last place."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward

pytestmark = pytest.mark.gpu


def assert_same_up_to_summation_order(a, b):
    np.testing.assert_allclose(a, b, rtol=2.0 ** -6, atol=2.0 ** -9)
    assert (a != b).mean() < 0.02              # and almost every element is the same bits


@pytest.mark.parametrize("dims,D,causal,H,Hkv", [
    ([8, 8, 8], 64, False, 12, 12),        # the paper's 512-token, three-level shape: hops 1, 2 fused
    ([16, 4, 4, 4], 64, False, 12, 12),    # 1024 tokens in four levels: three hops fused
    ([16, 16, 4], 64, True, 4, 2),
    ([4, 8, 16], 128, True, 8, 2),         # block = 128: one block per tile
    ([8, 16], 128, True, 4, 2),            # every hop fused; the first fused hop reads v through the KV head
    ([2, 3, 5, 7], 64, True, 4, 4),        # block = 105: partly filled tile, odd strides
    ([64, 2, 2, 2, 2, 2, 2], 128, False, 2, 1),   # six fused hops
    ([5, 1, 6, 1, 4], 64, True, 2, 2),     # unit dimensions inside the fused group
])
def test_fused_matches_oracle_and_unfused(dims, D, causal, H, Hkv):
    B, N = 2, math.prod(dims)
    plan = ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, 0)
    assert "tc-fused" in plan, plan
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", seed=501)
    fused = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16")
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)
    assert_close(fused, ref, "bf16")
    unfused = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", flags=ta.TA_FLAG_NO_HOP_FUSION)
    assert_same_up_to_summation_order(fused, unfused)


def test_large_problems_with_head_dim_64_stay_unfused():
    """At D = 64 the fused pass is bound by its softmax chain, not by HBM: the planner keeps it
    for problems small enough to be launch-bound (measured on B200)."""
    assert "tc-fused" in ta.ta_plan_describe(2, 12, 12, 512, 64, [8, 8, 8], False, ta.TA_DTYPE_BF16, 0)
    assert "tc-fused" not in ta.ta_plan_describe(512, 12, 12, 512, 64, [8, 8, 8], False, ta.TA_DTYPE_BF16, 0)
    assert "tc-fused" in ta.ta_plan_describe(512, 12, 12, 512, 128, [8, 8, 8], False, ta.TA_DTYPE_BF16, 0)


def test_fusion_is_off_where_it_cannot_apply():
    # Llama shapes: no trailing pair of dimensions fits a tile
    assert "tc-fused" not in ta.ta_plan_describe(1, 32, 8, 32768, 128, [32, 32, 32], True, ta.TA_DTYPE_BF16, 0)
    # saving hop outputs for the backward, or asking for it, keeps the hops apart
    for flags in (ta.TA_FLAG_NO_HOP_FUSION, ta.TA_FLAG_SAVE_HOPS):
        assert "tc-fused" not in ta.ta_plan_describe(1, 4, 2, 512, 64, [8, 8, 8], True, ta.TA_DTYPE_BF16, flags)


def test_many_tiles_and_launch_count():
    """Enough tiles for several per CTA (both load stages in use) and one launch fewer."""
    B, H, Hkv, D, dims = 2, 16, 4, 128, [64, 8, 8]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", seed=502)
    n0 = ta.ta_launch_count()
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16")
    assert ta.ta_launch_count() - n0 == 2          # hop 0, then hops 1 + 2 in one pass
    heads = [(0, 0), (1, 7), (1, 15)]
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, heads=heads)
    assert_close(np.stack([got[b, h] for b, h in heads]), ref, "bf16")
    unfused = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", flags=ta.TA_FLAG_NO_HOP_FUSION)
    assert_same_up_to_summation_order(got, unfused)
