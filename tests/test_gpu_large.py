"""Maximum-size edge cases: tensors of 2^31 and 2^32 elements, so that every element offset past
32 bits (and past 31) is exercised in the tensor maps and in the kernels' own pointer
arithmetic.  Inputs are drawn on the device; the heads compared with the fp64 oracle include
the last one of the last batch entry (the largest offsets) and are copied to the host one at a
time."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close

pytestmark = pytest.mark.gpu


def run_large(B, H, Hkv, N, D, dims, causal, seed, heads, flags=0, expect=None):
    import torch
    assert B * H * N * D >= 2 ** 31
    if expect is not None:
        plan = ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, flags)
        for e in expect:
            assert e in plan, plan
    q, k, v = ta_inputs.make_device_inputs(B, H, Hkv, N, D, seed)
    out = torch.full((B, H, N, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, causal, flags=flags)
    torch.cuda.synchronize()
    ta.ta_device_status()
    g = H // Hkv
    for b, h in heads:
        ref = oracle.forward(ta_inputs.head_to_host(q, b, h), ta_inputs.head_to_host(k, b, h // g),
                             ta_inputs.head_to_host(v, b, h // g), dims, causal)
        assert_close(out[b, h].float().cpu().numpy()[None, None], ref, "bf16")
    # every element was written (no NaN left from the fill), checked on the device per batch entry
    for b in range(B):
        assert not torch.isnan(out[b]).any()
    del q, k, v, out
    torch.cuda.empty_cache()


def test_short_segments_2_pow_32_elements():
    run_large(4, 32, 8, 64 ** 3, 128, [64, 64, 64], True, 901, [(3, 31), (2, 17), (0, 0)], expect=["tc"])


def test_long_segments_2_pow_31_elements():
    run_large(8, 32, 8, 64 * 1024, 128, [64, 1024], True, 902, [(7, 31), (4, 2)], expect=["tc-long"])


def test_many_heads_2_pow_31_elements_fused_and_generic():
    """131 072 (batch, head) pairs of 128 tokens: the head coordinate of the tensor maps is the
    large one here."""
    heads = [(4095, 31), (2048, 5), (0, 0)]
    run_large(4096, 32, 8, 128, 128, [8, 16], False, 903, heads, expect=["tc-fused"])
    run_large(4096, 32, 8, 128, 128, [8, 16], True, 904, heads, flags=ta.TA_FLAG_NO_TENSOR_CORE, expect=["simt"])
