"""Two adjacent hops in one L2-ordered launch (the pair kernel): the second hop's tiles wait on
completion counters of the first hop's tiles of the same block.  Same arithmetic as one launch
per hop, so the result must equal the hop-by-hop run bit for bit, and the oracle within the
forward tolerance."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward

pytestmark = pytest.mark.gpu
PAIR = ta.TA_FLAG_PAIR_HOPS


def plan(B, H, Hkv, D, dims, causal, flags=0):
    return ta.ta_plan_describe(B, H, Hkv, math.prod(dims), D, dims, causal, ta.TA_DTYPE_BF16, flags)


@pytest.mark.parametrize("B,H,Hkv,D,dims,causal,kw", [
    (1, 8, 2, 128, [4, 32, 32], True, {}),          # Llama-like: strided hop then contiguous hop
    (2, 4, 4, 128, [64, 64], True, {}),             # two hops: the first reads v through the KV head
    (1, 8, 2, 128, [2, 64, 64], False, {}),
    (1, 4, 2, 64, [16, 16, 16], True, {}),          # D = 64, eight segments per tile
    (1, 4, 1, 128, [3, 24, 40], True, {}),          # segment lengths that do not divide 128
    (2, 4, 2, 128, [6, 32, 32], True, {"window": [0, 5, 9]}),
    (1, 2, 2, 128, [4, 4, 16, 16], True, {}),       # four hops, two pairs
    (3, 6, 2, 64, [50, 20, 3], True, {}),           # the pair is hops 0 and 1 (the last hop is strided-free n = 3)
    (1, 32, 8, 128, [16, 32, 32], True, {}),        # more units than the lag: steady-state interleaving
])
def test_pair_launch_matches_hop_by_hop_and_oracle(B, H, Hkv, D, dims, causal, kw):
    N = math.prod(dims)
    assert "pair=first" in plan(B, H, Hkv, D, dims, causal, PAIR), plan(B, H, Hkv, D, dims, causal, PAIR)
    assert "pair=" not in plan(B, H, Hkv, D, dims, causal)
    assert "pair=" not in plan(B, H, Hkv, D, dims, causal, PAIR | ta.TA_FLAG_NO_HOP_FUSION)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 501)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", PAIR, **kw)
    hop_by_hop = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", ta.TA_FLAG_NO_HOP_FUSION, **kw)
    np.testing.assert_array_equal(got, hop_by_hop)
    heads = None if B * H * N <= 200000 else [(0, 0), (B - 1, H - 1)]
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, window=kw.get("window"), heads=heads)
    sel = got if heads is None else np.stack([got[b, h] for b, h in heads])
    assert_close(sel, ref, "bf16")


def test_pair_launch_repeats_bit_for_bit_and_takes_a_workspace():
    """The counters live in the caller's workspace when one is given (ta_workspace_bytes accounts
    for them); repeated calls -- the counters are cleared by every call -- reproduce the result."""
    import torch
    B, H, Hkv, D, dims = 1, 8, 2, 128, [8, 32, 32]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 502)
    ref = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", ta.TA_FLAG_NO_HOP_FUSION)
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_FORWARD)
    assert 0 < nbytes <= 1 << 20
    ws = torch.full((nbytes,), 0xAB, dtype=torch.uint8, device="cuda")      # stale contents on purpose
    for _ in range(5):
        got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", PAIR, workspace=ws, workspace_bytes=nbytes)
        np.testing.assert_array_equal(got, ref)
    for _ in range(5):
        np.testing.assert_array_equal(gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", PAIR), ref)


def test_pair_launches_from_concurrent_streams():
    """Two host threads, each with its own stream, run pair launches at the same time: the
    launches are cooperative (all CTAs of one resident before it starts), so neither can starve
    the other's producers; results equal the serial runs."""
    import threading

    import torch
    from helpers import to_device
    cases = [(1, 8, 2, 128, [8, 32, 32], True), (2, 4, 4, 128, [64, 64], True)]
    work = []
    for i, (B, H, Hkv, D, dims, causal) in enumerate(cases):
        N = math.prod(dims)
        inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 510 + i)
        q, k, v = (to_device(inp, n, "bf16") for n in ("q", "k", "v"))
        ref = torch.empty_like(q)
        ta.ta_forward_ex(q, k, v, ref, B, H, Hkv, N, D, dims, causal, flags=ta.TA_FLAG_NO_HOP_FUSION)
        work.append((q, k, v, ref, B, H, Hkv, N, D, dims, causal))
    torch.cuda.synchronize()
    errors = []

    def worker(w):
        q, k, v, ref, B, H, Hkv, N, D, dims, causal = w
        try:
            stream = torch.cuda.Stream()
            outs = [torch.empty_like(q) for _ in range(20)]
            for out in outs:
                ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, causal, flags=PAIR, stream=stream)
            stream.synchronize()
            for out in outs:
                if not torch.equal(out, ref):
                    errors.append(("mismatch", dims))
                    break
        except Exception as e:      # noqa: BLE001 - reported below
            errors.append((repr(e), dims))

    threads = [threading.Thread(target=worker, args=(w,)) for w in work]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    ta.ta_device_status()
    assert not errors, errors
