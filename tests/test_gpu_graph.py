"""The calls only enqueue work, so they can be captured into a CUDA graph (no allocation, no
synchronisation, no host read-back inside the call when a workspace is supplied or none is
needed): a captured forward / backward, replayed on new input values in the same buffers, must
reproduce the eager result bit for bit."""
import math

import numpy as np
import pytest

import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import to_device

pytestmark = pytest.mark.gpu


def fresh(B, H, Hkv, N, D, seed, with_dout=False):
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", seed, with_dout=with_dout)
    names = ("q", "k", "v", "dout") if with_dout else ("q", "k", "v")
    return [to_device(inp, n, "bf16") for n in names]


@pytest.mark.parametrize("B,H,Hkv,D,dims,causal,kw", [
    (1, 8, 2, 128, [8, 16, 32], True, {}),                       # per-hop kernels, overlapped launches
    (2, 4, 2, 128, [16, 4, 4], False, {}),                       # fused trailing hops
    (1, 2, 1, 64, [2, 300], True, {}),                           # long segments
    (1, 4, 2, 128, [16, 64], True, {"rope_base": 10000.0, "window": [4, 0]}),
])
def test_captured_forward_replays_on_new_inputs(B, H, Hkv, D, dims, causal, kw):
    import torch
    N = math.prod(dims)
    q, k, v = fresh(B, H, Hkv, N, D, 150)
    out = torch.empty_like(q)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, causal, **kw)     # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, causal, **kw)
    for seed in (151, 152):
        q2, k2, v2 = fresh(B, H, Hkv, N, D, seed)
        q.copy_(q2), k.copy_(k2), v.copy_(v2)
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        got = out.clone()
        ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, causal, **kw)
        torch.cuda.synchronize()
        ta.ta_device_status()
        assert torch.equal(got, out)


def test_captured_backward_replays_on_new_inputs():
    import torch
    B, H, Hkv, D, dims, causal = 1, 4, 2, 128, [8, 16, 32], True
    N = math.prod(dims)
    q, k, v, do = fresh(B, H, Hkv, N, D, 160, with_dout=True)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_BACKWARD)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")

    def call():
        ta.ta_backward_ex(do, q, k, v, dq, dk, dv, B, H, Hkv, N, D, dims, causal, workspace=ws, workspace_bytes=nbytes)

    call()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    q2, k2, v2, do2 = fresh(B, H, Hkv, N, D, 161, with_dout=True)
    q.copy_(q2), k.copy_(k2), v.copy_(v2), do.copy_(do2)
    for t in (dq, dk, dv):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    got = [t.clone() for t in (dq, dk, dv)]
    call()
    torch.cuda.synchronize()
    ta.ta_device_status()
    for a, b in zip(got, (dq, dk, dv)):
        assert torch.equal(a, b)
