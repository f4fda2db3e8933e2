"""The torch.autograd binding (`tensorized_attention`): forward and gradients through
`loss.backward()` against the fp64 oracle, with the hop inputs saved by the forward."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, to_device
from test_gpu_backward import assert_grad_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dims,D,causal,kw", [
    ([8, 16, 32], 128, True, {}),
    ([16, 1, 16], 64, False, {}),
    ([128], 128, True, {}),
    ([4, 200], 64, True, {}),                          # a hop on the generic backward
    ([8, 64], 128, True, {"rope_base": 10000.0, "window": [0, 20]}),
])
def test_autograd_matches_oracle(dims, D, causal, kw):
    import torch
    B, H, Hkv = 1, 4, 2
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 180, with_dout=True)
    q, k, v, do = (to_device(inp, n, "bf16") for n in ("q", "k", "v", "dout"))
    for t in (q, k, v):
        t.requires_grad_(True)
    out = ta.tensorized_attention(q, k, v, dims, causal=causal, **kw)
    (out.float() * do.float()).sum().backward()
    torch.cuda.synchronize()
    ta.ta_device_status()
    okw = {"rope_base": kw.get("rope_base"), "window": kw.get("window")}
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, **okw)
    assert_close(out.detach().float().cpu().numpy(), ref, "bf16")
    rq, rk, rv = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, **okw)
    for name, t, r in (("dq", q, rq), ("dk", k, rk), ("dv", v, rv)):
        assert_grad_close(t.grad.float().cpu().numpy().astype(np.float64), r, name, False,
                          sum(1 for n in dims if n > 1), rope=bool(kw.get("rope_base")))


def test_autograd_forward_only_and_argument_checks():
    import torch
    B, H, Hkv, D, dims = 1, 2, 2, 64, [16, 16]
    inp = ta_inputs.make_inputs(B, H, Hkv, 256, D, "f32", 181)
    q, k, v = (to_device(inp, n, "f32") for n in ("q", "k", "v"))
    with torch.no_grad():
        out = ta.tensorized_attention(q, k, v, dims, causal=False)
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy(), oracle.forward(inp["q"], inp["k"], inp["v"], dims, False), "f32")
    with pytest.raises(ValueError):
        ta.tensorized_attention(q, k, v, [16, 15])
    with pytest.raises(ValueError):
        ta.tensorized_attention(q.cpu(), k.cpu(), v.cpu(), dims)
    # fp32 tensors: gradients through the generic kernels, fp32 throughout
    for t in (q, k, v):
        t.requires_grad_(True)
    out = ta.tensorized_attention(q, k, v, dims, causal=False)
    out.sum().backward()
    torch.cuda.synchronize()
    ta.ta_device_status()
    ones = np.ones((B, H, 256, D))
    for t, r in zip((q, k, v), oracle.backward(ones, inp["q"], inp["k"], inp["v"], dims, False)):
        assert np.abs(t.grad.cpu().numpy() - r).max() <= 1e-4 * max(1.0, np.abs(r).max())
