"""bf16 head dims without a tensor-core kernel of their own (100 as in OpenLlama-3B, 96, 80, 40, odd
ones): the library runs the hops of Algorithm 1 on zero-padded copies (64 or 128 columns).  Zero
columns add nothing to Q K^T and give zero output columns, so the results must match the oracle on the
unpadded problem like any other tensor-core run -- forward, positional encoding (the rotation pairs
feature c with c + D/2 and uses base^(-2c/D): both must survive the padding), masks, windows, valid
lengths, hop ranges with saved hop inputs, and the backward with both gradient types."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, gpu_forward, real_hops, to_device
from test_gpu_backward import assert_grad_close, gpu_backward, hops_of

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dims,D,causal,H,Hkv", [
    ([8, 16, 32], 100, True, 4, 2),        # three tensor-core hops, padded to 128
    ([4, 4, 8], 100, False, 4, 4),         # trailing hops fused in shared memory
    ([16, 16], 40, True, 2, 1),            # padded to 64
    ([5, 24, 7], 96, True, 4, 2),          # ragged tiles
    ([3, 300], 80, False, 2, 2),           # a long-segment hop
    ([6, 20], 72, True, 4, 1),
    ([8, 16], 17, True, 2, 2),             # odd: halves of 8 and 9 columns
    ([16, 8], 2, False, 2, 1),
    ([4, 32], 127, True, 2, 2),
    ([32, 32], 65, False, 4, 2),
])
def test_forward_other_head_dims(dims, D, causal, H, Hkv):
    B, N = 2, math.prod(dims)
    plan = ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, 0)
    assert f"padded_head_dim={64 if D <= 64 else 128}" in plan and "simt" not in plan
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1301)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16")
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)
    assert_close(got, ref, "bf16", real_hops(dims))
    # the generic kernels on the unpadded tensors, when asked for, agree too
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", ta.TA_FLAG_NO_TENSOR_CORE)
    assert_close(got, ref, "bf16", real_hops(dims))


@pytest.mark.parametrize("dims,D,causal", [
    ([8, 16, 32], 100, True),
    ([16, 16], 40, False),
    ([2, 300], 96, True),                  # long-segment hop on rotated copies of the padded tensors
    ([6, 20], 6, True),
])
def test_forward_other_head_dims_with_positional_encoding(dims, D, causal):
    B, H, Hkv, N = 1, 4, 2, math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1302)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", rope_base=10000.0)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, rope_base=10000.0)
    assert np.abs(ref - oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)).max() > 0.05
    assert_close(got, ref, "bf16", real_hops(dims))


def test_forward_other_head_dims_with_masks_windows_lengths_and_scale():
    import torch
    B, H, Hkv, D, dims = 2, 4, 2, 100, [6, 20, 4]
    N = math.prod(dims)
    rng = np.random.default_rng(5)
    masks = []
    for n in dims:
        m = (rng.random((n, n)) < 0.6).astype(np.uint8)
        m[np.arange(n), np.arange(n)] = 1
        masks.append(m)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1303)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", hop_masks=masks)
    assert_close(got, oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, masks=masks), "bf16")
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, False, "bf16", window=[2, 5, 0])
    assert_close(got, oracle.forward(inp["q"], inp["k"], inp["v"], dims, False, window=[2, 5, 0]), "bf16")
    lens = [N - 37, 101]
    dev = torch.tensor(lens, dtype=torch.int32, device="cuda")
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", seq_lens=dev)
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, seq_lens=lens)
    for b, ln in enumerate(lens):
        assert_close(got[b, :, :ln], ref[b, :, :ln], "bf16")
    # an explicit scale is used as given; the default is 1 / sqrt(D) of the caller's D, not of the padded one
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", softmax_scale=0.05)
    assert_close(got, oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, scale=0.05), "bf16")


def test_saved_hop_inputs_come_back_unpadded():
    """TA_FLAG_SAVE_HOPS with a padded head dim: the caller's workspace receives X_1..X_{m-1} in the
    caller's layout (what ta_backward_ex's saved_hops and a later hop-range call expect)."""
    import torch
    B, H, Hkv, D, dims = 1, 4, 2, 100, [8, 16, 4]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1304)
    q, k, v = (to_device(inp, n, "bf16") for n in ("q", "k", "v"))
    out = torch.empty((B, H, N, D), dtype=torch.bfloat16, device="cuda")
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_FORWARD_SAVE)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    flags = ta.TA_FLAG_SAVE_HOPS | ta.TA_FLAG_NO_HOP_FUSION
    ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, True, flags=flags, workspace=ws, workspace_bytes=nbytes)
    torch.cuda.synchronize()
    ref_out, xs = oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, return_xs=True)
    assert_close(out.float().cpu().numpy(), ref_out, "bf16")
    saved_off = nbytes - (len(dims) - 1) * B * H * N * D * 2
    saved = ws[saved_off:].view(torch.bfloat16).view(len(dims) - 1, B, H, N, D).float().cpu().numpy()
    for j in range(1, len(dims)):
        assert_close(saved[j - 1], np.stack([x[j] for x in xs]).reshape(B, H, N, D), "bf16")


@pytest.mark.parametrize("dims,D,causal,B,H,Hkv,rope", [
    ([8, 16, 32], 100, True, 1, 4, 2, 0.0),
    ([16, 16], 40, False, 2, 4, 4, 0.0),
    ([5, 24, 7], 96, True, 1, 4, 2, 10000.0),
    ([3, 300], 80, True, 1, 2, 1, 0.0),           # long-segment backward on the padded tensors
    ([8, 16], 17, True, 1, 2, 2, 0.0),
])
@pytest.mark.parametrize("grad_f32", [False, True])
def test_backward_other_head_dims(dims, D, causal, B, H, Hkv, rope, grad_f32):
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1305, with_dout=True)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32, rope_base=rope)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, **({"rope_base": rope} if rope else {}))
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, grad_f32, hops_of(dims), rope=bool(rope))


def test_autograd_other_head_dim():
    import torch
    B, H, Hkv, D, dims = 1, 4, 2, 100, [8, 16, 8]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1306, with_dout=True)
    q, k, v = (to_device(inp, n, "bf16").requires_grad_(True) for n in ("q", "k", "v"))
    out = ta.tensorized_attention(q, k, v, dims, causal=True)
    out.backward(to_device(inp, "dout", "bf16"))
    torch.cuda.synchronize()
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, True)
    assert_close(out.detach().float().cpu().numpy(), oracle.forward(inp["q"], inp["k"], inp["v"], dims, True), "bf16")
    for name, t, r in zip(("dq", "dk", "dv"), (q, k, v), ref):
        assert_grad_close(t.grad.float().cpu().numpy().astype(np.float64), r, name, False, hops_of(dims))


def test_saved_hop_inputs_at_odd_offsets():
    """Tensor sizes that are no multiple of 16 bytes: the saved hop inputs behind the first one start
    at odd offsets in the caller's workspace and must still arrive intact."""
    import torch
    B, H, Hkv, D, dims = 1, 3, 3, 17, [3, 5, 7]
    N = math.prod(dims)
    assert (B * H * N * D * 2) % 16 != 0
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 1307)
    q, k, v = (to_device(inp, n, "bf16") for n in ("q", "k", "v"))
    out = torch.empty((B, H, N, D), dtype=torch.bfloat16, device="cuda")
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_FORWARD_SAVE)
    ws = torch.zeros(nbytes + 256, dtype=torch.uint8, device="cuda")
    ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, False, flags=ta.TA_FLAG_SAVE_HOPS, workspace=ws,
                     workspace_bytes=nbytes)
    torch.cuda.synchronize()
    ta.ta_device_status()
    ref_out, xs = oracle.forward(inp["q"], inp["k"], inp["v"], dims, False, return_xs=True)
    assert_close(out.float().cpu().numpy(), ref_out, "bf16")
    tensor = B * H * N * D * 2
    saved_off = nbytes - (len(dims) - 1) * tensor
    for j in range(1, len(dims)):
        got = ws[saved_off + (j - 1) * tensor: saved_off + j * tensor].clone().view(torch.bfloat16).view(B, H, N, D)
        assert_close(got.float().cpu().numpy(), np.stack([x[j] for x in xs]).reshape(B, H, N, D), "bf16")
    assert (ws[nbytes:] == 0).all()
