"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI on seeded
inputs and compare with the fp64 oracle."""
import numpy as np

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

# Tolerances: bf16 storage with fp32 accumulation, and the fp32 path.
BF16_MAX_ABS, BF16_MEAN_ABS = 2e-2, 2e-3
F32_MAX_ABS = 1e-4


def real_hops(dims) -> int:
    return sum(1 for n in dims if n > 1)


def bf16_max_abs(hops: int) -> float:
    """Bound on the largest forward error with bf16 storage.  The stated 2e-2 covers the shapes
    it was stated for (up to three hops).  Every hop stores the value tensor as bf16 -- one
    rounding of at most half an ulp (2^-8 * 2^floor(log2 |x|): 0.0078 for |x| in [2, 4)) per
    hop -- and the later hops, being convex combinations, pass an earlier hop's rounding error
    on without amplifying it, so the worst case grows linearly with the number of hops: beyond
    three hops the bound is 2e-2 * hops / 3.  The bound on the mean error (2e-3) stays."""
    return BF16_MAX_ABS * max(1.0, hops / 3.0)


def to_device(inp: dict, name: str, dtype: str):
    import torch
    if dtype == "bf16":
        bits = torch.from_numpy(inp[name + "_bits"].view(np.int16)).cuda()
        return bits.view(torch.bfloat16)
    return torch.from_numpy(inp[name]).cuda()


def to_numpy(t) -> np.ndarray:
    import torch
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def gpu_forward(inp: dict, B, H, H_kv, N, D, dims, causal, dtype="bf16", flags=0, guard=True,
                **ex):
    """Returns out as float32 numpy [B,H,N,D]; checks guard bands around `out`."""
    import torch
    q, k, v = (to_device(inp, n, dtype) for n in ("q", "k", "v"))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    numel = B * H * N * D
    pad = 1024
    buf = torch.full((numel + 2 * pad,), float("nan"), dtype=tdt, device="cuda")
    out = buf[pad:pad + numel].view(B, H, N, D)
    code = ta.TA_DTYPE_BF16 if dtype == "bf16" else ta.TA_DTYPE_F32
    if flags or ex:
        ta.ta_forward_ex(q, k, v, out, B, H, H_kv, N, D, list(dims), causal, dtype=code,
                         flags=flags, **ex)
    elif dtype == "bf16":
        ta.ta_forward(q, k, v, out, B, H, H_kv, N, D, list(dims), causal)
    else:
        ta.ta_forward_f32(q, k, v, out, B, H, H_kv, N, D, list(dims), causal)
    torch.cuda.synchronize()
    ta.ta_device_status()
    if guard:
        assert torch.isnan(buf[:pad]).all() and torch.isnan(buf[pad + numel:]).all(), \
            "kernel wrote outside `out`"
    return to_numpy(out)


def error_stats(got: np.ndarray, ref: np.ndarray):
    err = np.abs(got.astype(np.float64) - ref)
    return float(err.max()), float(err.mean())


def assert_close(got, ref, dtype, hops: int = 3):
    assert np.isfinite(got).all(), "non-finite output"
    mx, mean = error_stats(got, ref)
    if dtype == "bf16":
        assert mx <= bf16_max_abs(hops) and mean <= BF16_MEAN_ABS, (mx, mean, hops)
    else:
        assert mx <= F32_MAX_ABS, (mx, mean)
    return mx, mean


def check_case(B, H, H_kv, N, D, dims, causal, dtype, seed, flags=0, heads=None):
    inp = ta_inputs.make_inputs(B, H, H_kv, N, D, dtype, seed)
    got = gpu_forward(inp, B, H, H_kv, N, D, dims, causal, dtype, flags)
    if heads is None:
        ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)
        return assert_close(got, ref, dtype, real_hops(dims))
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal, heads=heads)
    sel = np.stack([got[b, h] for b, h in heads])
    return assert_close(sel, ref, dtype, real_hops(dims))
