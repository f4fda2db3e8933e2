"""ta_forward_static: the entry point for callers that are not allowed to allocate device
memory (serving loops where cudaMalloc's device-wide synchronisation is unacceptable, processes
whose memory belongs to a pool the library cannot reach, kernel-launch-only plug-ins).  Its
second value buffer is a fixed array inside the library, shared by all calls and never cleared,
so the check is run twice in a row: the second call starts from the first call's leftovers.

Collected last on purpose (file name), so a failure here cannot hide another test's result.
"""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, to_device, to_numpy

pytestmark = pytest.mark.gpu


def run_pair(B, H, Hkv, dims, D, causal, dtype, seed, check_memory):
    """(existing entry point, static entry point, oracle) outputs for the same seeded inputs."""
    import torch
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, dtype, seed)
    q, k, v = (to_device(inp, n, dtype) for n in ("q", "k", "v"))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    code = ta.TA_DTYPE_BF16 if dtype == "bf16" else ta.TA_DTYPE_F32
    ref = torch.empty((B, H, N, D), dtype=tdt, device="cuda")
    got = torch.full((B, H, N, D), float("nan"), dtype=tdt, device="cuda")
    # (a bf16 head dim other than 64 / 128: the allocating entry point would work on zero-padded copies
    # from its pool; the static one stays on the generic kernels, like TA_FLAG_NO_TENSOR_CORE)
    flags = ta.TA_FLAG_NO_TENSOR_CORE if dtype == "bf16" and D not in (64, 128) else 0
    ta.ta_forward_ex(q, k, v, ref, B, H, Hkv, N, D, dims, causal, dtype=code, flags=flags)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ta.ta_forward_static(q, k, v, got, B, H, Hkv, N, D, dims, causal, dtype=code)
    torch.cuda.synchronize()
    if check_memory:
        # no device memory was taken by the call (the driver's own count of free memory)
        assert torch.cuda.mem_get_info()[0] == free_before
    ta.ta_device_status()
    return to_numpy(ref), to_numpy(got), oracle.forward(inp["q"], inp["k"], inp["v"], dims, causal)


def test_static_scratch_matches_allocating_entry_point_twice():
    cases = [
        (1, 2, 2, [16, 16], 64, False, "f32", 201),      # fp32: both hops on the generic kernel
        (2, 4, 2, [3, 5, 7], 40, True, "f32", 202),      # three hops: out -> scratch -> out
        (1, 2, 1, [4, 160], 64, True, "bf16", 203),      # tensor-core hop into scratch, long-segment hop out
        (1, 4, 2, [6, 5, 7], 40, True, "bf16", 204),     # bf16 on the generic kernel (head dim 40)
    ]
    for call in range(2):            # second round reuses the array with the first round's contents
        for B, H, Hkv, dims, D, causal, dtype, seed in cases:
            ref, got, exact = run_pair(B, H, Hkv, dims, D, causal, dtype, seed + 10 * call, check_memory=call == 1)
            # same kernels in the same order, only the second buffer's address differs: same bits
            np.testing.assert_array_equal(got, ref, err_msg=f"{call} {dims} {dtype}")
            assert_close(got, exact, dtype)


def test_static_scratch_rejects_sizes_beyond_the_array():
    import torch
    # fp32, two generic hops: needs B*H*N*D*4 bytes of scratch = 32 MiB > 16 MiB
    B, H, N, D, dims = 1, 8, 16384, 64, [128, 128]
    assert B * H * N * D * 4 > ta.api.TA_STATIC_SCRATCH_BYTES
    x = torch.zeros((B, H, N, D), dtype=torch.float32, device="cuda")
    out = torch.empty_like(x)
    rc = ta.ta_forward_static(x, x, x, out, B, H, H, N, D, dims, True, dtype=ta.TA_DTYPE_F32, check=False)
    assert rc == ta.TA_ERR_TOO_LARGE
    # a problem that needs no second buffer has no such limit (all hops on the tensor-core kernel)
    B, H, N, D, dims = 1, 16, 16384, 128, [128, 128]
    xb = torch.zeros((B, H, N, D), dtype=torch.bfloat16, device="cuda")
    ob = torch.empty_like(xb)
    assert B * H * N * D * 2 > ta.api.TA_STATIC_SCRATCH_BYTES
    ta.ta_forward_static(xb, xb, xb, ob, B, H, H, N, D, dims, True, dtype=ta.TA_DTYPE_BF16)
    torch.cuda.synchronize()
    assert float(ob.float().abs().max()) == 0.0
