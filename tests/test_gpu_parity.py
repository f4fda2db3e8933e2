"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle, element by element
on the same seeded inputs.  Tolerances: bf16 storage max abs <= 2e-2 and mean abs <= 2e-3;
fp32 path max abs <= 1e-4."""
import math

import numpy as np
import pytest

import oracle
import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import assert_close, check_case, gpu_forward, to_device

pytestmark = pytest.mark.gpu


# ---------------------------------------------------------------- fp32 / generic kernel
def test_config1_f32():
    c = ta_inputs.CONFIGS[1]
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_forward(inp, c.B, c.H, c.H_kv, c.N, c.D, c.dims, c.causal, "f32")
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], c.dims, c.causal)
    assert_close(got, ref, "f32")


@pytest.mark.parametrize("dims,D,causal", [
    ([3, 5, 7], 40, True), ([3, 5, 7], 40, False), ([200], 64, True), ([70], 96, False),
    ([2, 33], 32, True), ([17, 1, 3], 8, True), ([1, 1], 16, False), ([4, 4, 4, 4], 72, True),
])
def test_generic_f32_ragged(dims, D, causal):
    check_case(2, 4, 2, math.prod(dims), D, dims, causal, "f32", seed=101)


@pytest.mark.parametrize("dims,D,causal", [([6, 20], 64, True), ([150], 128, False), ([3, 5, 7], 48, True)])
def test_generic_bf16(dims, D, causal):
    check_case(1, 4, 2, math.prod(dims), D, dims, causal, "bf16", seed=102,
               flags=ta.TA_FLAG_NO_TENSOR_CORE)


# ---------------------------------------------------------------- tensor-core kernel
@pytest.mark.parametrize("dims,D,causal", [
    ([4, 64], 128, True),          # strided hop with 32 segments/tile + contiguous hop, 2 segments/tile
    ([64, 64], 128, False),
    ([32, 8, 32], 128, True),      # three hops, 4 segments per tile
    ([16, 16], 64, True),          # D = 64, 8 segments per tile
    ([128, 3], 128, True),         # one segment per tile, ragged inner extent (3 < ci)
    ([2, 4, 12], 64, True),        # n does not divide 128: partly filled tiles
    ([5, 24, 7], 128, False),      # odd everything: clipped boxes on the inner dimension
    ([3, 100], 128, True),         # n = 100: single partly filled segment per tile
    ([2, 2, 2, 2, 2, 2, 2], 64, True),
])
def test_tensor_core_small(dims, D, causal):
    check_case(1, 4, 2, math.prod(dims), D, dims, causal, "bf16", seed=103)


# Shapes of the paper's bidirectional workloads (Section 3.3: 512 tokens as {32,16} and {8,8,8};
# Appendix D: 1024 patches as 2 to 4 levels), RoBERTa-like heads (H = 12, D = 64), non-causal.
@pytest.mark.parametrize("dims", [[32, 16], [8, 8, 8], [32, 32], [16, 16, 4], [16, 4, 4, 4], [8, 128], [128, 8]])
def test_encoder_shapes_noncausal(dims):
    check_case(2, 12, 12, math.prod(dims), 64, dims, False, "bf16", seed=112)


def test_tensor_core_batch_and_gqa_indexing():
    check_case(3, 8, 2, 512, 128, [8, 64], True, "bf16", seed=104)
    check_case(2, 6, 6, 256, 64, [16, 16], False, "bf16", seed=105)


def test_mixed_paths_use_scratch():
    # hop 0 on tensor cores, hop 1 (n = 160 > 128) on the generic kernel
    check_case(1, 2, 1, 4 * 160, 64, [4, 160], True, "bf16", seed=106)


# ---------------------------------------------------------------- long segments (n > 128): key-block loop
@pytest.mark.parametrize("dims,D,causal,H,Hkv", [
    ([256], 128, True, 4, 2),          # ordinary causal attention, two key blocks
    ([300], 64, False, 4, 4),          # ragged last block
    ([2, 384], 128, True, 8, 2),
    ([130, 3], 64, True, 2, 1),        # long hop over a strided dimension
    ([3, 129], 128, False, 2, 2),
    ([1000], 64, True, 2, 2),          # eight key blocks: running maximum moves many times
    ([181, 2], 128, True, 4, 1),       # two ragged query tiles per segment, strided, one item per tile
    ([2, 513], 64, False, 2, 2),       # five tiles, one position in the last
    ([1300], 64, True, 2, 1),          # past the one-tile-per-item range: pairs of query tiles, ragged
    ([1100, 2], 128, False, 2, 2),     # the same, strided and not causal
])
def test_long_segments_tensor_core(dims, D, causal, H, Hkv):
    plan = ta.ta_plan_describe(1, H, Hkv, math.prod(dims), D, dims, causal, ta.TA_DTYPE_BF16, 0)
    assert "tc-long" in plan
    # segments of up to 1 024 positions: one query tile per work item (two CTAs per SM); longer: pairs
    assert ("tiles_per_item=1" if max(dims) <= 1024 else "tiles_per_item=2") in plan
    check_case(2, H, Hkv, math.prod(dims), D, dims, causal, "bf16", seed=113)


@pytest.mark.parametrize("n,growth", [(1000, 3.0), (1300, 3.0), (1024, 0.4), (640, -0.12)])
def test_long_segments_running_maximum_jumps(n, growth):
    """Keys whose size changes from key block to key block: with growth 3 the row maxima jump by many
    units (log2 domain) at most blocks, with 0.4 by a few, with a negative growth they never rise after
    the first block.  The kernel rescales the accumulated output whenever a row's maximum moved; all
    three regimes must give the oracle's rows (one query tile per item up to 1 024 positions, pairs of
    tiles beyond)."""
    from paper_2410_20926_b200.inputs import bf16_bits, bf16_to_f32
    B, H, Hkv, D = 1, 2, 1, 64
    inp = ta_inputs.make_inputs(B, H, Hkv, n, D, "bf16", 117)
    factor = (1.0 + growth * (np.arange(n) // 128)).astype(np.float32)
    bits = bf16_bits(inp["k"] * factor[None, None, :, None])
    inp["k"], inp["k_bits"] = bf16_to_f32(bits), bits
    got = gpu_forward(inp, B, H, Hkv, n, D, [n], False, "bf16")
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], [n], False)
    assert_close(got, ref, "bf16", 1)
    got = gpu_forward(inp, B, H, Hkv, n, D, [n], True, "bf16")
    assert_close(got, oracle.forward(inp["q"], inp["k"], inp["v"], [n], True), "bf16", 1)


def test_full_attention_4096_sampled_heads():
    """One dimension = ordinary attention (Eq. 1) at a length where the loop runs 32 key blocks."""
    check_case(1, 8, 2, 4096, 128, [4096], True, "bf16", seed=114, heads=[(0, 0), (0, 5)])


def test_full_attention_8192_llama_heads_sampled():
    """Ordinary causal attention at 8 192 tokens with Llama head shapes (64 key blocks per segment,
    32 pairs of query tiles): one whole head against the oracle."""
    check_case(1, 32, 8, 8192, 128, [8192], True, "bf16", seed=115, heads=[(0, 13)])


def test_unit_dims_and_broadcast():
    check_case(1, 4, 2, 64, 64, [1, 64, 1], True, "bf16", seed=107)
    inp = ta_inputs.make_inputs(2, 4, 2, 1, 64, "bf16", 108)
    got = gpu_forward(inp, 2, 4, 2, 1, 64, [1], True, "bf16")
    np.testing.assert_array_equal(got, np.repeat(inp["v"], 2, axis=1))


def test_hop_range_matches_oracle_intermediates():
    B, H, Hkv, D, dims = 1, 2, 1, 128, [8, 16, 32]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 109)
    _, xs = oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, return_xs=True)
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", hop_begin=0, hop_end=1)
    assert_close(got, np.stack([x[1] for x in xs])[None], "bf16")


def test_save_hops_workspace():
    import torch
    B, H, Hkv, D, dims = 1, 2, 1, 64, [4, 8, 16]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 110)
    nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_FORWARD_SAVE)
    assert nbytes == 2 * B * H * N * D * 2
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    got = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", flags=ta.TA_FLAG_SAVE_HOPS,
                      workspace=ws, workspace_bytes=nbytes)
    ref, xs = oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, return_xs=True)
    assert_close(got, ref, "bf16")
    saved = ws.view(torch.bfloat16).view(2, B, H, N, D).float().cpu().numpy()
    for j in range(2):
        assert_close(saved[j], np.stack([x[j + 1] for x in xs])[None], "bf16")


def test_deterministic_and_in_place_safe():
    c = ta_inputs.CONFIGS[2]
    inp = ta_inputs.make_inputs(1, 4, 2, c.N, c.D, "bf16", 111)
    a = gpu_forward(inp, 1, 4, 2, c.N, c.D, c.dims, True, "bf16")
    b = gpu_forward(inp, 1, 4, 2, c.N, c.D, c.dims, True, "bf16")
    np.testing.assert_array_equal(a, b)


# ---------------------------------------------------------------- the benchmark configurations
def test_config2_bf16():
    c = ta_inputs.CONFIGS[2]
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_forward(inp, c.B, c.H, c.H_kv, c.N, c.D, c.dims, c.causal, "bf16")
    ref = oracle.forward(inp["q"], inp["k"], inp["v"], c.dims, c.causal)
    assert_close(got, ref, "bf16")


HIST_EDGES = [0.0, 1e-4, 1e-3, 2e-3, 4e-3, 8e-3, 1.2e-2, 1.6e-2, 2e-2, 1.0]


@pytest.mark.parametrize("idx", [3, 4, 5])
def test_full_size_configs_every_head(idx):
    """Full-size runs in the launch configuration the benchmark times; EVERY head is compared
    with the oracle element by element (the oracle computes one head at a time, so the
    reference never exists as a whole).  Also collects the histogram of the absolute errors;
    with TA_ERROR_HISTOGRAM=<file> it is appended there as text."""
    import os
    c = ta_inputs.CONFIGS[idx]
    inp = ta_inputs.make_config_inputs(c)
    got = gpu_forward(inp, c.B, c.H, c.H_kv, c.N, c.D, c.dims, c.causal, "bf16")
    hist = np.zeros(len(HIST_EDGES) - 1, dtype=np.int64)
    worst, total, count = 0.0, 0.0, 0
    for b in range(c.B):
        for h in range(c.H):
            ref = oracle.forward(inp["q"], inp["k"], inp["v"], c.dims, c.causal, heads=[(b, h)])[0]
            err = np.abs(got[b, h].astype(np.float64) - ref)
            mx, mean = assert_close(got[b, h], ref, "bf16")        # per head: max <= 2e-2, mean <= 2e-3
            worst = max(worst, mx)
            total += float(err.sum())
            count += err.size
            hist += np.histogram(err, bins=HIST_EDGES)[0]
    assert hist.sum() == count and hist[-1] == 0
    path = os.environ.get("TA_ERROR_HISTOGRAM")
    if path:
        with open(path, "a") as f:
            f.write(f"config {idx}: {count} outputs, max abs err {worst:.5f}, mean abs err {total / count:.6f}\n")
            for lo, hi, n in zip(HIST_EDGES[:-1], HIST_EDGES[1:], hist):
                f.write(f"  [{lo:g}, {hi:g}): {int(n)} ({n / count:.3e})\n")
    # properties that hold at any size: finite, inside the range of V per column
    assert np.isfinite(got).all()
    g = c.H // c.H_kv
    vmax = np.repeat(inp["v"].max(axis=2), g, axis=1)[:, :, None, :]
    vmin = np.repeat(inp["v"].min(axis=2), g, axis=1)[:, :, None, :]
    assert (got <= vmax + 0.05).all() and (got >= vmin - 0.05).all()


@pytest.mark.parametrize("B,H,Hkv,D,dims,dtype,flags", [
    (1, 4, 2, 128, [8, 16, 32], "bf16", 0),                       # tensor-core hops
    (1, 4, 2, 40, [5, 6, 7], "bf16", 0),                          # generic hops (head dim 40)
    (2, 2, 1, 64, [4, 160, 2], "bf16", 0),                        # tensor-core, long-segment, tensor-core
    (1, 2, 2, 32, [4, 4, 8], "f32", 0),                           # fp32
    (1, 4, 2, 128, [8, 16, 32], "bf16", "save"),                  # with the hop inputs saved
    (1, 4, 2, 40, [5, 6, 7], "bf16", "save"),
])
def test_hop_ranges_compose_to_the_single_call(B, H, Hkv, D, dims, dtype, flags):
    """Running hops [0, j) and then [j, m) (the second call reads its value tensor from `out`)
    gives the result of the single call, for every split point and every kind of plan --
    including plans in which the first hop of the second call cannot update `out` in place."""
    import torch
    N = math.prod(dims)
    m = len(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, dtype, 116)
    q, k, v = (to_device(inp, n, dtype) for n in ("q", "k", "v"))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    code = ta.TA_DTYPE_BF16 if dtype == "bf16" else ta.TA_DTYPE_F32
    ref_out, xs = oracle.forward(inp["q"], inp["k"], inp["v"], dims, True, return_xs=True)
    whole = torch.empty((B, H, N, D), dtype=tdt, device="cuda")
    # (bf16 between the hops, as a call that stops after hop j must leave it in `out`)
    base = ta.TA_FLAG_NO_HOP_FUSION | ta.TA_FLAG_BF16_INTERMEDIATES
    ta.ta_forward_ex(q, k, v, whole, B, H, Hkv, N, D, dims, True, dtype=code, flags=base)
    for j in range(1, m):
        out = torch.empty((B, H, N, D), dtype=tdt, device="cuda")
        kw = {}
        if flags == "save":
            nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, code, ta.TA_WS_FORWARD_SAVE) + B * H * N * D * 4
            kw = dict(workspace=torch.empty(nbytes, dtype=torch.uint8, device="cuda"), workspace_bytes=nbytes)
        f = base | (ta.TA_FLAG_SAVE_HOPS if flags == "save" else 0)
        ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, True, dtype=code, flags=f, hop_begin=0, hop_end=j, **kw)
        torch.cuda.synchronize()
        mid = out.float().cpu().numpy()
        assert_close(mid, np.stack([x[j] for x in xs]).reshape(B, H, N, D), dtype)
        ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, True, dtype=code, flags=f, hop_begin=j, hop_end=m, **kw)
        torch.cuda.synchronize()
        ta.ta_device_status()
        assert torch.equal(out, whole), (j, dims)
    assert_close(whole.float().cpu().numpy(), ref_out, dtype)


def test_out_overlapping_an_input_is_rejected():
    import torch
    B, H, N, D = 1, 2, 256, 64
    x = torch.zeros((B, H, N, D), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((2, B, H, N, D), dtype=torch.bfloat16, device="cuda")
    assert ta.ta_forward(x, x, x, x, B, H, H, N, D, [16, 16], True, check=False) == ta.TA_ERR_INVALID_ARG
    assert ta.ta_forward(x, y[0], x, y.view(-1)[64:64 + x.numel()].view_as(x), B, H, H, N, D, [16, 16], True,
                         check=False) == ta.TA_ERR_INVALID_ARG
    assert ta.ta_forward(x, x, x, y[1], B, H, H, N, D, [16, 16], True, check=False) == ta.TA_OK


def test_forward_host_back_to_back_calls_use_both_staging_sets():
    """Host-buffer entry point: three calls in a row on one stream (uploads overlap the previous
    call's kernels and download); every result must equal the device-resident run of its input."""
    import torch
    B, H, Hkv, D, dims = 1, 4, 2, 128, [8, 16, 32]
    N = math.prod(dims)
    stream = torch.cuda.current_stream()
    outs, refs = [], []
    for i in range(3):
        inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 120 + i)
        host = [torch.from_numpy(inp[n + "_bits"].view(np.int16)).view(torch.bfloat16).pin_memory() for n in "qkv"]
        out_h = torch.empty((B, H, N, D), dtype=torch.bfloat16).pin_memory()
        ta.ta_forward_host(host[0], host[1], host[2], out_h, B, H, Hkv, N, D, dims, True, stream=stream)
        outs.append((host, out_h))
        refs.append(gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16"))
    torch.cuda.synchronize()
    ta.ta_device_status()
    for (host, out_h), ref in zip(outs, refs):
        np.testing.assert_array_equal(out_h.float().numpy(), ref)


@pytest.mark.parametrize("B,H,Hkv,D,dims,causal,kw", [
    (1, 4, 2, 128, [8, 16, 32], True, {}),
    (2, 8, 2, 64, [16, 4, 4, 4], False, {}),
    (1, 16, 4, 128, [32, 32, 32], True, {}),
    (1, 4, 2, 128, [16, 8, 64], True, {"rope_base": 10000.0}),
    (1, 4, 2, 128, [4, 300, 16], True, {}),          # short, long, short segments
    (2, 8, 2, 128, [16, 4, 4, 4], False, {"fused": True}),   # the fused pass follows hop 0
])
def test_overlapped_hop_launches_give_identical_results(B, H, Hkv, D, dims, causal, kw):
    """A hop's kernel may start while the previous hop drains (it prefetches Q and K, then waits
    for that hop before it touches the value tensor).  Repeated runs must reproduce, bit for
    bit, the run whose launches are fully serialised."""
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 130)
    kw = dict(kw)
    base = 0 if kw.pop("fused", False) else ta.TA_FLAG_NO_HOP_FUSION
    if base == 0:
        assert "tc-fused" in ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, 0)
    ref = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", base | ta.TA_FLAG_NO_HOP_OVERLAP, **kw)
    for _ in range(10):
        got = gpu_forward(inp, B, H, Hkv, N, D, dims, causal, "bf16", base, **kw)
        np.testing.assert_array_equal(got, ref)


def test_concurrent_host_threads_and_streams():
    """Six host threads, each with its own stream and problem, call the library at the same time
    and repeatedly; every result must equal the one the same problem gives when run alone."""
    import threading

    import torch
    # (three of them need a scratch tensor of the same size, which each call takes for itself)
    cases = [(1, 4, 2, 128, [8, 16, 32], True), (2, 4, 4, 64, [16, 4, 4, 4], False),
             (1, 2, 1, 128, [2, 300], True), (1, 8, 2, 128, [32, 32], True),
             (1, 2, 1, 128, [300, 2], True), (1, 2, 2, 128, [2, 300], False)]
    work = []
    for i, (B, H, Hkv, D, dims, causal) in enumerate(cases):
        N = math.prod(dims)
        inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 140 + i)
        q, k, v = (to_device(inp, n, "bf16") for n in ("q", "k", "v"))
        ref = torch.empty_like(q)
        ta.ta_forward(q, k, v, ref, B, H, Hkv, N, D, dims, causal)
        work.append((q, k, v, ref, B, H, Hkv, N, D, dims, causal))
    torch.cuda.synchronize()
    errors = []

    def worker(w):
        q, k, v, ref, B, H, Hkv, N, D, dims, causal = w
        try:
            stream = torch.cuda.Stream()
            outs = [torch.empty_like(q) for _ in range(25)]
            for out in outs:
                ta.ta_forward(q, k, v, out, B, H, Hkv, N, D, dims, causal, stream=stream)
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


def test_forward_host_groups_of_heads_and_scratch():
    """Host-buffer entry point on a call large enough to be cut into groups of (batch, KV head)
    pairs that pipeline through upload, kernels and download, and on an fp32 problem whose hops
    need the library's scratch tensor; results must equal the device-resident runs."""
    import torch
    stream = torch.cuda.current_stream()
    # 2 x 8 KV heads x 4 query heads x 4096 tokens x 128 x 2 B = 64 MB of queries per batch entry
    B, H, Hkv, D, dims = 2, 32, 8, 128, [64, 64]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 145)
    host = [torch.from_numpy(inp[n + "_bits"].view(np.int16)).view(torch.bfloat16).pin_memory() for n in "qkv"]
    out_h = torch.empty((B, H, N, D), dtype=torch.bfloat16).pin_memory()
    for _ in range(2):
        out_h.fill_(float("nan"))
        ta.ta_forward_host(host[0], host[1], host[2], out_h, B, H, Hkv, N, D, dims, True, stream=stream)
        torch.cuda.synchronize()
        ta.ta_device_status()
        np.testing.assert_array_equal(out_h.float().numpy(), gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16"))
    B, H, Hkv, D, dims = 1, 2, 2, 64, [4, 4, 16]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "f32", 146)
    host = [torch.from_numpy(inp[n]).pin_memory() for n in "qkv"]
    out_h = torch.empty((B, H, N, D), dtype=torch.float32).pin_memory()
    ta.ta_forward_host(host[0], host[1], host[2], out_h, B, H, Hkv, N, D, dims, True, dtype=ta.TA_DTYPE_F32,
                       stream=stream)
    torch.cuda.synchronize()
    ta.ta_device_status()
    np.testing.assert_array_equal(out_h.numpy(), gpu_forward(inp, B, H, Hkv, N, D, dims, True, "f32"))
