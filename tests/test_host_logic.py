"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, validates
arguments before touching CUDA, and plans hops as documented."""
import ctypes
import os
import re

import pytest

import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ta.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ta_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(api.LIB_PATH)
    names = declared_symbols()
    assert "ta_forward" in names and "ta_backward" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(api.EXPORTS) == sorted(n for n in names)


def test_version_and_status_strings():
    assert ta.ta_version() >= 100
    assert ta.ta_status_string(0) == "ok"
    for code in range(-9, 0):
        assert ta.ta_status_string(code) not in ("ok", "unknown status")


ARGS = dict(B=1, H=4, H_kv=2, N=64, D=64)


def fwd(dims, q=16, k=16, v=16, out=16, **kw):
    a = dict(ARGS, **kw)
    return ta.ta_forward(q, k, v, out, a["B"], a["H"], a["H_kv"], a["N"], a["D"], dims, True,
                         stream=0, check=False)


def test_argument_validation_happens_before_cuda():
    assert fwd([8, 8], q=0) == ta.TA_ERR_INVALID_ARG
    assert fwd([8, 8], out=0) == ta.TA_ERR_INVALID_ARG
    assert fwd([8, 8], B=0) == ta.TA_ERR_INVALID_ARG
    assert fwd([8, 0]) == ta.TA_ERR_INVALID_ARG
    assert fwd([2] * 9, N=512) == ta.TA_ERR_INVALID_ARG          # more than TA_MAX_DIMS
    assert fwd([8, 7]) == ta.TA_ERR_SHAPE
    assert fwd([8, 8], H=3) == ta.TA_ERR_SHAPE
    assert fwd([8, 8], D=512) == ta.TA_ERR_UNSUPPORTED
    assert fwd([8, 8], q=8) == ta.TA_ERR_ALIGNMENT
    with pytest.raises(ta.TaError):
        ta.ta_forward(16, 16, 16, 16, 1, 4, 2, 64, 64, [8, 7], True, stream=0)


def test_forward_ex_rejects_bad_struct_and_workspace():
    lib = api.load()
    p = api.ta_params()
    p.struct_bytes = 8
    assert lib.ta_forward_ex(ctypes.byref(p)) == ta.TA_ERR_INVALID_ARG
    # fp32 with two hops needs a second value buffer: a too-small workspace is an error
    rc = ta.ta_forward_ex(16, 16, 16, 16, 1, 2, 2, 256, 64, [16, 16], False, dtype=ta.TA_DTYPE_F32,
                          workspace=256, workspace_bytes=16, stream=0, check=False)
    assert rc == ta.TA_ERR_WORKSPACE
    rc = ta.ta_forward_ex(16, 16, 16, 16, 1, 2, 2, 256, 64, [16, 16], False,
                          flags=ta.TA_FLAG_SAVE_HOPS, stream=0, check=False)
    assert rc == ta.TA_ERR_WORKSPACE
    rc = ta.ta_forward_ex(16, 16, 16, 16, 1, 2, 2, 256, 64, [16, 16], False, flags=1 << 9,
                          stream=0, check=False)
    assert rc == ta.TA_ERR_UNSUPPORTED


def test_workspace_bytes():
    e = 1 * 2 * 256 * 64
    assert ta.ta_workspace_bytes(1, 2, 2, 256, 64, [16, 16], ta.TA_DTYPE_F32) == 4 * e
    # two adjacent tensor-core hops run as one pair launch: a few bytes of completion counters
    assert ta.ta_workspace_bytes(1, 2, 2, 256, 64, [16, 16], ta.TA_DTYPE_BF16) == 256
    assert ta.ta_workspace_bytes(1, 2, 2, 256, 64, [16], ta.TA_DTYPE_BF16) == 0
    assert ta.ta_workspace_bytes(1, 2, 2, 256, 64, [16, 16], ta.TA_DTYPE_BF16,
                                 ta.TA_WS_FORWARD_SAVE) == 2 * e
    assert ta.ta_workspace_bytes(1, 2, 2, 256, 64, [16, 15], ta.TA_DTYPE_BF16) == 0


def parse_plan(text):
    lines = text.strip().splitlines()
    head = dict(kv.split("=") for kv in lines[0].split())
    hops = [dict(kv.split("=") for kv in ln.split()) for ln in lines[1:]]
    return head, hops


def test_plan_llama_128k():
    head, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 131072, 128, [32, 64, 64], True))
    assert head["hops"] == "3" and head["scratch_bytes"] == "0"
    assert [h["path"] for h in hops] == ["tc"] * 3
    assert [(h["n"], h["stride"], h["outer"]) for h in hops] == \
        [("32", "4096", "1"), ("64", "64", "32"), ("64", "1", "2048")]
    assert [(h["ci"], h["co"], h["rows"]) for h in hops] == \
        [("4", "1", "128"), ("2", "1", "128"), ("1", "2", "128")]
    assert [(h["src"], h["dst"]) for h in hops] == [("v", "out"), ("out", "out"), ("out", "out")]


def test_plan_intermediates_and_pair_launches():
    dims = [32, 32, 32]
    # between tensor-core hops the value tensor is fp16 (same bytes, finer rounding); the last hop writes bf16
    _, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 32768, 128, dims, True))
    assert [h.get("dst_type") for h in hops] == ["f16", "f16", None]
    assert all("pair" not in h for h in hops)
    _, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 32768, 128, dims, True, flags=ta.TA_FLAG_BF16_INTERMEDIATES))
    assert [h.get("dst_type") for h in hops] == [None, None, None]
    # the forward that saves the hop inputs for the backward keeps them bf16
    _, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 32768, 128, dims, True, flags=ta.TA_FLAG_SAVE_HOPS))
    assert [h.get("dst_type") for h in hops] == [None, None, None]
    assert [h["dst"] for h in hops] == ["save", "save", "out"]
    # a hop next to a long-segment or generic hop stays bf16
    _, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 16 * 16 * 200, 64, [16, 16, 200], True))
    assert [h.get("dst_type") for h in hops] == ["f16", None, None]
    # pair launches: opt-in, the last two hops of the Llama shapes; counters in the workspace
    _, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 32768, 128, dims, True, flags=ta.TA_FLAG_PAIR_HOPS))
    assert [h.get("pair") for h in hops] == [None, "first", "second"]
    _, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 131072, 128, [32, 64, 64], True, flags=ta.TA_FLAG_PAIR_HOPS))
    assert [h.get("pair") for h in hops] == [None, "first", "second"]
    _, hops = parse_plan(ta.ta_plan_describe(1, 32, 8, 32768, 128, dims, True,
                                             flags=ta.TA_FLAG_PAIR_HOPS | ta.TA_FLAG_NO_HOP_FUSION))
    assert all("pair" not in h for h in hops)
    assert ta.ta_workspace_bytes(1, 32, 8, 32768, 128, dims, ta.TA_DTYPE_BF16) == 8 * 32 * 4 + 256


def test_plan_skips_unit_dims_and_routes_generic_hops():
    _, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 256, 64, [16, 1, 16], False))
    assert [h["hop"] for h in hops] == ["0", "2"]
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 256, 64, [1, 1, 1, 256], False))
    assert [h["path"] for h in hops] == ["tc-long"]                    # n > 128: key-block loop
    # a bf16 head dim the tensor-core kernels lack runs on zero-padded copies, unless told otherwise
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 256, 96, [1, 1, 1, 256], False))
    assert [h["path"] for h in hops] == ["tc-long"] and head["padded_head_dim"] == "128"
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 256, 40, [16, 16], False))
    assert [h["path"] for h in hops] == ["tc", "tc"] and head["padded_head_dim"] == "64"
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 256, 96, [1, 1, 1, 256], False, flags=ta.TA_FLAG_NO_TENSOR_CORE))
    assert [h["path"] for h in hops] == ["simt"] and "padded_head_dim" not in head
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 256, 96, [1, 1, 1, 256], False, dtype=ta.TA_DTYPE_F32))
    assert [h["path"] for h in hops] == ["simt"] and "padded_head_dim" not in head
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 16384, 64, [4, 4096], False))
    assert [(h["path"], h["src"], h["dst"]) for h in hops] == \
        [("tc", "v", "scratch"), ("tc-long", "scratch", "out")]        # the long hop is not in place
    assert int(head["scratch_bytes"]) == 2 * 16384 * 64 * 2
    head, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 27, 64, [3, 3, 3], True,
                                                dtype=ta.TA_DTYPE_F32))
    assert [(h["src"], h["dst"]) for h in hops] == [("v", "out"), ("out", "scratch"),
                                                    ("scratch", "out")]
    head, _ = parse_plan(ta.ta_plan_describe(1, 2, 2, 1, 64, [1], True))
    assert head["hops"] == "0"


def test_plan_tiles_never_straddle_heads():
    # n = 12: 10 segments would fit a 128-row tile, but outer = 8 is not a multiple of 10
    _, hops = parse_plan(ta.ta_plan_describe(1, 2, 2, 96, 64, [2, 4, 12], False,
                                             flags=ta.TA_FLAG_NO_HOP_FUSION))
    last = hops[-1]
    assert int(last["co"]) == 8 and int(last["rows"]) == 96
    for h in hops:
        assert int(h["rows"]) <= 128 and int(h["rows"]) == int(h["ci"]) * int(h["co"]) * int(h["n"])
        assert int(h["outer"]) % int(h["co"]) == 0


def test_backward_validation_and_workspace_sizes():
    e = 1 * 4 * 512 * 128                      # elements of a q-shaped tensor
    kv = e // 2
    need = ta.ta_workspace_bytes(1, 4, 2, 512, 128, [8, 64], ta.TA_DTYPE_BF16, ta.TA_WS_BACKWARD)
    assert need == 2 * e + 2 * e + 4 * e + 2 * 4 * kv     # X_1, G, dq fp32, dk + dv fp32
    need32 = ta.ta_workspace_bytes(1, 4, 2, 512, 128, [8, 64], ta.TA_DTYPE_BF16,
                                   ta.TA_WS_BACKWARD_F32_GRADS)
    assert need32 == 2 * e + 2 * e
    rc = ta.ta_backward(16, 16, 16, 16, None, 16, 16, 16, 1, 4, 2, 512, 128, [8, 63], True,
                        workspace=256, workspace_bytes=1 << 30, stream=0, check=False)
    assert rc == ta.TA_ERR_SHAPE
    rc = ta.ta_backward(0, 16, 16, 16, None, 16, 16, 16, 1, 4, 2, 512, 128, [8, 64], True,
                        workspace=256, workspace_bytes=1 << 30, stream=0, check=False)
    assert rc == ta.TA_ERR_INVALID_ARG
    rc = ta.ta_backward(16, 16, 16, 16, None, 16, 16, 16, 1, 4, 2, 512, 128, [8, 64], True,
                        workspace=256, workspace_bytes=1024, stream=0, check=False)
    assert rc == ta.TA_ERR_WORKSPACE
    rc = ta.ta_backward(16, 16, 16, 16, None, 16, 16, 16, 1, 4, 2, 512, 320, [8, 64], True,
                        workspace=256, workspace_bytes=1 << 30, stream=0, check=False)
    assert rc == ta.TA_ERR_UNSUPPORTED          # head dims above 256 have no backward
    # hops on the generic backward kernels (segments > 128, other head dims) add a second G
    # buffer (three or more hops) and two floats per query row
    e96 = 4 * 512 * 96
    need96 = ta.ta_workspace_bytes(1, 4, 2, 512, 96, [8, 64], ta.TA_DTYPE_BF16, ta.TA_WS_BACKWARD_F32_GRADS)
    assert need96 == 2 * e96 + 2 * e96 + 4 * 512 * 8
    need3 = ta.ta_workspace_bytes(1, 4, 2, 512, 128, [2, 2, 128], ta.TA_DTYPE_BF16, ta.TA_WS_BACKWARD_F32_GRADS)
    assert need3 == 2 * 2 * e + 2 * e
    need3g = ta.ta_workspace_bytes(1, 4, 2, 512, 128, [2, 1, 256], ta.TA_DTYPE_BF16, ta.TA_WS_BACKWARD_F32_GRADS)
    assert need3g == 2 * e + 2 * e + 4 * 512 * 8      # two hops: one G buffer, statistics
    need4g = ta.ta_workspace_bytes(1, 4, 2, 1024, 128, [2, 2, 256], ta.TA_DTYPE_BF16, ta.TA_WS_BACKWARD_F32_GRADS)
    assert need4g == 2 * 2 * (2 * e) + 2 * (2 * e) + 2 * (2 * e) + 4 * 1024 * 8


def test_plan_fuses_trailing_dimensions_that_fit_a_tile():
    text = ta.ta_plan_describe(1, 12, 12, 512, 64, [8, 8, 8], False, ta.TA_DTYPE_BF16, 0)
    assert "hops=2" in text.splitlines()[0]
    assert "path=tc-fused hops=2 block=64 blocks_per_tile=2" in text and "sub=8x8,8x1" in text
    text = ta.ta_plan_describe(1, 12, 12, 1024, 64, [16, 4, 4, 4], False, ta.TA_DTYPE_BF16, 0)
    assert "path=tc-fused hops=3 block=64" in text and "sub=4x16,4x4,4x1" in text
    text = ta.ta_plan_describe(1, 4, 4, 128, 128, [8, 16], True, ta.TA_DTYPE_BF16, 0)
    assert text.splitlines()[0].startswith("hops=1") and "src=v dst=out" in text
    # not when the block exceeds a tile, hops are kept apart on request, or a hop is generic
    assert "tc-fused" not in ta.ta_plan_describe(1, 4, 4, 512, 64, [32, 16], True, ta.TA_DTYPE_BF16, 0)
    assert "tc-fused" not in ta.ta_plan_describe(1, 4, 4, 512, 64, [8, 8, 8], True, ta.TA_DTYPE_BF16,
                                                 ta.TA_FLAG_NO_HOP_FUSION)
    assert "tc-fused" not in ta.ta_plan_describe(1, 4, 4, 512, 64, [8, 8, 8], True, ta.TA_DTYPE_F32, 0)


def test_autograd_binding_refuses_cpu_tensors_and_bad_shapes():
    """The torch.autograd binding has no CPU path: it must say so before any library call."""
    import torch
    q = torch.zeros(1, 2, 16, 64, dtype=torch.bfloat16)
    with pytest.raises(ValueError, match="CUDA"):
        ta.tensorized_attention(q, q, q, [4, 4])
