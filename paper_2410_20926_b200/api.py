"""ctypes binding of libta_b200.so: the same names and arguments as include/ta.h.

Argument marshalling only -- every step of the computation runs in the CUDA library.  Tensor
arguments may be torch tensors (``.data_ptr()``), numpy arrays (host variants) or raw integer
addresses.  Shapes are passed explicitly, exactly as in the C header.  A non-zero status is
raised as ``TaError`` unless ``check=False``.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libta_b200.so")

TA_OK = 0
TA_ERR_INVALID_ARG, TA_ERR_SHAPE, TA_ERR_UNSUPPORTED, TA_ERR_ALIGNMENT = -1, -2, -3, -4
TA_ERR_WORKSPACE, TA_ERR_ARCH, TA_ERR_CUDA, TA_ERR_TIMEOUT, TA_ERR_TOO_LARGE = -5, -6, -7, -8, -9
TA_DTYPE_BF16, TA_DTYPE_F32 = 0, 1
TA_FLAG_NO_TENSOR_CORE, TA_FLAG_NO_HOP_FUSION, TA_FLAG_SAVE_HOPS, TA_FLAG_NO_HOP_OVERLAP = 1, 2, 4, 8
TA_FLAG_PAIR_HOPS = 16
TA_FLAG_BF16_INTERMEDIATES = 32
TA_WS_FORWARD, TA_WS_FORWARD_SAVE, TA_WS_BACKWARD, TA_WS_BACKWARD_F32_GRADS = 0, 1, 2, 3

EXPORTS = ("ta_forward", "ta_forward_f32", "ta_forward_ex", "ta_backward", "ta_workspace_bytes",
           "ta_forward_host", "ta_plan_describe", "ta_device_status", "ta_launch_count",
           "ta_release", "ta_status_string", "ta_version", "ta_forward_static", "ta_backward_ex",
           "ta_last_cuda_error", "ta_selftest_wait_timeout")
TA_STATIC_SCRATCH_BYTES = 16 << 20


class TaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ta_status_string(status)
        if status == TA_ERR_CUDA:
            detail += f", cudaError {ta_last_cuda_error()}"
        super().__init__(f"{where} failed: {status} ({detail})")


class ta_params(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_size_t),
                ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("out", ctypes.c_void_p),
                ("B", ctypes.c_int), ("H", ctypes.c_int), ("H_kv", ctypes.c_int),
                ("N", ctypes.c_int), ("D", ctypes.c_int),
                ("dims", ctypes.POINTER(ctypes.c_int)), ("ndims", ctypes.c_int),
                ("causal", ctypes.c_int), ("dtype", ctypes.c_int),
                ("softmax_scale", ctypes.c_float),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("flags", ctypes.c_uint), ("hop_begin", ctypes.c_int), ("hop_end", ctypes.c_int),
                ("rope_base", ctypes.c_float),
                ("window", ctypes.POINTER(ctypes.c_int)),
                ("hop_masks", ctypes.POINTER(ctypes.c_void_p)),
                ("seq_lens", ctypes.c_void_p),
                ("masks_per_head", ctypes.c_int),
                ("stream", ctypes.c_void_p)]


class ta_bwd_params(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_size_t),
                ("dout", ctypes.c_void_p), ("q", ctypes.c_void_p), ("k", ctypes.c_void_p),
                ("v", ctypes.c_void_p),
                ("dq", ctypes.c_void_p), ("dk", ctypes.c_void_p), ("dv", ctypes.c_void_p),
                ("B", ctypes.c_int), ("H", ctypes.c_int), ("H_kv", ctypes.c_int),
                ("N", ctypes.c_int), ("D", ctypes.c_int),
                ("dims", ctypes.POINTER(ctypes.c_int)), ("ndims", ctypes.c_int),
                ("causal", ctypes.c_int), ("dtype", ctypes.c_int), ("grad_dtype", ctypes.c_int),
                ("softmax_scale", ctypes.c_float), ("rope_base", ctypes.c_float),
                ("window", ctypes.POINTER(ctypes.c_int)),
                ("hop_masks", ctypes.POINTER(ctypes.c_void_p)),
                ("seq_lens", ctypes.c_void_p),
                ("masks_per_head", ctypes.c_int),
                ("saved_hops", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("stream", ctypes.c_void_p)]


_lib = None


def load():
    """Load the CUDA library; fails loudly if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2410_20926_b200.csrc.build` "
            "(nvcc, sm_100a).  There is no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, ip = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int)
    fwd = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ip, ci, ci, vp]
    lib.ta_forward.argtypes = fwd
    lib.ta_forward_f32.argtypes = fwd
    lib.ta_forward_ex.argtypes = [ctypes.POINTER(ta_params)]
    lib.ta_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ip, ci, ci, vp,
                                ctypes.c_size_t, vp]
    lib.ta_backward_ex.argtypes = [ctypes.POINTER(ta_bwd_params)]
    lib.ta_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ip, ci, ci, ci]
    lib.ta_workspace_bytes.restype = ctypes.c_size_t
    lib.ta_forward_host.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ip, ci, ci, ci, vp]
    lib.ta_forward_static.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ip, ci, ci, ci, vp]
    lib.ta_plan_describe.argtypes = [ci, ci, ci, ci, ci, ip, ci, ci, ci, ctypes.c_uint,
                                     ctypes.c_char_p, ctypes.c_size_t]
    lib.ta_device_status.argtypes = []
    lib.ta_selftest_wait_timeout.argtypes = [ctypes.c_uint, ctypes.POINTER(ctypes.c_uint), vp]
    lib.ta_launch_count.argtypes = []
    lib.ta_launch_count.restype = ctypes.c_ulonglong
    lib.ta_release.argtypes = []
    lib.ta_status_string.argtypes = [ci]
    lib.ta_status_string.restype = ctypes.c_char_p
    lib.ta_last_cuda_error.argtypes = []
    lib.ta_last_cuda_error.restype = ctypes.c_int
    lib.ta_version.argtypes = []
    for name in EXPORTS:
        getattr(lib, name)          # every symbol of include/ta.h must be exported
    _lib = lib
    return lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(f"cannot take the address of {type(x)}")


def _dims(dims: Sequence[int]):
    arr = (ctypes.c_int * len(dims))(*[int(d) for d in dims])
    return arr, len(dims)


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _done(status: int, where: str, check: bool) -> int:
    if check and status != TA_OK:
        raise TaError(status, where)
    return status


def ta_status_string(status: int) -> str:
    return load().ta_status_string(int(status)).decode()


def ta_last_cuda_error() -> int:
    """cudaError_t behind the last TA_ERR_CUDA this thread got from a forward / backward call."""
    return int(load().ta_last_cuda_error())


def ta_version() -> int:
    return int(load().ta_version())


def ta_launch_count() -> int:
    return int(load().ta_launch_count())


def ta_device_status(check: bool = True) -> int:
    return _done(load().ta_device_status(), "ta_device_status", check)


def ta_selftest_wait_timeout(limit_us: int, stream=None, check: bool = True):
    """Returns (status, [expired, left_through_abort_flag, copy_landed, waited_ns])."""
    report = (ctypes.c_uint * 4)()
    rc = _done(load().ta_selftest_wait_timeout(int(limit_us), report, _stream(stream)),
               "ta_selftest_wait_timeout", check)
    return rc, list(report)


def ta_release() -> int:
    return int(load().ta_release())


def ta_forward(q, k, v, out, B, H, H_kv, N, D, dims, causal, stream=None, check=True) -> int:
    d, nd = _dims(dims)
    return _done(load().ta_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N, D, d, nd,
                                   int(bool(causal)), _stream(stream)), "ta_forward", check)


def ta_forward_f32(q, k, v, out, B, H, H_kv, N, D, dims, causal, stream=None, check=True) -> int:
    d, nd = _dims(dims)
    return _done(load().ta_forward_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N, D, d,
                                       nd, int(bool(causal)), _stream(stream)), "ta_forward_f32",
                 check)


def _window(window, nd):
    """Per-dimension sliding windows as a C int array (None stays NULL)."""
    if window is None:
        return None
    w = [int(x) for x in window]
    if len(w) != nd:
        raise ValueError("window needs one entry per dimension")
    return (ctypes.c_int * nd)(*w)


def _hop_masks(hop_masks, dims, H=None):
    """Per-dimension explicit masks M_i as a C array of host pointers (None stays NULL).

    `hop_masks` has one entry per dimension: None (no explicit mask for that hop) or an n_i x n_i
    array whose non-zero entries mark the visible (query position, key position) pairs -- or, for
    every masked dimension alike, an H x n_i x n_i array with one matrix per query head.  Returns
    (pointer array, buffers to keep alive until the call returns, masks_per_head flag).
    """
    if hop_masks is None:
        return None, None, 0
    import numpy as np
    dims = [int(x) for x in dims]
    if len(hop_masks) != len(dims):
        raise ValueError("hop_masks needs one entry per dimension")
    keep, arr = [], (ctypes.c_void_p * len(dims))()
    ranks = {np.asarray(m).ndim for m in hop_masks if m is not None}
    if len(ranks) > 1:
        raise ValueError("hop_masks: either every mask is n x n or every mask is H x n x n")
    per_head = int(ranks == {3})
    for i, (m, n) in enumerate(zip(hop_masks, dims)):
        if m is None:
            arr[i] = None
            continue
        m8 = np.ascontiguousarray((np.asarray(m) != 0).astype(np.uint8))
        want = (H, n, n) if per_head else (n, n)
        if m8.shape != want:
            raise ValueError(f"hop_masks[{i}] must have shape {want}")
        keep.append(m8)
        arr[i] = m8.ctypes.data
    return arr, keep, per_head


def ta_forward_ex(q, k, v, out, B, H, H_kv, N, D, dims, causal, dtype=TA_DTYPE_BF16,
                  softmax_scale=0.0, workspace=None, workspace_bytes=0, flags=0, hop_begin=0,
                  hop_end=0, rope_base=0.0, window=None, hop_masks=None, seq_lens=None, stream=None,
                  check=True) -> int:
    d, nd = _dims(dims)
    p = ta_params()
    p.struct_bytes = ctypes.sizeof(ta_params)
    p.q, p.k, p.v, p.out = _ptr(q), _ptr(k), _ptr(v), _ptr(out)
    p.B, p.H, p.H_kv, p.N, p.D = B, H, H_kv, N, D
    p.dims, p.ndims = d, nd
    p.causal, p.dtype, p.softmax_scale = int(bool(causal)), dtype, softmax_scale
    p.workspace, p.workspace_bytes = _ptr(workspace), workspace_bytes
    p.flags, p.hop_begin, p.hop_end = flags, hop_begin, hop_end
    p.rope_base = rope_base
    win = _window(window, nd)          # kept alive until the call returns
    if win is not None:
        p.window = win
    masks, _keep, p.masks_per_head = _hop_masks(hop_masks, dims, H)
    if masks is not None:
        p.hop_masks = masks
    p.seq_lens = _ptr(seq_lens)        # device int32 tensor [B] or None
    p.stream = _stream(stream)
    return _done(load().ta_forward_ex(ctypes.byref(p)), "ta_forward_ex", check)


def ta_backward(dout, q, k, v, out, dq, dk, dv, B, H, H_kv, N, D, dims, causal, workspace=None,
                workspace_bytes=0, stream=None, check=True) -> int:
    d, nd = _dims(dims)
    return _done(load().ta_backward(_ptr(dout), _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(dq),
                                    _ptr(dk), _ptr(dv), B, H, H_kv, N, D, d, nd,
                                    int(bool(causal)), _ptr(workspace), workspace_bytes,
                                    _stream(stream)), "ta_backward", check)


def ta_backward_ex(dout, q, k, v, dq, dk, dv, B, H, H_kv, N, D, dims, causal,
                   grad_dtype=TA_DTYPE_BF16, softmax_scale=0.0, saved_hops=None, workspace=None, dtype=TA_DTYPE_BF16,
                   workspace_bytes=0, rope_base=0.0, window=None, hop_masks=None, seq_lens=None,
                   stream=None, check=True) -> int:
    d, nd = _dims(dims)
    p = ta_bwd_params()
    p.struct_bytes = ctypes.sizeof(ta_bwd_params)
    p.dout, p.q, p.k, p.v = _ptr(dout), _ptr(q), _ptr(k), _ptr(v)
    p.dq, p.dk, p.dv = _ptr(dq), _ptr(dk), _ptr(dv)
    p.B, p.H, p.H_kv, p.N, p.D = B, H, H_kv, N, D
    p.dims, p.ndims, p.causal = d, nd, int(bool(causal))
    p.dtype, p.grad_dtype, p.softmax_scale = dtype, grad_dtype, softmax_scale
    p.rope_base = rope_base
    win = _window(window, nd)
    if win is not None:
        p.window = win
    masks, _keep, p.masks_per_head = _hop_masks(hop_masks, dims, H)
    if masks is not None:
        p.hop_masks = masks
    p.seq_lens = _ptr(seq_lens)
    p.saved_hops = _ptr(saved_hops)
    p.workspace, p.workspace_bytes = _ptr(workspace), workspace_bytes
    p.stream = _stream(stream)
    return _done(load().ta_backward_ex(ctypes.byref(p)), "ta_backward_ex", check)


def ta_workspace_bytes(B, H, H_kv, N, D, dims, dtype=TA_DTYPE_BF16, mode=TA_WS_FORWARD) -> int:
    d, nd = _dims(dims)
    return int(load().ta_workspace_bytes(B, H, H_kv, N, D, d, nd, dtype, mode))


def ta_forward_host(q_host, k_host, v_host, out_host, B, H, H_kv, N, D, dims, causal,
                    dtype=TA_DTYPE_BF16, stream=None, check=True) -> int:
    d, nd = _dims(dims)
    return _done(load().ta_forward_host(_ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(out_host),
                                        B, H, H_kv, N, D, d, nd, int(bool(causal)), dtype,
                                        _stream(stream)), "ta_forward_host", check)


def ta_forward_static(q, k, v, out, B, H, H_kv, N, D, dims, causal, dtype=TA_DTYPE_BF16,
                      stream=None, check=True) -> int:
    """Forward pass that allocates no device memory (scratch is a fixed array inside the
    library, TA_STATIC_SCRATCH_BYTES); see include/ta.h for who needs this and its limits."""
    d, nd = _dims(dims)
    return _done(load().ta_forward_static(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N, D,
                                          d, nd, int(bool(causal)), dtype, _stream(stream)),
                 "ta_forward_static", check)


def ta_plan_describe(B, H, H_kv, N, D, dims, causal, dtype=TA_DTYPE_BF16, flags=0,
                     check=True) -> str:
    d, nd = _dims(dims)
    buf = ctypes.create_string_buffer(4096)
    _done(load().ta_plan_describe(B, H, H_kv, N, D, d, nd, int(bool(causal)), dtype, flags, buf,
                                  len(buf)), "ta_plan_describe", check)
    return buf.value.decode()
