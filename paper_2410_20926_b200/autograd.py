"""torch.autograd binding of the C-ABI library: ``tensorized_attention(q, k, v, dims, ...)``.

Marshalling only.  The forward is ``ta_forward_ex`` (with ``TA_FLAG_SAVE_HOPS`` when a gradient is
needed, so the hop inputs X_1..X_{m-1} are kept instead of recomputed), the backward is
``ta_backward_ex`` on those saved hops; every step runs in the library's CUDA kernels and there
is no fallback.  q: [B, H, N, D]; k, v: [B, H_kv, N, D]; contiguous CUDA tensors, all bfloat16
(tensor-core kernels) or all float32 (generic kernels, fp32 arithmetic throughout).
"""
from __future__ import annotations

import math

from . import api as ta


def _check(q, k, v, dims):
    import torch
    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise ValueError("tensorized_attention needs CUDA tensors (there is no CPU path)")
    if q.dim() != 4 or k.dim() != 4 or v.shape != k.shape:
        raise ValueError("expected q [B,H,N,D] and k, v [B,H_kv,N,D]")
    B, H, N, D = q.shape
    if k.shape[0] != B or k.shape[2] != N or k.shape[3] != D:
        raise ValueError("q and k, v disagree in batch, length or head dim")
    if math.prod(int(x) for x in dims) != N:
        raise ValueError("prod(dims) must equal the sequence length")
    if q.dtype not in (torch.bfloat16, torch.float32) or k.dtype != q.dtype or v.dtype != q.dtype:
        raise ValueError("q, k, v must all be bfloat16 or all float32")
    return B, H, k.shape[1], N, D


def _function():
    import torch

    class _TensorizedAttention(torch.autograd.Function):
        @staticmethod
        def forward(ctx, q, k, v, dims, causal, softmax_scale, rope_base, window, hop_masks, seq_lens):
            B, H, H_kv, N, D = _check(q, k, v, dims)
            q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
            dims = [int(x) for x in dims]
            need_grad = any(ctx.needs_input_grad[:3])
            dtype = ta.TA_DTYPE_BF16 if q.dtype == torch.bfloat16 else ta.TA_DTYPE_F32
            mode = ta.TA_WS_FORWARD_SAVE if need_grad else ta.TA_WS_FORWARD
            nbytes = ta.ta_workspace_bytes(B, H, H_kv, N, D, dims, dtype, mode)
            ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
            out = torch.empty_like(q)
            with torch.cuda.device(q.device):
                ta.ta_forward_ex(q, k, v, out, B, H, H_kv, N, D, dims, causal, dtype=dtype,
                                 softmax_scale=softmax_scale or 0.0, workspace=ws, workspace_bytes=nbytes,
                                 flags=ta.TA_FLAG_SAVE_HOPS if need_grad else 0, rope_base=rope_base or 0.0,
                                 window=window, hop_masks=hop_masks, seq_lens=seq_lens)
            if need_grad:
                # the saved hop inputs X_1..X_{m-1} are the tail of the workspace (after the scratch
                # tensor, if the plan has one)
                real_hops = sum(1 for n in dims if n > 1)
                save_bytes = max(real_hops - 1, 0) * q.numel() * q.element_size()
                ctx.save_for_backward(q, k, v)
                ctx.saved_ws, ctx.saved_off = ws, nbytes - save_bytes
                ctx.args = (B, H, H_kv, N, D, dims, causal, softmax_scale, rope_base, window, hop_masks, seq_lens)
            return out

        @staticmethod
        def backward(ctx, dout):
            q, k, v = ctx.saved_tensors
            B, H, H_kv, N, D, dims, causal, softmax_scale, rope_base, window, hop_masks, seq_lens = ctx.args
            dout = dout.contiguous()
            dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
            f32 = q.dtype == torch.float32
            dtype = ta.TA_DTYPE_F32 if f32 else ta.TA_DTYPE_BF16
            nbytes = ta.ta_workspace_bytes(B, H, H_kv, N, D, dims, dtype,
                                           ta.TA_WS_BACKWARD_F32_GRADS if f32 else ta.TA_WS_BACKWARD)
            ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
            real_hops = sum(1 for n in dims if n > 1)
            saved = ctx.saved_ws[ctx.saved_off:] if real_hops > 1 else None
            with torch.cuda.device(q.device):
                ta.ta_backward_ex(dout, q, k, v, dq, dk, dv, B, H, H_kv, N, D, dims, causal,
                                  dtype=dtype, grad_dtype=dtype, softmax_scale=softmax_scale or 0.0,
                                  saved_hops=saved, workspace=ws,
                                  workspace_bytes=nbytes, rope_base=rope_base or 0.0, window=window,
                                  hop_masks=hop_masks, seq_lens=seq_lens)
            return dq, dk, dv, None, None, None, None, None, None, None

    return _TensorizedAttention


_FN = None


def tensorized_attention(q, k, v, dims, causal=True, softmax_scale=None, rope_base=None, window=None,
                         hop_masks=None, seq_lens=None):
    """Algorithm 1 of the paper on the GPU, differentiable with respect to q, k, v.

    dims: the tensor shape n_1..n_m (prod = N).  rope_base: tensorized positional encoding
    applied inside the kernels (Section 3.2).  window / hop_masks: per-hop sparsity masks.
    seq_lens: int32 CUDA tensor [B] of valid lengths.  Returns out [B, H, N, D].
    """
    global _FN
    if _FN is None:
        _FN = _function()
    return _FN.apply(q, k, v, tuple(int(x) for x in dims), bool(causal), softmax_scale, rope_base, window,
                     hop_masks, seq_lens)
