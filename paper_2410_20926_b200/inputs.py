"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds none of the method's arithmetic: it draws N(0,1) tensors with the shapes
of the paper's workloads (Llama-8B attention heads: H=32, H_kv=8, D=128; training length
32768 = 32x32x32, extrapolated to 131072 = 32x64x64; Section 4.1 and 4.4), rounds them to the
storage dtype and hands the same values to whoever asks.  The paper's own data (RedPajama,
Proof-pile) and weights are not available; only the shapes are taken from it.

Recipe: ``numpy.random.default_rng(seed)``, ``standard_normal(float32)`` drawn in the order
q, k, v, (dout); seed = 20241020 + config index; bf16 configs are rounded to bf16 with
round-to-nearest-even and returned as float32 values that are exactly representable in bf16
(plus the raw 16-bit patterns).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 20241020


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    H: int
    H_kv: int
    N: int
    D: int
    dims: tuple
    causal: bool
    dtype: str          # "bf16" or "f32"
    backward: bool = False
    index: int = 0

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


CONFIGS = {
    1: Config("c1_f32_16x16", 1, 2, 2, 256, 64, (16, 16), False, "f32", False, 1),
    2: Config("c2_bf16_64x64", 1, 8, 8, 4096, 128, (64, 64), True, "bf16", False, 2),
    3: Config("c3_llama8b_32k", 1, 32, 8, 32768, 128, (32, 32, 32), True, "bf16", False, 3),
    4: Config("c4_llama8b_128k", 1, 32, 8, 131072, 128, (32, 64, 64), True, "bf16", False, 4),
    5: Config("c5_llama8b_32k_train", 2, 32, 8, 32768, 128, (32, 32, 32), True, "bf16", True, 5),
}


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32 (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def draw(shape, rng: np.random.Generator, dtype: str):
    """One N(0,1) tensor in the storage dtype: (float32 values, raw bits or None)."""
    x = rng.standard_normal(shape, dtype=np.float32)
    if dtype == "bf16":
        bits = bf16_bits(x)
        return bf16_to_f32(bits), bits
    if dtype == "f32":
        return x, None
    raise ValueError(dtype)


def make_inputs(B, H, H_kv, N, D, dtype: str, seed: int, with_dout: bool = False) -> dict:
    """q:[B,H,N,D], k,v:[B,H_kv,N,D] (+dout:[B,H,N,D]); values float32, '<name>_bits' for bf16."""
    rng = np.random.default_rng(seed)
    out = {}
    names = [("q", (B, H, N, D)), ("k", (B, H_kv, N, D)), ("v", (B, H_kv, N, D))]
    if with_dout:
        names.append(("dout", (B, H, N, D)))
    for name, shape in names:
        val, bits = draw(shape, rng, dtype)
        out[name] = val
        if bits is not None:
            out[name + "_bits"] = bits
    return out


def make_config_inputs(cfg: Config) -> dict:
    return make_inputs(cfg.B, cfg.H, cfg.H_kv, cfg.N, cfg.D, cfg.dtype, cfg.seed, cfg.backward)


def make_device_inputs(B, H, H_kv, N, D, seed: int, device="cuda"):
    """bf16 q [B,H,N,D], k, v [B,H_kv,N,D] ~ N(0,1) drawn on the device, one batch entry at a
    time (for tensors too large to draw on the host).  Recipe: ``torch.Generator(device)`` seeded
    with `seed`; per batch entry ``randn`` of q, then k, then v in float32, rounded to bf16."""
    import torch
    gen = torch.Generator(device=device).manual_seed(seed)
    q = torch.empty(B, H, N, D, dtype=torch.bfloat16, device=device)
    k = torch.empty(B, H_kv, N, D, dtype=torch.bfloat16, device=device)
    v = torch.empty(B, H_kv, N, D, dtype=torch.bfloat16, device=device)
    for b in range(B):
        for t, heads in ((q, H), (k, H_kv), (v, H_kv)):
            for h0 in range(0, heads, 8):
                h1 = min(heads, h0 + 8)
                t[b, h0:h1] = torch.randn(h1 - h0, N, D, device=device, generator=gen).bfloat16()
    return q, k, v


def head_to_host(t, b: int, h: int) -> np.ndarray:
    """One head of a device tensor as a float64 array [1,1,N,D] (exact: bf16 -> fp64)."""
    return t[b, h].float().cpu().numpy().astype(np.float64)[None, None]
