"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests.

This module holds none of the method's arithmetic: it only draws i.i.d. normal
values from a seeded CPU generator, rounds them to the 16-bit storage type and
describes the benchmark configurations.  Both the oracle and the CUDA path read
the SAME rounded 16-bit values.

The paper benchmarks synthetic tensors at FlashAttention's shapes (Section 4.1:
sequence 512..16k, 16k tokens per batch, hidden size 2048, head dim 64/128, with
and without the causal mask); the five configurations below are the synthetic
stand-ins used here.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

DTYPE_FP16 = 0
DTYPE_BF16 = 1
DTYPE_FP8_E4M3 = 2   # 8-bit inputs (stored as uint8 bit patterns), bf16 output

BASE_SEED = 20250612


@dataclass(frozen=True)
class AttnConfig:
    name: str
    index: int          # 1-based configuration number, enters the seed
    dtype: int          # DTYPE_FP16 / DTYPE_BF16
    causal: bool
    B: int
    H: int
    Sq: int
    Sk: int
    D: int
    sigma: float = 1.0  # standard deviation of Q, K, V entries before rounding

    @property
    def scale(self) -> float:
        # The value handed to the library is an fp32; keep exactly that number.
        return float(np.float32(1.0) / np.sqrt(np.float32(self.D)))

    @property
    def flops(self) -> float:
        f = 4.0 * self.B * self.H * self.Sq * self.Sk * self.D
        return f / 2 if self.causal else f

    @property
    def min_hbm_bytes(self) -> int:
        e = 2
        return (self.B * self.H * (2 * self.Sq * self.D * e + 2 * self.Sk * self.D * e)
                + 4 * self.B * self.H * self.Sq)

    @property
    def workload(self) -> str:
        return "%s: MHA fwd %s %s B=%d H=%d Sq=Sk=%d D=%d" % (
            self.name, "causal" if self.causal else "non-causal",
            "bf16" if self.dtype == DTYPE_BF16 else "fp16", self.B, self.H, self.Sq, self.D)


CONFIGS = {
    "C1": AttnConfig("C1", 1, DTYPE_FP16, False, 1, 2, 128, 128, 64),
    "C2": AttnConfig("C2", 2, DTYPE_FP16, False, 8, 16, 1024, 1024, 64),
    "C3": AttnConfig("C3", 3, DTYPE_BF16, True, 4, 32, 2048, 2048, 128),
    "C4": AttnConfig("C4", 4, DTYPE_FP16, False, 2, 16, 4096, 4096, 256, 0.5),
    "C5": AttnConfig("C5", 5, DTYPE_BF16, True, 1, 32, 16384, 16384, 128),
}


def torch_dtype(dtype: int) -> torch.dtype:
    return torch.float16 if dtype == DTYPE_FP16 else torch.bfloat16


def randn16(shape, seed: int, dtype: int, sigma: float = 1.0) -> torch.Tensor:
    """sigma * N(0,1) drawn in fp32 on the CPU from `seed`, rounded (RN-even) to the 16-bit type."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    x = torch.randn(tuple(shape), generator=g, dtype=torch.float32)
    if sigma != 1.0:
        x = x * sigma
    return x.to(torch_dtype(dtype)).contiguous()


def make_qkv(B, H, Sq, Sk, D, dtype, seed, sigma=1.0):
    """Q [B,H,Sq,D], K, V [B,H,Sk,D] as 16-bit CPU tensors; seeds seed+0/1/2."""
    q = randn16((B, H, Sq, D), seed + 0, dtype, sigma)
    k = randn16((B, H, Sk, D), seed + 1, dtype, sigma)
    v = randn16((B, H, Sk, D), seed + 2, dtype, sigma)
    return q, k, v


def randn8(shape, seed: int, sigma: float = 1.0, factor: float = 1.0) -> torch.Tensor:
    """E4M3 bit patterns (uint8) of sigma * N(0,1) / factor, drawn in fp32 on the CPU from `seed`,
    clamped to the format's finite range (+-448) and rounded RN-even: the stored tensor whose
    dequantised value is factor * e4m3(bits)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    x = torch.randn(tuple(shape), generator=g, dtype=torch.float32) * (sigma / factor)
    return x.clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()


def make_qkv_fp8(B, H, Hkv, Sq, Sk, D, seed, sigma=1.0, factors=(1.0, 1.0, 1.0)):
    """Q [B,H,Sq,D], K, V [B,Hkv,Sk,D] as uint8 E4M3 bit patterns; seeds seed+0/1/2; one
    dequantisation factor per tensor."""
    q = randn8((B, H, Sq, D), seed + 0, sigma, factors[0])
    k = randn8((B, Hkv, Sk, D), seed + 1, sigma, factors[1])
    v = randn8((B, Hkv, Sk, D), seed + 2, sigma, factors[2])
    return q, k, v


def make_config_inputs(cfg: AttnConfig):
    return make_qkv(cfg.B, cfg.H, cfg.Sq, cfg.Sk, cfg.D, cfg.dtype,
                    BASE_SEED + 1000 * cfg.index, cfg.sigma)


def bits(t: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of a CPU fp16/bf16 tensor as a uint16 numpy array."""
    assert t.dtype in (torch.float16, torch.bfloat16) and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def sample_rows(cfg_rows: int, Sq: int, n_random: int, seed: int) -> np.ndarray:
    """A deterministic row subset of a [B*H*Sq] row space: the first and last 4 rows of the
    first and last head, every tile edge near 128-multiples of the first head, and n_random
    uniformly drawn rows."""
    rng = np.random.default_rng(seed)
    picks = set()
    heads = cfg_rows // Sq
    for bh in (0, heads - 1):
        base = bh * Sq
        for i in list(range(min(4, Sq))) + list(range(max(0, Sq - 4), Sq)):
            picks.add(base + i)
        for edge in range(128, Sq, max(128, (Sq // 8) // 128 * 128)):
            picks.add(base + edge - 1)
            picks.add(base + edge)
    picks.update(int(r) for r in rng.integers(0, cfg_rows, size=n_random))
    return np.array(sorted(picks), dtype=np.int64)
