"""Seeded synthetic inputs shared by the tests, the oracle-side checks and the benchmark.

This module holds no RaZeR arithmetic: it only draws random tensors with the shapes
and value distributions of the workloads (LLM-shaped layers: heavy-tailed weights with
a few outliers, Gaussian activations with a few outlier channels) and, for kernel
timing, random code/scale bytes.  Everything is drawn on the CPU from a seeded
torch.Generator so both the CUDA path and the CPU oracle see identical inputs.
"""
from __future__ import annotations

import math

import torch


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def student_t_weights(N: int, K: int, seed: int, outlier_frac: float = 0.0,
                      outlier_scale: float = 10.0, scale: float = 0.02,
                      nu: int = 5, rows_per_chunk: int = 2048) -> torch.Tensor:
    """fp32 [N, K] weights: scale * Student-t(nu) (a normal over the root of a mean of
    nu squared normals); a Bernoulli(outlier_frac) mask multiplies entries by
    outlier_scale."""
    g = _gen(seed)
    out = torch.empty((N, K), dtype=torch.float32)
    for r0 in range(0, N, rows_per_chunk):
        r1 = min(N, r0 + rows_per_chunk)
        z = torch.randn((r1 - r0, K), generator=g, dtype=torch.float32)
        chi = torch.zeros((r1 - r0, K), dtype=torch.float32)
        for _ in range(nu):
            n = torch.randn((r1 - r0, K), generator=g, dtype=torch.float32)
            chi += n * n
        w = scale * z / torch.sqrt(chi / nu)
        if outlier_frac > 0:
            m = torch.rand((r1 - r0, K), generator=g) < outlier_frac
            w = torch.where(m, w * outlier_scale, w)
        out[r0:r1] = w
    return out


def activations(M: int, K: int, seed: int, outlier_channel_frac: float = 0.0,
                outlier_scale: float = 20.0) -> torch.Tensor:
    """bf16 [M, K] activations N(0,1); the first ceil(frac*K) channels of a seeded
    permutation of K are multiplied by outlier_scale."""
    g = _gen(seed + 7919)
    x = torch.randn((M, K), generator=g, dtype=torch.float32)
    if outlier_channel_frac > 0:
        perm = torch.randperm(K, generator=g)
        n = int(math.ceil(outlier_channel_frac * K))
        x[:, perm[:n]] *= outlier_scale
    return x.to(torch.bfloat16)


def random_codes(N: int, K: int, seed: int, meta_bits: int = 2, scale_lo: int = 24,
                 scale_hi: int = 56, zero_block_frac: float = 0.0):
    """Random quantized tensor for kernel tests and timing: every FP4 code (both zero
    codes included) uniformly, scale codes uniform in [scale_lo, scale_hi), metadata
    uniform.  Returns (codes uint8 [N, K/2], scale bytes uint8 [N, K/16])."""
    g = _gen(seed + 104729)
    codes = torch.randint(0, 256, (N, K // 2), generator=g, dtype=torch.uint8)
    sc = torch.randint(scale_lo, scale_hi, (N, K // 16), generator=g, dtype=torch.int32)
    meta = torch.randint(0, 1 << meta_bits, (N, K // 16), generator=g, dtype=torch.int32)
    sb = (meta << (8 - meta_bits)) | sc
    if zero_block_frac > 0:
        z = torch.rand((N, K // 16), generator=g) < zero_block_frac
        sb = torch.where(z, torch.zeros_like(sb), sb)
    return codes, sb.to(torch.uint8)


def bf16_to_bits(t: torch.Tensor):
    """torch bf16 tensor -> numpy uint16 bit patterns."""
    return t.contiguous().view(torch.int16).numpy().view("uint16")


def bits_to_bf16(a) -> torch.Tensor:
    """numpy uint16 bit patterns -> torch bf16 tensor."""
    import numpy as np
    return torch.from_numpy(np.ascontiguousarray(a).view("int16")).view(torch.bfloat16)
