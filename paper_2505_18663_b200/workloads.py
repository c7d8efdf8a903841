"""Seeded synthetic inputs shaped like the paper's video-DiT workloads.

This module holds NO arithmetic of the method (no rotation, no quantizer): it only draws
random tensors and lists layer shapes, so that the CUDA path and the CPU oracle can be fed
the same bits.  The real HunyuanVideo / Wan2.1 activations and weights are not available;
these tensors stand in for them with the layer shapes, token counts and outlier structure of
the benchmark configurations (heavy-tailed channels, a few outlier channels, per-token
magnitude spread).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import torch


@dataclass(frozen=True)
class Layer:
    K: int          # input channels
    N: int          # output channels
    rot_block: int  # Hadamard block B (divides K)
    bits: int       # activation bits of this layer (4 or 6)
    act: int = 0    # 1: tanh-GELU on the output
    bias: bool = False
    name: str = ""


@dataclass(frozen=True)
class Workload:
    name: str
    M: int                 # tokens
    layers: Tuple[Layer, ...]
    dist: str              # activation distribution key, see make_activations
    outlier_frac: float = 0.0
    outlier_gain: float = 1.0
    n_outliers: Optional[int] = None
    seed: int = 0
    chain: bool = False    # layers feed each other (FFN chain) instead of sharing the input recipe


def _rot_block(K: int) -> int:
    """Largest power of two <= 1024 that divides K (256 for 8960, 512 for 1536 / 13824, else 1024)."""
    b = 1024
    while K % b:
        b //= 2
    return b


def _mixed_bits(n_layers: int, frac_a6: float, seed: int) -> List[int]:
    """Seeded per-layer mask: round(frac * n) layers run at 6 bits, the rest at 4."""
    g = torch.Generator().manual_seed(seed)
    order = torch.randperm(n_layers, generator=g).tolist()
    n6 = int(round(frac_a6 * n_layers))
    bits = [4] * n_layers
    for i in order[:n6]:
        bits[i] = 6
    return bits


def _layers(shapes, bits):
    return tuple(Layer(K=k, N=n, rot_block=_rot_block(k), bits=b, name=f"{k}x{n}") for (k, n), b in zip(shapes, bits))


_HY_SHAPES = [(3072, 3072), (3072, 9216), (3072, 12288), (12288, 3072)]
_W13_SHAPES = [(1536, 1536), (1536, 4608), (1536, 8960), (8960, 1536)]
_W14_SHAPES = [(5120, 5120), (5120, 15360), (5120, 13824), (13824, 5120)]

WORKLOADS = {
    # single W4A4 linear, tiny
    "tiny": Workload("tiny", 256, _layers([(256, 256)], [4]), "normal", n_outliers=4, outlier_gain=20.0, seed=0),
    # Wan-1.3B-shaped W4A4 linears
    "wan1p3b": Workload("wan1p3b", 32760, _layers(_W13_SHAPES, [4] * 4), "normal", outlier_frac=0.005,
                        outlier_gain=30.0, seed=1),
    # HunyuanVideo-shaped linears, 25 % of the layers switched up to 6-bit activations
    "hunyuan": Workload("hunyuan", 65536, _layers(_HY_SHAPES, _mixed_bits(4, 0.25, 2)), "student_t4",
                        outlier_frac=0.01, outlier_gain=50.0, seed=2),
    # Wan-14B-shaped, all activations 6-bit, per-token magnitudes log-uniform in [0.1, 10]
    "wan14b": Workload("wan14b", 32760, _layers(_W14_SHAPES, [6] * 4), "normal_token_loguniform", seed=3),
    # DiT-block FFN chain at a 720p-length sequence
    "ffn_chain": Workload("ffn_chain", 118800,
                          (Layer(3072, 12288, 1024, 4, act=1, name="up+gelu"),
                           Layer(12288, 3072, 1024, 6, bias=True, name="down+bias")),
                          "normal", outlier_frac=0.01, outlier_gain=40.0, seed=4, chain=True),
}


def _gen(device, seed: int) -> torch.Generator:
    return torch.Generator(device=device).manual_seed(int(seed))


def make_activations(wl: Workload, K: int, M: Optional[int] = None, device="cpu", salt: int = 0) -> torch.Tensor:
    """bf16 [M, K] activations of workload `wl` for a layer with K input channels."""
    M = wl.M if M is None else M
    base = wl.seed * 1000003 + K * 7 + salt
    g = _gen(device, base)
    out = torch.empty(M, K, dtype=torch.bfloat16, device=device)
    # outlier channels are a property of the layer, not of the token chunk
    gc = torch.Generator().manual_seed(base + 1)
    n_out = wl.n_outliers if wl.n_outliers is not None else int(round(wl.outlier_frac * K))
    gain = torch.ones(K, dtype=torch.float32)
    if n_out > 0:
        gain[torch.randperm(K, generator=gc)[:n_out]] = wl.outlier_gain
    gain = gain.to(device)
    rows_per_chunk = max(1, (1 << 24) // K)
    for r0 in range(0, M, rows_per_chunk):
        r1 = min(M, r0 + rows_per_chunk)
        x = torch.randn(r1 - r0, K, generator=g, device=device, dtype=torch.float32)
        if wl.dist == "student_t4":
            chi = torch.zeros_like(x)
            for _ in range(4):
                chi += torch.randn(r1 - r0, K, generator=g, device=device, dtype=torch.float32) ** 2
            x = x / torch.sqrt(chi / 4.0)
        elif wl.dist == "normal_token_loguniform":
            u = torch.rand(r1 - r0, 1, generator=g, device=device, dtype=torch.float32)
            x = x * torch.exp(math.log(0.1) + u * (math.log(10.0) - math.log(0.1)))
        elif wl.dist != "normal":
            raise ValueError(wl.dist)
        out[r0:r1] = (x * gain).to(torch.bfloat16)
    return out


def make_weights(wl: Workload, layer: Layer, device="cpu") -> torch.Tensor:
    """bf16 [N, K] weights ~ N(0, 0.02)."""
    g = _gen(device, wl.seed * 7919 + layer.K * 31 + layer.N)
    return (torch.randn(layer.N, layer.K, generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)


def make_bias(wl: Workload, layer: Layer, device="cpu") -> Optional[torch.Tensor]:
    if not layer.bias:
        return None
    g = _gen(device, wl.seed * 104729 + layer.N)
    return (torch.randn(layer.N, generator=g, device=device, dtype=torch.float32) * 0.1).to(torch.bfloat16)


def make_weight_codes(layer: Layer, seed: int, device="cpu", symmetric: bool = True):
    """Random weights ALREADY in the 4-bit code format (codes 0..15, step, zero point), for
    runs that need a full-size packed matrix without an offline quantizer.  Codes are a sum of
    five uniform draws from {0..3}: bell-shaped over 0..15 like the codes of Gaussian weights."""
    g = _gen(device, seed)
    u = torch.zeros(layer.N, layer.K, dtype=torch.uint8, device=device)
    for _ in range(5):
        u += torch.randint(0, 4, (layer.N, layer.K), generator=g, device=device, dtype=torch.uint8)
    if symmetric:
        z = torch.full((layer.N,), 8, dtype=torch.int32, device=device)
    else:
        z = torch.randint(4, 12, (layer.N,), generator=g, device=device, dtype=torch.int32)
    delta = 0.0086 * (0.75 + 0.5 * torch.rand(layer.N, generator=g, device=device, dtype=torch.float32))
    return u, delta, z


def sample_rows(M: int, n: int, tile: int = 128, seed: int = 0) -> torch.Tensor:
    """Row indices for sampled parity checks at full size: the first tile, the last full tile,
    the ragged tail and seeded rows in between (sorted, unique)."""
    g = torch.Generator().manual_seed(seed)
    picks = list(range(0, min(tile, M), max(1, tile // 8)))
    last_full = (M // tile - 1) * tile if M >= 2 * tile else 0
    picks += list(range(last_full, min(last_full + tile, M), max(1, tile // 8)))
    picks += list(range((M // tile) * tile, M))[:tile]
    picks += [M - 1]
    extra = max(0, n - len(set(picks)))
    if extra:
        picks += torch.randint(0, M, (extra,), generator=g).tolist()
    return torch.tensor(sorted(set(p for p in picks if 0 <= p < M)), dtype=torch.int64)
