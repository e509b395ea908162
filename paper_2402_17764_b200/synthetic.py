"""Seeded synthetic inputs shared by the CUDA path's tests, the oracle's tests
and the benchmark.

This module holds NONE of the method's arithmetic: it only draws latent
weights and activations with the shapes and value distributions of the
paper's workloads (LLaMA-shaped BitLinear layers, Section 2 "LLaMA-alike
Components"; model sizes of Section 3) and lists those shapes.  The trained
checkpoints of the paper are not available, so random-init latent weights
N(0, 0.02^2) and Gaussian activations with a few large "outlier" feature
channels stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

SIGMA_W = 0.02


def latent_weights(N: int, K: int, seed: int, device="cpu", sigma: float = SIGMA_W) -> torch.Tensor:
    """fp32 [N, K] ~ N(0, sigma^2), row-major (out x in, like nn.Linear.weight)."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    w = torch.randn((N, K), generator=g, device=device, dtype=torch.float32)
    return w.mul_(sigma)


def activations(M: int, K: int, seed: int, device="cpu", outlier_frac: float = 0.0,
                outlier_scale: float = 1.0) -> torch.Tensor:
    """bf16 [M, K]: N(0,1) in fp32, a fixed set of feature channels scaled up, cast to bf16 last."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) + 7919)
    x = torch.randn((M, K), generator=g, device=device, dtype=torch.float32)
    n_out = int(outlier_frac * K)
    if n_out > 0:
        perm = torch.randperm(K, generator=g, device=device)
        x[:, perm[:n_out]] *= outlier_scale
    return x.to(torch.bfloat16)


@dataclass(frozen=True)
class LayerShape:
    name: str
    N: int  # out features
    K: int  # in features


def decoder_layer_shapes(hidden: int, ffn: int, kv_dim: int | None = None) -> list[LayerShape]:
    """The seven BitLinear projections of one LLaMA-style decoder layer."""
    kv = hidden if kv_dim is None else kv_dim
    return [
        LayerShape("q", hidden, hidden),
        LayerShape("k", kv, hidden),
        LayerShape("v", kv, hidden),
        LayerShape("o", hidden, hidden),
        LayerShape("gate", ffn, hidden),
        LayerShape("up", ffn, hidden),
        LayerShape("down", hidden, ffn),
    ]


# The five workloads named by the benchmark definition.
CONFIGS = {
    "single": dict(layers=[LayerShape("single", 4096, 1536)], n_layers=1, M=[8],
                   outlier_frac=0.01, outlier_scale=20.0),
    "3b_decode": dict(layers=decoder_layer_shapes(3200, 8640), n_layers=26, M=[1],
                      outlier_frac=0.0, outlier_scale=1.0),
    "7b_batched": dict(layers=[LayerShape("attn", 4096, 4096), LayerShape("up", 11008, 4096),
                               LayerShape("down", 4096, 11008)], n_layers=1, M=[1, 4, 16, 64],
                       outlier_frac=0.005, outlier_scale=30.0),
    "13b_prefill": dict(layers=[LayerShape("up", 13824, 5120), LayerShape("down", 5120, 13824)],
                        n_layers=1, M=[512, 2048, 8192], outlier_frac=0.0, outlier_scale=1.0),
    "70b_decode": dict(layers=decoder_layer_shapes(8192, 28672, kv_dim=1024), n_layers=80, M=[1, 16],
                       outlier_frac=0.0, outlier_scale=1.0),
}


def packed_weight_bytes(N: int, K: int) -> int:
    """Algorithmic bytes of the 2-bit weights of one matrix (no padding counted)."""
    return N * K // 4
