"""Seeded synthetic inputs shaped like the workloads of the UE5M3 FP4 recipe.

This module serves both the oracle-side tests and the CUDA-side tests/benchmark and therefore
holds none of the method's arithmetic: it only draws random tensors.  Every generator takes a
seed and a device; the same bytes are then handed to the oracle (as numpy) and to the kernels.

Recipes (stand-ins for the training tensors the paper measured on; it reports heavy-tailed,
nearly dense upstream gradients, outlier-bearing activations and small-variance weights):
  * activations  X[M,K]  = N(0,1) * s_k,      s_k = 10^U(-1,1) per channel k
  * weights      W[N,K]  = N(0, 0.02^2)
  * gradients    dY[M,N] = 1e-3 * t_3/sqrt(3) (Student-t, nu = 3, variance-normalised)
  * outlier activations (small forward case): N(0,1), each entry x100 with probability 1e-3
  * bandwidth sweep rows: N(0,1) * r_row,     r_row = 10^U(-1,1) per row
  * drifting activation at step t: std0 * drift^t * N(0,1), each entry x1000 w.p. 1e-4
"""
from __future__ import annotations

import math

import numpy as np
import torch

# (name, in_features K, out_features N) of the eligible linears of one 8B-hybrid-shaped layer stack
LAYER_STACK = (
    ("attn_qkv", 4096, 6144),
    ("attn_out", 4096, 4096),
    ("mlp_up", 4096, 16384),
    ("mlp_down", 16384, 4096),
    ("mamba_in", 4096, 16384),
    ("mamba_out", 8192, 4096),
)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, g, device):
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def _rand(shape, g, device):
    return torch.rand(shape, generator=g, device=device, dtype=torch.float32)


def outlier_activation(rows, cols, seed, device="cpu", dtype=torch.float32, factor=100.0, prob=1e-3):
    g = _gen(seed, device)
    x = _randn((rows, cols), g, device)
    hit = _rand((rows, cols), g, device) < prob
    x = torch.where(hit, x * factor, x)
    return x.to(dtype).contiguous()


def channel_scaled_activation(rows, cols, seed, device="cpu", dtype=torch.bfloat16):
    g = _gen(seed, device)
    s = torch.pow(10.0, _rand((1, cols), g, device) * 2.0 - 1.0)
    x = _randn((rows, cols), g, device) * s
    return x.to(dtype).contiguous()


def row_scaled_tensor(rows, cols, seed, device="cpu", dtype=torch.bfloat16):
    g = _gen(seed, device)
    s = torch.pow(10.0, _rand((rows, 1), g, device) * 2.0 - 1.0)
    x = _randn((rows, cols), g, device)
    x.mul_(s)
    return x.to(dtype).contiguous()


def weight(rows, cols, seed, device="cpu", dtype=torch.bfloat16, std=0.02):
    g = _gen(seed, device)
    return (_randn((rows, cols), g, device) * std).to(dtype).contiguous()


def heavy_tailed_gradient(rows, cols, seed, device="cpu", dtype=torch.bfloat16, std=1e-3):
    g = _gen(seed, device)
    z = _randn((rows, cols), g, device)
    chi = torch.zeros((rows, cols), device=device, dtype=torch.float32)
    for _ in range(3):
        chi.addcmul_(*([_randn((rows, cols), g, device)] * 2))
    t = z / torch.sqrt(chi / 3.0)
    return (t * (std / math.sqrt(3.0))).to(dtype).contiguous()


def drifting_activation(rows, cols, step, device="cpu", dtype=torch.bfloat16, drift=1.05,
                        spike_prob=1e-4, spike_factor=1000.0, base_seed=1000):
    g = _gen(base_seed + step, device)
    x = _randn((rows, cols), g, device) * (drift ** step)
    hit = _rand((rows, cols), g, device) < spike_prob
    x = torch.where(hit, x * spike_factor, x)
    return x.to(dtype).contiguous()


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view for the oracle: float32 as is, bfloat16 as its uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy()
    if t.dtype == torch.float32:
        return t.numpy()
    raise TypeError(t.dtype)
