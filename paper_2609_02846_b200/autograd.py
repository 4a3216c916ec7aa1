"""A linear layer whose three GEMMs run through the UE5M3-FP4 library, as a torch.autograd.Function.

Nothing is computed here: forward and backward only call `quantize`, `gemm` and `sample_amax` of the C ABI in
the order the recipe prescribes (X and W rounded to nearest even, the upstream gradient rounded stochastically
once per backward GEMM, one sample-and-hold tensor reference per quantized operand).  With a process group the
freshly sampled maxima are MAX-all-reduced on refresh steps, so that all data-parallel ranks scale by the same
reference; this is the only exchange the path has, one float per operand every `interval` steps.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B


def reduce_amax_(amax: torch.Tensor, group=None) -> torch.Tensor:
    """In-place MAX all-reduce of a sampled tensor maximum over a process group (no-op without one)."""
    if group is not None and torch.distributed.is_initialized() and torch.distributed.get_world_size(group) > 1:
        torch.distributed.all_reduce(amax, op=torch.distributed.ReduceOp.MAX, group=group)
    return amax


class OperandScale:
    """Sample-and-hold reference of one quantized operand, optionally agreed across ranks on refresh steps."""

    def __init__(self, interval: int = 50, group=None):
        self.cache = B.AmaxCache(interval)
        self.group = group

    def get(self, x: torch.Tensor, step: int) -> torch.Tensor:
        refresh = self.cache.refreshes_at(step)
        held = self.cache.get(x, step)
        if refresh:
            reduce_amax_(held, self.group)
        return held


_layer_counter = 0            # layers built so far in this process: the default stream id of a new layer


def sr_stream_seed(layer_seed: int, rank: int, step: int) -> int:
    """Base seed of one backward pass.  Eq. "sr" wants independent draws: two layers of the same shape, two
    data-parallel ranks and two steps must not share a draw stream (the draw depends only on the seed and the element
    index), otherwise their rounding errors are correlated and do not average out in the gradient all-reduce.
    The three fields sit in disjoint bit ranges (step: 24 bits, rank: 14 bits, layer: 24 bits) of a 62-bit value,
    since `linear_backward` uses 4 * seed and 4 * seed + 1 for its two quantizations."""
    return ((int(layer_seed) & 0xFFFFFF) << 38) | ((int(rank) & 0x3FFF) << 24) | (int(step) & 0xFFFFFF)


def _group_rank(group) -> int:
    if group is not None and torch.distributed.is_initialized():
        return torch.distributed.get_rank(group)
    return 0


def _check_dims(M: int, K: int, N: int, multiple: int = 128) -> None:
    """Every dimension is an output dimension of one GEMM and the contraction of another: multiples of 128 for
    ue5m3_gemm, of 256 under the output model (ue5m3_gemm_probe_matched)."""
    for name, v in (("tokens", M), ("in_features", K), ("out_features", N)):
        if v % multiple:
            raise ValueError(f"{name} = {v}: the three GEMMs of this linear need every dimension to be a multiple of {multiple}")


class _Ue5m3LinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, w, layer, step):
        M, K = x.shape
        N = w.shape[0]
        _check_dims(M, K, N, 128 if layer.grid_denominator is None else 256)
        ax = layer.scale_x.get(x, step)
        aw = layer.scale_w.get(w, step)
        y, _, qw = B.linear_forward(x, w, ax, aw, layer.target_T, x.dtype, grid_denominator=layer.grid_denominator)
        ctx.save_for_backward(x)
        ctx.qw, ctx.ax, ctx.layer, ctx.step = qw, ax, layer, step
        return y

    @staticmethod
    def backward(ctx, dy):
        (x,) = ctx.saved_tensors
        layer, step = ctx.layer, ctx.step
        dy = dy.contiguous()
        ag = layer.scale_dy.get(dy, step)
        dx, dw = B.linear_backward(dy, x, ctx.qw, ag, ctx.ax, seed=sr_stream_seed(layer.seed, layer.rank, step), target_T=layer.target_T,
                                   target_T_wgrad_dy=layer.target_T_wgrad_dy, out_dtype=dy.dtype,
                                   grid_denominator=layer.grid_denominator, grad_rounding=layer.grad_rounding)
        return dx, dw, None, None


class Ue5m3Linear(torch.nn.Module):
    """y = x W^T with UE5M3-FP4 operands in all three GEMMs.  `x` is [tokens, in_features] (bfloat16 or float32);
    call `advance()` once per optimizer step so that the held references refresh every `interval` steps.
    `grid_denominator` not None runs the three products under the Section 6.2 output model (0: without its grid
    step); `grad_rounding` is the rounding of the upstream gradient (stochastic by default).  `seed` names the layer's
    stochastic-rounding stream (default: the count of layers built before it); the rank inside `group` and the step are
    mixed in, so layers, ranks and steps draw independently."""

    def __init__(self, in_features: int, out_features: int, device="cuda", dtype=torch.bfloat16, interval: int = 50,
                 target_T: float = 448.0, target_T_wgrad_dy: Optional[float] = None, seed: Optional[int] = None, group=None,
                 grid_denominator: Optional[int] = None, grad_rounding: int = B.ROUND_SR):
        super().__init__()
        self.weight = torch.nn.Parameter(torch.empty(out_features, in_features, device=device, dtype=dtype).normal_(0, 0.02))
        self.target_T = float(target_T)
        self.target_T_wgrad_dy = float(target_T if target_T_wgrad_dy is None else target_T_wgrad_dy)
        global _layer_counter
        self.seed = _layer_counter if seed is None else int(seed)     # default: a stream of its own per layer
        _layer_counter += 1
        self.rank = _group_rank(group)          # mixed into the draws only; the tensor references stay rank-independent
        self.grid_denominator = grid_denominator
        self.grad_rounding = int(grad_rounding)
        self.step = 0
        self.scale_x, self.scale_w, self.scale_dy = (OperandScale(interval, group) for _ in range(3))

    def advance(self) -> None:
        self.step += 1

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return _Ue5m3LinearFn.apply(x, self.weight, self, self.step)
