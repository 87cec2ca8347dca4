"""The benchmark / parity workloads: layer shapes and GRASS settings per configuration.

Shapes are the paper's LLaMA model-dimension table; a "block" is the seven
linear projections of one transformer layer.  Row selection acts on the output
features m of every projection.  Nothing here computes.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from . import binding as B
from .synthetic import LLAMA_DIMS, llama_projections


@dataclass
class Workload:
    name: str
    shapes: list                  # [(proj_name, m, n)] of one block
    layers: int                   # number of blocks
    T: int
    r: int
    method: int
    K: int
    dtype: torch.dtype
    alpha: float = 0.25
    reset_state: bool = True
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    notes: dict = field(default_factory=dict)

    def layer_list(self):
        return [(li, pi, name, m, n) for li in range(self.layers)
                for pi, (name, m, n) in enumerate(self.shapes)]

    def flops_regular(self):
        """2 r T n per layer-step (the projection; Adam and the apply add ~14 r n)."""
        return sum(2.0 * min(self.r, m) * self.T * n for _, m, n in self.shapes) * self.layers

    def flops_refresh_extra(self):
        """2 m T n per layer for the dense gradient a refresh forms."""
        return sum(2.0 * m * self.T * n for _, m, n in self.shapes) * self.layers


def _llama(size, layers, T, r, method, K, reset, name=None):
    hidden, ffn = LLAMA_DIMS[size]
    return Workload(name or f"llama{size.lower()}", llama_projections(hidden, ffn), layers, T, r,
                    method, K, torch.bfloat16, reset_state=reset)


def get(name: str, r: int | None = None, T: int | None = None, layers: int | None = None) -> Workload:
    if name == "config1":
        w = Workload("config1", [("w", 256, 256)], 1, 512, 32, B.SEL_TOPR, 1, torch.float32, alpha=1.0)
    elif name == "llama60m":
        w = _llama("60M", 8, 65536, 128, B.SEL_MULTINOMIAL_NORM, 200, True)
    elif name == "llama350m":
        w = _llama("350M", 24, 65536, 256, B.SEL_TOPR, 5, True)
    elif name == "llama1b":
        w = _llama("1B", 24, 65536, 512, B.SEL_MULTINOMIAL_NORM, 200, False)
    elif name == "llama7b_block":
        w = _llama("7B", 1, 32768, 1024, B.SEL_TOPR, 200, True, name)
    elif name == "llama13b_block":
        w = _llama("13B", 1, 32768, 1024, B.SEL_TOPR, 200, True, name)
    else:
        raise ValueError(f"unknown workload {name}")
    w.notes["w_is_bf16"] = w.dtype == torch.bfloat16
    if r is not None:
        w.r = r
    if T is not None:
        w.T = T
    if layers is not None:
        w.layers = layers
    return w


NAMES = ["config1", "llama60m", "llama350m", "llama1b", "llama7b_block", "llama13b_block"]
