"""Seeded synthetic layer inputs shaped like the paper's LLaMA workloads.

This module only draws random tensors; it holds none of the method's
arithmetic, so both the CUDA path and the test oracle may be fed from it.

Recipe (one linear layer W: m x n, T tokens):
    X[t, c]  ~ N(0, 1)
    dY[t, k] = z[t, k] * exp(sigma_s * g[k]),  z, g ~ N(0, 1), g fixed per layer
               (log-normal per-feature scale: heavy-tailed, persistent row norms)
    W[k, c]  ~ N(0, 0.02^2)
Each tensor is rounded once to the requested dtype.  The seed of a tensor is
    seed0 + 1_000_003 * step + 7_919 * (7 * layer + proj) + kind
with kind 0 = X, 1 = z, 2 = W, 3 = g (g always uses step 0).
"""
from __future__ import annotations

import torch

KIND_X, KIND_Z, KIND_W, KIND_G = 0, 1, 2, 3

# (name, out_features m, in_features n) of the seven projections of a LLaMA block
def llama_projections(hidden: int, ffn: int):
    return [("q", hidden, hidden), ("k", hidden, hidden), ("v", hidden, hidden),
            ("o", hidden, hidden), ("gate", ffn, hidden), ("up", ffn, hidden),
            ("down", hidden, ffn)]


LLAMA_DIMS = {  # hidden, FFN (the paper's model-dimension table)
    "60M": (512, 1376), "350M": (1024, 2736), "1B": (2048, 5461),
    "7B": (4096, 11008), "13B": (5120, 13824),
}


def tensor_seed(seed0: int, step: int, layer: int, proj: int, kind: int) -> int:
    return seed0 + 1_000_003 * step + 7_919 * (7 * layer + proj) + kind


def _randn(shape, seed, device):
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def pad_to(n: int, mult: int) -> int:
    return (n + mult - 1) // mult * mult


def _padded(t: torch.Tensor, ld: int) -> torch.Tensor:
    """Return a view with logical shape t.shape inside a buffer of row pitch ld."""
    rows, cols = t.shape
    if ld == cols:
        return t.contiguous()
    buf = torch.zeros((rows, ld), dtype=t.dtype, device=t.device)
    buf[:, :cols] = t
    return buf[:, :cols]


def make_X(T, n, dtype, seed0=0, step=0, layer=0, proj=0, device="cpu", ld=None):
    x = _randn((T, n), tensor_seed(seed0, step, layer, proj, KIND_X), device).to(dtype)
    return _padded(x, ld or n)


def make_dY(T, m, dtype, seed0=0, step=0, layer=0, proj=0, device="cpu",
            sigma_s=1.0, ld=None):
    z = _randn((T, m), tensor_seed(seed0, step, layer, proj, KIND_Z), device)
    g = _randn((m,), tensor_seed(seed0, 0, layer, proj, KIND_G), device)
    z.mul_(torch.exp(sigma_s * g)[None, :])
    return _padded(z.to(dtype), ld or m)


def make_W(m, n, dtype, seed0=0, layer=0, proj=0, device="cpu", ld=None):
    w = (_randn((m, n), tensor_seed(seed0, 0, layer, proj, KIND_W), device) * 0.02).to(dtype)
    return _padded(w, ld or n)


def to_f32_numpy(t: torch.Tensor):
    """Exact widening of a (possibly bf16, possibly padded) tensor to a float32 numpy array."""
    return t.detach().to("cpu", torch.float32).contiguous().numpy()
