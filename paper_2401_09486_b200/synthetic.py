"""Seeded synthetic inputs for the LoMA attention path.

This module only draws random numbers and allocates tensors.  It contains none
of the method's arithmetic (no layout, mask, softmax or cache logic), so both
the CUDA library's callers and the CPU checker can be fed from it without
sharing anything else.

Distributions follow the workload description: Q/K/V entries are i.i.d. normal
with a chosen standard deviation (1 for tolerance checks, 1/sqrt(D) for
Llama-2-7B-shaped timing runs), stored in the requested dtype (rounded once,
here), laid out [B, H, S, D] with D contiguous.
"""

from __future__ import annotations

import torch


def _generator(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal_tensor(shape, seed: int, std: float = 1.0, dtype=torch.float32, device="cpu") -> torch.Tensor:
    """N(0, std^2) tensor of `shape`, drawn in fp32 from a seeded generator on
    `device`, then rounded to `dtype`."""
    g = _generator(seed, device)
    x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(dtype)


def qkv(B: int, H: int, S: int, D: int, seed: int, std: float = 1.0, dtype=torch.float32, device="cpu"):
    """Three independent [B, H, S, D] tensors (Q, K, V) from seeds derived from
    `seed` (3*seed, 3*seed+1, 3*seed+2)."""
    return tuple(normal_tensor((B, H, S, D), 3 * seed + i, std, dtype, device) for i in range(3))


def big_normal_(out: torch.Tensor, seed: int, std: float = 1.0, slab_elems: int = 1 << 28) -> torch.Tensor:
    """Fill a large tensor in place with N(0, std^2), slab by slab, so that no
    fp32 temporary as large as the tensor itself is ever allocated."""
    g = _generator(seed, out.device)
    flat = out.view(-1)
    n = flat.numel()
    for lo in range(0, n, slab_elems):
        hi = min(n, lo + slab_elems)
        tmp = torch.randn(hi - lo, generator=g, device=out.device, dtype=torch.float32)
        if std != 1.0:
            tmp.mul_(std)
        flat[lo:hi].copy_(tmp)
        del tmp
    return out
