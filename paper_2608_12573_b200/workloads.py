"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module holds input recipes only -- none of the method's arithmetic.  Every
tensor comes from a `torch.Generator` seeded with the given seed, on the CPU by
default; the billion-element cases may be drawn on the GPU (`device="cuda"`,
still seeded, still deterministic for a given device type) because drawing and
sorting 2^30 numbers on the host takes minutes.  The same bytes go to the
library and to the oracle.

The recipes stand in for the paper's synthetic workloads (Uniform, Standard
Normal and heavy-tailed Pareto tensors, N in [2^22, 2^30], Section 5
"Experimental setup") and for the post-ReLU activations of its BatchTopK SAE
experiment (Section 5 "Application"), whose model and data set are not
available here.
"""
from __future__ import annotations

import numpy as np
import torch


def _gen(seed: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _check(x: torch.Tensor) -> torch.Tensor:
    """No NaN and no negative zero: on such inputs every reading of the order agrees."""
    xf = x.float() if x.dtype != torch.float32 else x
    assert not torch.isnan(xf).any(), "generator produced NaN"
    neg_zero = (xf == 0) & torch.signbit(xf)
    assert not neg_zero.any(), "generator produced -0.0"
    return x


def uniform(n: int, seed: int, device: str = "cpu") -> torch.Tensor:
    """i.i.d. Uniform[0,1), fp32."""
    return _check(torch.rand(n, generator=_gen(seed, device), device=device, dtype=torch.float32))


def normal(rows: int, n: int, seed: int, dtype: torch.dtype = torch.float32,
           device: str = "cpu") -> torch.Tensor:
    """i.i.d. N(0,1), drawn in fp32 and rounded to `dtype`; shape (rows, n)."""
    x = torch.randn(rows, n, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return _check(x.to(dtype))


def relu_gaussian(n: int, seed: int, shift: float = -0.5, dtype: torch.dtype = torch.bfloat16,
                  device: str = "cpu") -> torch.Tensor:
    """ReLU(x), x ~ N(shift, 1): the flattened BatchTopK pre-activation stand-in."""
    x = torch.randn(n, generator=_gen(seed, device), device=device, dtype=torch.float32)
    x = torch.clamp_min(x + shift, 0.0)
    return _check(x.to(dtype))


def cauchy(n: int, seed: int, device: str = "cpu") -> torch.Tensor:
    x = torch.empty(n, dtype=torch.float32, device=device)
    x.cauchy_(0.0, 1.0, generator=_gen(seed, device))
    x = torch.nan_to_num(x, nan=0.0)
    x[x == 0] = 0.0
    return _check(x)


def pareto(n: int, seed: int, alpha: float = 1.1, device: str = "cpu") -> torch.Tensor:
    """Pareto(alpha) with scale 1, as (1 - U)^(-1/alpha)."""
    u = torch.rand(n, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return _check((1.0 - u).pow_(-1.0 / alpha))


def sorted_uniform(n: int, seed: int, device: str = "cpu") -> torch.Tensor:
    """Uniform[0,1) sorted ascending: every top element sits at the very end."""
    return torch.sort(uniform(n, seed, device)).values


def few_values(n: int, seed: int, distinct: int = 16, device: str = "cpu") -> torch.Tensor:
    """Each element drawn i.i.d. uniformly from `distinct` constants j / distinct."""
    j = torch.randint(0, distinct, (n,), generator=_gen(seed, device), device=device)
    return _check(j.to(torch.float32) / float(distinct))


def spikes(n: int, seed: int, count: int = 64, device: str = "cpu") -> torch.Tensor:
    """All zeros except `count` distinct random positions set to +1."""
    x = torch.zeros(n, dtype=torch.float32, device=device)
    g = _gen(seed, device)
    pos = torch.unique(torch.randint(0, n, (4 * count,), generator=g, device=device))
    perm = torch.randperm(pos.numel(), generator=g, device=device)
    x[pos[perm[:count]]] = 1.0
    return _check(x)


ADVERSARIAL = {           # name -> (recipe, seed) for the heavy-tailed / adversarial sweep
    "cauchy": (cauchy, 4),
    "pareto": (pareto, 5),
    "sorted": (sorted_uniform, 6),
    "few_values": (few_values, 7),
    "spikes": (spikes, 8),
}


def as_numpy(x: torch.Tensor) -> np.ndarray:
    """Host NumPy view of the same bytes; bf16 becomes its uint16 bit patterns."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()
