"""Seeded synthetic inputs shaped like the router's workloads.

Holds no routing arithmetic: only the shapes, dtypes and random draws of the
five workloads (token batches through a gate of E experts) plus the per-expert
Zipf bias of the skewed workload.  Both the CUDA path and the CPU checker are
fed from here, on the host, with a seeded torch.Generator, so that they see
identical bits.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    d_model: int
    E: int
    k: int
    capacity_factor: float
    dtype: str            # "f32" or "bf16": hidden, W_gate, expert buffers
    skew: bool = False    # add the Zipf expert bias
    temperature: float = 1.0

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


WORKLOADS = {
    "tiny": Workload("tiny", 512, 256, 8, 2, 1.0, "f32"),
    "k2e16": Workload("k2e16", 4096, 1024, 16, 2, 1.0, "bf16"),
    "k8e64": Workload("k8e64", 8192, 2048, 64, 8, 1.0, "bf16"),
    "skew": Workload("skew", 16384, 2048, 64, 8, 1.25, "bf16", skew=True),
    "stress": Workload("stress", 65536, 4096, 128, 8, 1.0, "bf16"),
}


def scaled(w: Workload, T: int | None = None, d_model: int | None = None) -> Workload:
    """Same workload with fewer tokens / narrower rows (for quick checks)."""
    return replace(w, T=T or w.T, d_model=d_model or w.d_model,
                   name=f"{w.name}[T={T or w.T},d={d_model or w.d_model}]")


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000003 + stream)
    return g


def hidden(w: Workload, seed: int = 0) -> torch.Tensor:
    """H[T, d_model] i.i.d. N(0,1), rounded to the workload's dtype."""
    return torch.randn(w.T, w.d_model, generator=_gen(seed, 1), dtype=torch.float32).to(w.torch_dtype)


def w_gate(w: Workload, seed: int = 0) -> torch.Tensor:
    """W_g[d_model, E] i.i.d. N(0, 1/d_model), rounded to the workload's dtype."""
    x = torch.randn(w.d_model, w.E, generator=_gen(seed, 2), dtype=torch.float32)
    return (x / math.sqrt(w.d_model)).to(w.torch_dtype)


def expert_bias(w: Workload, seed: int = 0):
    """b_e = 2 ln(r_e^-1.1), r a seeded permutation of 1..E; None unless skewed."""
    if not w.skew:
        return None
    ranks = torch.randperm(w.E, generator=_gen(seed, 3)).to(torch.float64) + 1.0
    return (2.0 * (-1.1) * torch.log(ranks)).to(torch.float32)


def upstream_grad(w: Workload, seed: int = 0) -> torch.Tensor:
    """dY[T, d_model] i.i.d. N(0,1) over the combine output."""
    return torch.randn(w.T, w.d_model, generator=_gen(seed, 4), dtype=torch.float32).to(w.torch_dtype)


def logits_like(T: int, E: int, seed: int = 0, bias: torch.Tensor | None = None) -> torch.Tensor:
    """fp32 stand-in for gate logits (N(0,1) entries), for solver-only checks."""
    x = torch.randn(T, E, generator=_gen(seed, 5), dtype=torch.float32)
    return x + bias if bias is not None else x


def integers(T: int, E: int, lo: int, hi: int, seed: int = 0) -> torch.Tensor:
    """int64 matrix uniform in [lo, hi): small ranges give heavily tied scores."""
    return torch.randint(lo, hi, (T, E), generator=_gen(seed, 6), dtype=torch.int64)
