"""Seeded synthetic workloads for the LocMoE router path.

This module only draws random inputs with the shapes, dtypes and structure of
the five benchmark configurations; it contains none of the router's
arithmetic.  Both the CUDA tests/bench and the CPU oracle's tests take their
inputs from here so that they see the same bits.

Tokens are drawn with ``torch.randn`` in fixed chunks of 65 536 tokens from a
generator seeded per configuration (``1234 + 100 * config``) on the device that
is asked for.  The CPU and CUDA generators produce different streams, so a
comparison always draws once and copies the bits to the other side.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

BASE_SEED = 1234
CHUNK = 65536


@dataclass(frozen=True)
class Workload:
    name: str
    config: int
    T: int
    H: int
    E: int
    n_nodes: int
    dev_per_node: int
    dtype: str           # "f32" | "bf16"
    tokens: str          # "normal" | "zipf_mixture"
    src: str             # "uniform" | "mod"
    y_dtype: str = "same"  # dtype of the expert outputs fed to combine ("same" | "f32")
    note: str = ""

    @property
    def D(self) -> int:
        return self.n_nodes * self.dev_per_node

    @property
    def seed(self) -> int:
        return BASE_SEED + 100 * self.config

    def scaled(self, T: int) -> "Workload":
        """Same configuration with fewer tokens (parity-test sizes)."""
        return replace(self, T=T, name=f"{self.name}[T={T}]")


CONFIGS = {
    1: Workload("tiny", 1, 4096, 1024, 8, 2, 4, "f32", "normal", "uniform"),
    2: Workload("pangu_sigma_like", 2, 65536, 5120, 64, 8, 8, "bf16", "normal", "mod"),
    3: Workload("skewed_zipf", 3, 262144, 4096, 128, 16, 8, "bf16", "zipf_mixture", "mod"),
    4: Workload("large_batch", 4, 1048576, 5120, 256, 32, 8, "bf16", "normal", "mod", y_dtype="f32"),
    5: Workload("full_layer_router", 5, 65536, 2560, 32, 4, 8, "bf16", "normal", "mod"),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def mixture_centres(w: Workload) -> torch.Tensor:
    """Config 3: 128 centres of norm 3, centre k along the unit block-indicator
    direction of group perm[k] (one direction per expert), perm seeded."""
    g = w.H // w.E
    rng = np.random.default_rng(w.seed + 3)
    perm = rng.permutation(w.E)
    n_centres = 128
    c = torch.zeros(n_centres, w.H, dtype=torch.float32)
    for k in range(n_centres):
        e = int(perm[k % w.E])
        c[k, e * g:(e + 1) * g] = 3.0 / float(np.sqrt(g))
    return c


def mixture_labels(w: Workload) -> torch.Tensor:
    """Config 3: centre label per token, Zipf(s = 1.2) weights over 128 centres."""
    rng = np.random.default_rng(w.seed + 2)
    p = 1.0 / np.arange(1, 129, dtype=np.float64) ** 1.2
    p /= p.sum()
    return torch.from_numpy(rng.choice(128, size=w.T, p=p).astype(np.int64))


def make_tokens(w: Workload, device="cpu") -> torch.Tensor:
    """x[T][H] in the workload's dtype on ``device``."""
    dev = torch.device(device)
    gen = _gen(dev, w.seed)
    out = torch.empty(w.T, w.H, dtype=torch_dtype(w.dtype), device=dev)
    centres = labels = None
    if w.tokens == "zipf_mixture":
        centres = mixture_centres(w).to(dev)
        labels = mixture_labels(w).to(dev)
    sub = 8192  # keeps the fp32 staging buffer small
    for s in range(0, w.T, CHUNK):
        n = min(CHUNK, w.T - s)
        for s2 in range(s, s + n, sub):
            m = min(sub, s + n - s2)
            z = torch.randn(m, w.H, generator=gen, device=dev, dtype=torch.float32)
            if centres is not None:
                z += centres[labels[s2:s2 + m]]
            out[s2:s2 + m] = z.to(out.dtype)
    return out


def make_src(w: Workload, device="cpu") -> torch.Tensor:
    """Source device of each token, int32[T]."""
    if w.src == "mod":
        s = torch.arange(w.T, dtype=torch.int64) % w.D
    else:
        rng = np.random.default_rng(w.seed + 1)
        s = torch.from_numpy(rng.integers(0, w.D, size=w.T))
    return s.to(torch.int32).to(device)


def make_expert_out(w: Workload, rows: int, device="cpu", dtype: str = "f32") -> torch.Tensor:
    """Random expert outputs y[rows][H] in slot layout (config 4's fused combine)."""
    dev = torch.device(device)
    gen = _gen(dev, w.seed + 4)
    out = torch.empty(rows, w.H, dtype=torch_dtype(dtype), device=dev)
    sub = 8192
    for s in range(0, rows, sub):
        m = min(sub, rows - s)
        out[s:s + m] = torch.randn(m, w.H, generator=gen, device=dev, dtype=torch.float32).to(out.dtype)
    return out


def make_expert_weights(w: Workload, F: int, device="cpu", std: float = 0.02):
    """Random-init expert weights of config 5: W_in [E][F][H], W_out [E][H][F], bf16, N(0, std)."""
    dev = torch.device(device)
    gen = _gen(dev, w.seed + 5)
    def draw(a, b, c):
        out = torch.empty(a, b, c, dtype=torch.bfloat16, device=dev)
        for e in range(a):
            out[e] = (torch.randn(b, c, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)
        return out
    return draw(w.E, F, w.H), draw(w.E, w.H, F)


def host_bits(x: torch.Tensor) -> np.ndarray:
    """Raw storage on the host: float32 array, or uint16 array holding bf16 bits."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16)
    if x.dtype == torch.float32:
        return x.numpy()
    raise TypeError(x.dtype)
