"""Seeded synthetic gradients with the shapes of the paper's workloads.

This module only draws inputs.  It holds none of LoCo's arithmetic and imports
neither the CUDA binding nor the oracle; both sides are fed the same bytes that
come out of here.  The paper trains LLAMA2 / Mixtral models on corpora that are
not available offline, so every gradient here is random noise laid out like
those models' flattened parameter lists (bf16 by default, cut into buckets or
kept as one flat buffer).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import torch

_MASK63 = (1 << 63) - 1


def mix_seed(*parts: int) -> int:
    """Fold integers into one 63-bit generator seed (splitmix64 finaliser per part)."""
    x = 0x9E3779B97F4A7C15
    for p in parts:
        x = (x ^ (int(p) & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
        x = (x + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
        x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        x = x ^ (x >> 31)
    return x & _MASK63


def _gen(device, *parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(mix_seed(*parts))
    return g


# --------------------------------------------------------------------------- model shapes

@dataclass(frozen=True)
class Layout:
    """A flattened parameter list: consecutive segments (numel, group) in order."""
    name: str
    segments: Tuple[Tuple[int, int], ...]   # (numel, group id); one scale is drawn per group
    n_groups: int

    @property
    def numel(self) -> int:
        return sum(s for s, _ in self.segments)


def dense_transformer(name: str, layers: int, d_model: int, d_ffn: int, vocab: int) -> Layout:
    """Llama-style decoder: embedding, `layers` x (4 attention + 3 FFN matrices + 2 norms), final norm, head."""
    segs: List[Tuple[int, int]] = [(vocab * d_model, 0)]
    for l in range(layers):
        g = 1 + l
        segs += [(d_model * d_model, g)] * 4
        segs += [(d_model * d_ffn, g)] * 3
        segs += [(d_model, g)] * 2
    segs.append((d_model, layers + 1))
    segs.append((vocab * d_model, layers + 2))
    return Layout(name, tuple(segs), layers + 3)


def llama2_7b() -> Layout:
    """32 layers, d_model 4096, FFN 11008, vocab 32000: 6,738,415,616 elements."""
    return dense_transformer("llama2-7b", 32, 4096, 11008, 32000)


def dense_13b() -> Layout:
    """40 layers, d_model 5120, FFN 13824, vocab 32000: 13,015,864,320 elements."""
    return dense_transformer("dense-13b", 40, 5120, 13824, 32000)


def mixtral_layer(d_model: int = 4096, d_ffn: int = 14336, experts: int = 8, kv_dim: int = 1024) -> Layout:
    """One Mixtral-8x7B decoder layer: attention (GQA), router, 2 norms, then 8 experts of 3 matrices.

    Groups: 0 = shared part, 1..experts = one per expert (so that experts can be zeroed).
    """
    segs: List[Tuple[int, int]] = [(d_model * d_model, 0), (d_model * kv_dim, 0), (d_model * kv_dim, 0),
                                   (d_model * d_model, 0), (d_model * experts, 0), (d_model, 0), (d_model, 0)]
    for e in range(experts):
        segs += [(d_model * d_ffn, 1 + e)] * 3
    return Layout("mixtral-layer", tuple(segs), 1 + experts)


def bucket_ranges(total: int, bucket: int) -> List[Tuple[int, int]]:
    """Cut [0, total) into consecutive buckets of `bucket` elements; the last may be shorter."""
    return [(lo, min(lo + bucket, total)) for lo in range(0, total, bucket)]


def group_scales(seed: int, n_groups: int, low_exp: float = -1.0, high_exp: float = 1.0) -> List[float]:
    """One multiplier 10^U(low, high) per group (log-uniform in [0.1, 10] by default), drawn once."""
    g = _gen("cpu", seed, 0x5CA1E)
    u = torch.rand(n_groups, generator=g, dtype=torch.float64)
    return [float(10.0 ** (low_exp + (high_exp - low_exp) * x)) for x in u]


# --------------------------------------------------------------------------- value draws

def gaussian(n: int, sigma: float, *, seed: int, worker: int = 0, step: int = 0, tag: int = 0,
             dtype=torch.float32, device="cpu") -> torch.Tensor:
    """n i.i.d. N(0, sigma^2) values, rounded once to `dtype`."""
    g = _gen(device, seed, worker, step, tag)
    x = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    return (x * sigma).to(dtype)


def student_t(n: int, nu: float, scale: float, *, seed: int, worker: int = 0, step: int = 0, tag: int = 0,
              dtype=torch.float32, device="cpu") -> torch.Tensor:
    """n i.i.d. Student-t(nu) values times `scale`: z / sqrt(chi2_nu / nu) with integer nu."""
    g = _gen(device, seed, worker, step, tag)
    z = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    chi2 = torch.zeros(n, device=device, dtype=torch.float32)
    for _ in range(int(nu)):
        w = torch.randn(n, generator=g, device=device, dtype=torch.float32)
        chi2 += w * w
    return (z / torch.sqrt(chi2 / float(nu)) * scale).to(dtype)


def layout_slice(layout: Layout, lo: int, hi: int, scales: List[float], base: float, *, seed: int,
                 worker: int = 0, step: int = 0, dist: str = "gaussian", nu: float = 3.0,
                 dtype=torch.bfloat16, device="cpu") -> torch.Tensor:
    """Elements [lo, hi) of a flattened model gradient: noise times base * scales[group of the element].

    A scale of 0 gives an all-zero segment (an expert that received no token).
    """
    n = hi - lo
    tag = lo & _MASK63
    if dist == "gaussian":
        x = gaussian(n, 1.0, seed=seed, worker=worker, step=step, tag=tag, device=device)
    elif dist == "student_t":
        x = student_t(n, nu, 1.0, seed=seed, worker=worker, step=step, tag=tag, device=device)
    else:
        raise ValueError(dist)
    pos = 0
    for numel, grp in layout.segments:
        a, b = max(pos, lo), min(pos + numel, hi)
        if a < b:
            x[a - lo:b - lo] *= base * scales[grp]
        pos += numel
        if pos >= hi:
            break
    return x.to(dtype)


def zero_expert_scales(seed: int, layer: int, experts: int = 8, zeros: int = 2) -> List[float]:
    """Group scales for one Mixtral layer with `zeros` of the experts unrouted (scale 0)."""
    g = _gen("cpu", seed, layer, 0xE0)
    dead = torch.randperm(experts, generator=g)[:zeros].tolist()
    return [1.0] + [0.0 if e in dead else 1.0 for e in range(experts)]


def as_numpy_bits(t: torch.Tensor):
    """Host copy for the CPU side: float32 array, or uint16 bit patterns for bf16."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
