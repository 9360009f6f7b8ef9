"""Seeded synthetic key/value generators for the five benchmark workloads.

This module only *makes data*: it contains none of the compression method's
arithmetic (no sketching, scoring, selection or gathering), so both the CUDA
path and the CPU oracle may be fed from it.  Everything is drawn from a
``torch.Generator`` seeded from (workload seed, sequence, layer, head), on the
device that is asked for; the resulting bf16 bit patterns are what both sides
receive.

Recipe per unit (one sequence x layer x KV head), d channels, n tokens:

    K_pre  = (G diag(s) Q + 1 b^T) diag(c)
             G ~ N(0,1) [n x d];  s_j = j^-p (j = 1..d);
             Q  = orthogonal factor of a Gaussian d x d matrix, signs fixed so
                  that the triangular factor has a positive diagonal;
             b ~ N(0, 0.5^2) [d], the same for every token;
             c_j = 10 on `n_out` channels drawn without replacement, else 1.
    near-duplicates (only where `dup_frac` > 0): a `dup_frac` share of rows is
             overwritten by another row of the same unit + N(0, 0.01^2) noise.
    K_rope = rotate-half rotary embedding of K_pre: pairs (j, j + d/2),
             inverse frequency theta^(-2j/d), positions 0..n-1 within the
             sequence.
    V      ~ N(0,1) [n x d].
All three are rounded to bf16.

These tensors stand in for the prefill keys/values of Llama-3.1 / Qwen-2.5
models on long-context evaluation inputs, which are not available offline.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch


@dataclass
class Workload:
    """Shape and recipe of one benchmark configuration."""

    name: str
    layers: int
    heads: int
    d: int
    seqlens: List[int]                  # tokens per sequence (batch = len)
    ratios: List[float]                 # retention ratio per sequence
    p: float = 1.0                      # spectrum exponent: s_j = j^-p
    n_out: int = 4                      # outlier channels scaled x10
    theta: float = 5e5                  # rotary base
    dup_frac: float = 0.0               # share of near-duplicate rows
    seed: int = 0
    m: int = 48                         # sketch dimension (paper's setting)

    @property
    def batch(self) -> int:
        return len(self.seqlens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    @property
    def cu_seqlens(self) -> List[int]:
        out = [0]
        for n in self.seqlens:
            out.append(out[-1] + int(n))
        return out

    @property
    def units(self) -> int:
        return self.layers * self.heads * self.batch


def _uniform01(seed: int, count: int) -> List[float]:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.rand(count, generator=g, dtype=torch.float64).tolist()


def workload(name: str, layers: Optional[int] = None, seed: Optional[int] = None) -> Workload:
    """The five named configurations.  `layers` overrides the layer count (to
    take a slice of a large model shape); `seed` overrides the base seed."""
    name = name.lower()
    if name in ("c0", "tiny"):
        w = Workload("c0-tiny", 1, 2, 128, [1024], [0.5], p=1.0, n_out=4, theta=5e5, seed=0)
    elif name in ("c1", "llama8b"):
        w = Workload("c1-llama3.1-8b", 32, 8, 128, [8192], [0.3], p=0.7, n_out=4, theta=5e5, seed=1)
    elif name in ("c2", "qwen7b"):
        s = 2 if seed is None else seed
        r = 0.2 + 0.4 * _uniform01(1000 + s, 1)[0]
        w = Workload("c2-qwen2.5-7b", 28, 4, 128, [32768], [r], p=1.0, n_out=8, theta=1e6, seed=s)
    elif name in ("c3", "qwen32b"):
        w = Workload("c3-qwen2.5-32b", 64, 8, 128, [131072], [0.32], p=1.0, n_out=4, theta=5e5,
                     dup_frac=0.05, seed=3)
    elif name in ("c4", "ragged"):
        s = 4 if seed is None else seed
        u = _uniform01(2000 + s, 32)
        lo, hi = math.log(2048.0), math.log(65536.0)
        lens = [int(round(math.exp(lo + (hi - lo) * u[i]))) for i in range(16)]
        choices = (0.2, 0.3, 0.5)
        ratios = [choices[min(2, int(u[16 + i] * 3))] for i in range(16)]
        w = Workload("c4-ragged-llama3.1-8b", 32, 8, 128, lens, ratios, p=0.7, n_out=4, theta=5e5, seed=s)
    else:
        raise ValueError(f"unknown workload {name!r}")
    if layers is not None:
        w.layers = int(layers)
    if seed is not None:
        w.seed = int(seed)
    return w


def _unit_seed(base: int, seq: int, layer: int, head: int) -> int:
    # A fixed mixing of the four integers into one 63-bit seed.
    x = (base * 0x9E3779B97F4A7C15 + seq * 0xBF58476D1CE4E5B9
         + layer * 0x94D049BB133111EB + head * 0xD6E8FEB86659FD93 + 0x2545F4914F6CDD1D)
    return x & 0x7FFFFFFFFFFFFFFF


def make_unit(w: Workload, seq: int, layer: int, head: int, device="cpu"):
    """One unit's (K_pre, K_rope, V), each bf16 [n, d] on `device`."""
    n, d = int(w.seqlens[seq]), w.d
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(_unit_seed(w.seed, seq, layer, head))
    f32 = dict(dtype=torch.float32, device=dev)

    A = torch.randn(d, d, generator=g, **f32)
    Q, R = torch.linalg.qr(A.double().cpu())
    Q = (Q * torch.sign(torch.diagonal(R))).to(dev).float()
    s = torch.arange(1, d + 1, **f32) ** (-w.p)
    b = 0.5 * torch.randn(d, generator=g, **f32)
    perm = torch.randperm(d, generator=g, device=dev)
    c = torch.ones(d, **f32)
    c[perm[: w.n_out]] = 10.0

    G = torch.randn(n, d, generator=g, **f32)
    K = (G * s) @ Q
    K = (K + b) * c
    if w.dup_frac > 0.0 and n > 1:
        n_dup = int(w.dup_frac * n)
        dst = torch.randperm(n, generator=g, device=dev)[:n_dup]
        src = torch.randint(0, n, (n_dup,), generator=g, device=dev)
        noise = 0.01 * torch.randn(n_dup, d, generator=g, **f32)
        K[dst] = K[src] + noise
    V = torch.randn(n, d, generator=g, **f32)

    half = d // 2
    inv_freq = w.theta ** (-torch.arange(0, half, dtype=torch.float64, device=dev) * 2.0 / d)
    ang = torch.arange(n, dtype=torch.float64, device=dev)[:, None] * inv_freq[None, :]
    cos, sin = torch.cos(ang).float(), torch.sin(ang).float()
    k1, k2 = K[:, :half], K[:, half:]
    K_rope = torch.cat([k1 * cos - k2 * sin, k2 * cos + k1 * sin], dim=1)

    return K.to(torch.bfloat16), K_rope.to(torch.bfloat16), V.to(torch.bfloat16)


def make_tensors(w: Workload, device="cpu", want_pre: bool = True, layers: Optional[Sequence[int]] = None):
    """Packed tensors for a whole workload (or the listed layers of it).

    Returns (K_pre or None, K_rope, V), each bf16 [L, H, total_tokens, d] with
    sequences packed back to back along the token axis."""
    layer_ids = list(range(w.layers)) if layers is None else list(layers)
    L, H, T, d = len(layer_ids), w.heads, w.total_tokens, w.d
    dev = torch.device(device)
    kp = torch.empty(L, H, T, d, dtype=torch.bfloat16, device=dev) if want_pre else None
    kr = torch.empty(L, H, T, d, dtype=torch.bfloat16, device=dev)
    v = torch.empty(L, H, T, d, dtype=torch.bfloat16, device=dev)
    cu = w.cu_seqlens
    for li, layer in enumerate(layer_ids):
        for h in range(H):
            for b in range(w.batch):
                a, k, vv = make_unit(w, b, layer, h, device=dev)
                if want_pre:
                    kp[li, h, cu[b]:cu[b + 1]] = a
                kr[li, h, cu[b]:cu[b + 1]] = k
                v[li, h, cu[b]:cu[b + 1]] = vv
    return kp, kr, v


def make_sketch_matrix(d: int, m: int, seed: int) -> torch.Tensor:
    """A Gaussian sketch drawn with torch's CPU generator: fp32 [d, m], entries
    N(0, 1/m).  Data for both sides; the library's own seeded generator is a
    separate convenience."""
    g = torch.Generator(device="cpu")
    g.manual_seed(0x5EED0000 + seed)
    return (torch.randn(d, m, generator=g, dtype=torch.float64) / math.sqrt(m)).float()


def make_attention_scores(w: Workload, seed: int = 0, device="cpu") -> torch.Tensor:
    """A stand-in for the caller-supplied attention term: positive, heavy-tailed
    fp32 [L, H, total_tokens] (a softmax column sum is positive with a few
    large columns)."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(0xA77E0000 + seed)
    x = torch.randn(w.layers, w.heads, w.total_tokens, generator=g, dtype=torch.float32, device=dev)
    return torch.exp(0.75 * x)


def make_queries(w: Workload, q_per_kv: int, device="cpu", seed: int = 0) -> torch.Tensor:
    """Stand-in query vectors for the attention term: bf16 [L, H * q_per_kv, total_tokens, d], Gaussian with a
    per-head channel scale (a few heads attend sharply, most diffusely)."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(0x9E7700 + 131 * w.seed + seed)
    hq = w.heads * q_per_kv
    q = torch.randn(w.layers, hq, w.total_tokens, w.d, generator=g, dtype=torch.float32, device=dev)
    sharp = 0.5 + 2.0 * torch.rand(w.layers, hq, 1, 1, generator=g, dtype=torch.float32, device=dev)
    return (q * sharp).to(torch.bfloat16)
