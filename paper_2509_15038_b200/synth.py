"""Seeded synthetic KV caches and sketch matrices.

This module only draws random inputs; it holds none of the method's
arithmetic, so both the CUDA path and the CPU oracle may be fed from it.
The workloads stand in, by shape and value structure only, for the paper's
LongBench / Ruler / long-text runs on LLaMA-3.1-8B and Mistral-7B (32 layers,
8 KV heads, 32 query heads, head_dim 128): outlier channels in K and
heavy-tailed row norms in V mimic known KV-cache statistics.

Layers are folded into the batch axis: tensors are ``[L*B, Hkv, n_max, d]``
bf16, element ``lb = layer * B + b``.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    batch: int
    kv_heads: int
    q_heads: int
    n_max: int
    d: int
    r: int
    budget: int            # k per head, forced tokens included
    num_sink: int
    window: int
    adaptive: bool = False
    alpha: float = 0.20
    kind: str = "llm"      # "planted" (config 1) or "llm" (configs 2-5)
    ragged: Optional[tuple] = None   # (lo, hi) inclusive length range, else None
    data_seed: int = 0

    @property
    def folded_batch(self) -> int:
        return self.layers * self.batch


def _k(n, frac, w):
    return int(np.floor(frac * n)) + w


# The five benchmark configurations (seeds: data seed = config number, G seed 0).
CONFIGS = {
    "cfg1": Workload("cfg1", 1, 1, 8, 8, 1024, 128, 32, 128, 0, 32, kind="planted", data_seed=1),
    "cfg2": Workload("cfg2", 32, 1, 8, 32, 8192, 128, 32, _k(8192, 0.2, 64), 0, 64, data_seed=2),
    "cfg3": Workload("cfg3", 32, 4, 8, 32, 32768, 128, 32, _k(32768, 0.1, 64), 0, 64, data_seed=3),
    "cfg3_b1": Workload("cfg3_b1", 32, 1, 8, 32, 32768, 128, 32, _k(32768, 0.1, 64), 0, 64, data_seed=3),
    "cfg4": Workload("cfg4", 32, 1, 8, 32, 131072, 128, 64, _k(131072, 0.05, 128), 0, 128,
                     adaptive=True, alpha=0.20, data_seed=4),
    "cfg5": Workload("cfg5", 32, 16, 8, 32, 16384, 128, 32, 512, 0, 32, ragged=(2048, 16384),
                     data_seed=5),
}


def shrink(w: Workload, **kw) -> Workload:
    """A smaller case of the same recipe (for parity tests and CPU samples)."""
    return replace(w, **kw)


def make_G(d: int, r: int, seed: int = 0, heads: int = 0) -> np.ndarray:
    """Host fp32 sketch matrix with i.i.d. N(0, 1/r) entries; ``heads`` > 0 gives [heads, d, r]."""
    rng = np.random.default_rng(seed)
    shape = (heads, d, r) if heads else (d, r)
    return (rng.standard_normal(shape) / np.sqrt(r)).astype(np.float32)


def make_seqlens(w: Workload, seed: int = 0) -> Optional[np.ndarray]:
    """Per folded-batch element lengths (int32 [L*B]) for ragged workloads, else None."""
    if w.ragged is None:
        return None
    lo, hi = w.ragged
    rng = np.random.default_rng(seed)
    per_b = rng.integers(lo, hi + 1, size=w.batch, dtype=np.int64)
    return np.tile(per_b, w.layers).astype(np.int32)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_kv_element(w: Workload, lb: int, device="cpu"):
    """K, V of one folded-batch element: bf16 ``[Hkv, n_max, d]`` each."""
    H, n, d = w.kv_heads, w.n_max, w.d
    g = _gen(device, w.data_seed * 1_000_003 + lb)
    K = torch.randn((H, n, d), generator=g, device=device, dtype=torch.float32)
    if w.kind == "planted":
        V = torch.randn((H, n, d), generator=g, device=device, dtype=torch.float32)
        n_planted = min(8, n)
        for h in range(H):
            pos = torch.randperm(n, generator=g, device=device)[:n_planted]
            K[h, pos] *= 20.0
            V[h, pos] *= 20.0
    else:
        for h in range(H):
            ch = torch.randperm(d, generator=g, device=device)[:4]
            K[h][:, ch] *= 10.0
        direction = torch.randn((H, n, d), generator=g, device=device, dtype=torch.float32)
        direction /= direction.norm(dim=-1, keepdim=True).clamp_min(1e-20)
        z = torch.randn((H, n, 1), generator=g, device=device, dtype=torch.float32)
        V = direction * (float(np.sqrt(d)) * torch.exp(0.5 * z))
    return K.to(torch.bfloat16), V.to(torch.bfloat16)


def make_kv(w: Workload, device="cpu"):
    """Whole workload: K, V bf16 ``[L*B, Hkv, n_max, d]`` and seqlens (int32 numpy or None)."""
    LB = w.folded_batch
    K = torch.empty((LB, w.kv_heads, w.n_max, w.d), dtype=torch.bfloat16, device=device)
    V = torch.empty_like(K)
    for lb in range(LB):
        k, v = make_kv_element(w, lb, device)
        K[lb].copy_(k)
        V[lb].copy_(v)
    return K, V, make_seqlens(w)


def to_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> host numpy uint16 bit patterns (same shape)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_u16(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Host uint16 bit patterns -> bf16 tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def f64_to_bf16_u16(x: np.ndarray) -> np.ndarray:
    """Round a host float array to bf16 (round-to-nearest-even via torch) and return the bits."""
    return to_u16(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def u16_to_f64(a: np.ndarray) -> np.ndarray:
    """Decode bf16 bit patterns to float64 exactly (format conversion only)."""
    return (np.asarray(a, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
