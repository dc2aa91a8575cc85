"""Synthetic attention inputs with heavy-tailed column sums.

Recipe (all tensors are drawn from seeded ``torch.Generator`` streams):

* ``g ~ N(0, 1)`` element-wise for q, k and v.
* Every head ``h`` has a fixed unit vector ``u_h``; queries are ``g + 1.5 u_h``.
* 2 % of the token positions of a sequence (shared by its heads) are outliers
  whose key is ``g + 4 u_h``; with the default ``1/sqrt(d)`` scale such a key
  receives a visibly larger softmax weight from every query, which gives the
  accumulated attention scores a heavy tail.
* Values are rounded to the storage dtype (bf16 round-to-nearest-even for the
  bf16 workloads) once, here; whoever consumes them sees the same bytes.

Nothing in this file computes attention, scores or selections.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence, Tuple

import numpy as np
import torch

_KIND = {"q": 1, "k": 2, "v": 3}
OUTLIER_FRACTION = 0.02
OUTLIER_KEY_SHIFT = 4.0
QUERY_MEAN_SHIFT = 1.5


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_heads: int
    head_dim: int
    dtype: str  # "f32" | "bf16"
    prompt_lens: Tuple[int, ...]  # one per sequence
    decode_steps: int
    heavy: Tuple[int, ...]  # k_s per sequence
    recent: Tuple[int, ...]  # r_s per sequence
    layers: int = 1
    seed: int = 20230614

    @property
    def total_tokens(self) -> int:
        return int(sum(self.prompt_lens))

    @property
    def units(self) -> int:
        return self.batch * self.n_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def cu_seqlens(self) -> np.ndarray:
        cu = np.zeros(self.batch + 1, dtype=np.int32)
        cu[1:] = np.cumsum(np.asarray(self.prompt_lens, dtype=np.int64))
        return cu

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def budgets_for(prompt_lens: Sequence[int], fraction: float = 0.2) -> Tuple[Tuple[int, ...], Tuple[int, ...]]:
    """Split ``fraction`` of each prompt length evenly into heavy and recent slots.

    ``ceil(fraction/2 * n)`` each: 205 + 205 for n = 2048 and 52 + 52 for n = 512.
    """
    half = [int(math.ceil(round(fraction / 2.0 * n, 9))) for n in prompt_lens]
    return tuple(half), tuple(half)


def ragged_prompt_lengths(batch: int, lo: int, hi: int, seed: int) -> Tuple[int, ...]:
    g = torch.Generator(device="cpu")
    g.manual_seed(_mix(seed, 0, 7, 0))
    return tuple(int(x) for x in torch.randint(lo, hi + 1, (batch,), generator=g))


def _mix(seed: int, layer: int, kind: int, step: int) -> int:
    """Derive an independent 63-bit stream seed from the four counters."""
    x = (seed * 0x9E3779B97F4A7C15 + layer * 0xBF58476D1CE4E5B9 + kind * 0x94D049BB133111EB + step * 0xD6E8FEB86659FD93) & (
        (1 << 64) - 1
    )
    x ^= x >> 31
    x = (x * 0x7FB5D329728EA185) & ((1 << 64) - 1)
    x ^= x >> 27
    return x & ((1 << 63) - 1)


def _head_directions(wl: Workload, layer: int) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(_mix(wl.seed, layer, 11, 0))
    u = torch.randn(wl.n_heads, wl.head_dim, generator=g, dtype=torch.float64)
    u = u / u.norm(dim=1, keepdim=True)
    return u.to(torch.float32)


def _outlier_mask(wl: Workload, layer: int, step: int, count: int) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(_mix(wl.seed, layer, 13, step))
    return torch.rand(count, generator=g) < OUTLIER_FRACTION


def _draw(wl: Workload, layer: int, kind: str, step: int, rows: int, device) -> torch.Tensor:
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(_mix(wl.seed, layer, _KIND[kind], step))
    return torch.randn(rows, wl.n_heads, wl.head_dim, generator=g, dtype=torch.float32, device=dev)


def _make(wl: Workload, layer: int, step: int, rows: int, device):
    u = _head_directions(wl, layer).to(device)
    mask = _outlier_mask(wl, layer, step, rows).to(device)
    q = _draw(wl, layer, "q", step, rows, device)
    q += QUERY_MEAN_SHIFT * u[None]
    q = q.to(wl.torch_dtype)
    k = _draw(wl, layer, "k", step, rows, device)
    k += (OUTLIER_KEY_SHIFT * mask.to(torch.float32))[:, None, None] * u[None]
    k = k.to(wl.torch_dtype)
    v = _draw(wl, layer, "v", step, rows, device).to(wl.torch_dtype)
    return q.contiguous(), k.contiguous(), v.contiguous()


def make_prompt_inputs(wl: Workload, layer: int = 0, device="cpu"):
    """q, k, v of shape ``[total_tokens, n_heads, head_dim]`` (token-major, ragged) and cu_seqlens."""
    q, k, v = _make(wl, layer, 0, wl.total_tokens, device)
    return q, k, v, wl.cu_seqlens()


def make_decode_inputs(wl: Workload, step: int, layer: int = 0, device="cpu"):
    """q, k_new, v_new of shape ``[batch, n_heads, head_dim]`` for decode step ``step`` (0-based)."""
    return _make(wl, layer, 1 + step, wl.batch, device)


def _uniform(name, batch, heads, d, dtype, n, steps, k, r, layers=1, seed=20230614) -> Workload:
    return Workload(name, batch, heads, d, dtype, (n,) * batch, steps, (k,) * batch, (r,) * batch, layers, seed)


def _config5() -> Workload:
    seed = 20230614 + 4
    lens = ragged_prompt_lengths(128, 128, 4096, seed)
    k, r = budgets_for(lens, 0.2)
    return Workload("c5_ragged_32layer", 128, 32, 128, "bf16", lens, 128, k, r, 32, seed)


CONFIGS = {
    "c1_tiny": _uniform("c1_tiny", 1, 4, 64, "f32", 256, 64, 32, 32, seed=20230614 + 0),
    "c2_opt6p7b": _uniform("c2_opt6p7b", 8, 32, 128, "bf16", 2048, 256, 205, 205, seed=20230614 + 1),
    "c3_opt30b": _uniform("c3_opt30b", 64, 56, 128, "bf16", 512, 32, 52, 52, seed=20230614 + 2),
    "c4_longctx": _uniform("c4_longctx", 1, 32, 128, "bf16", 32768, 512, 1024, 1024, seed=20230614 + 3),
    "c5_ragged_32layer": _config5(),
}
