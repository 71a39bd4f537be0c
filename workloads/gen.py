"""Seeded synthetic inputs for the compressed-KV decode path.

This module only draws numbers.  It contains none of the method's arithmetic
(no attention, no scoring, no budget split) and is the one piece of code both
the CPU oracle's tests and the CUDA path's tests/benchmark share.

Recipe (stands in for the paper's "synthetic datasets" used for its efficiency
measurements on LLaMA2-7B/13B shapes, Sec. 4.1/4.2): per (layer, kv-head) a unit
direction u; queries q = N(0, I) + c*u (the G queries of a group share u);
ordinary keys k = N(0, I); heavy-hitter keys -- position 0 and an iid 2 % of all
other positions, prompt and decode alike -- k = N(0, I) + c*u; values N(0, I);
c = sqrt(4*sqrt(d)), which puts a heavy hitter's expected logit 4 above an
ordinary token's unit-variance logit.  Everything is rounded once to the
storage dtype before anyone sees it.

Streams are torch generators seeded from (seed, layer, step).  A CPU generator
and a CUDA generator give different streams for the same seed: small cases are
drawn on the CPU and copied to the GPU; full-size cases are drawn on the GPU and
the units the oracle re-computes are copied to the host.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_TORCH_DTYPE = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}
HEAVY_FRACTION = 0.02


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str            # "f32" | "f16" | "bf16": storage type of q, k, v, out and token slots
    prompt_len: int
    decode_steps: int
    window: int           # prompt queries used for the initial scores
    budget: Optional[int]  # slots per head; None -> drawn per head (see head_budgets)
    seed: int
    budget_lo: int = 64
    budget_hi: int = 2048

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return _TORCH_DTYPE[self.dtype]

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five configurations the path is judged on.  c4 comes in three budgets.
C1 = Workload("c1_tiny", 1, 1, 4, 4, 64, "f32", 512, 64, 512, 64, 1)
C2 = Workload("c2_llama7b_layer", 1, 1, 32, 32, 128, "f16", 4096, 256, 32, 205, 2)
C3 = Workload("c3_llama7b_b16", 32, 16, 32, 32, 128, "f16", 16384, 512, 32, 819, 3)
C4_5 = Workload("c4_54k_5pct", 32, 1, 32, 32, 128, "f16", 54000, 1024, 32, 2700, 4)
C4_10 = Workload("c4_54k_10pct", 32, 1, 32, 32, 128, "f16", 54000, 1024, 32, 5400, 4)
C4_20 = Workload("c4_54k_20pct", 32, 1, 32, 32, 128, "f16", 54000, 1024, 32, 10800, 4)
C5 = Workload("c5_gqa_ragged", 32, 8, 32, 8, 128, "bf16", 32768, 512, 32, None, 5)

WORKLOADS = {w.name: w for w in (C1, C2, C3, C4_5, C4_10, C4_20, C5)}


def head_budgets(w: Workload) -> np.ndarray:
    """Total slots per (layer, kv-head), int32 [n_layers, n_kv_heads].

    Uniform when the workload fixes a budget; otherwise lo + round((hi-lo) *
    Beta(3.84, 1)), whose mean is about 5 % of a 32 768-token prompt for the
    default [64, 2048] range.
    """
    if w.budget is not None:
        return np.full((w.n_layers, w.n_kv_heads), int(w.budget), dtype=np.int32)
    rs = np.random.RandomState(w.seed)
    x = rs.beta(3.84, 1.0, size=(w.n_layers, w.n_kv_heads))
    return (w.budget_lo + np.rint((w.budget_hi - w.budget_lo) * x)).astype(np.int32)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _boost(w: Workload) -> float:
    return math.sqrt(4.0 * math.sqrt(float(w.head_dim)))


def directions(w: Workload, device="cpu") -> torch.Tensor:
    """Unit vectors u, fp32 [n_layers, n_kv_heads, d]."""
    g = _gen(device, w.seed * 1_000_003 + 17)
    u = torch.randn(w.n_layers, w.n_kv_heads, w.head_dim, generator=g, device=device)
    return u / u.norm(dim=-1, keepdim=True)


def prompt(w: Workload, layer: int, device="cpu", u: Optional[torch.Tensor] = None):
    """One layer's prompt: K, V [batch, n_kv_heads, T, d] and the last `window`
    queries Qw [batch, n_q_heads, W, d], all in the storage dtype."""
    if u is None:
        u = directions(w, device)
    ul = u[layer].to(device)                                   # [Hkv, d]
    g = _gen(device, w.seed * 1_000_003 + 7919 * (layer + 1) + 1)
    b, hk, hq, T, d, W = w.batch, w.n_kv_heads, w.n_q_heads, w.prompt_len, w.head_dim, w.window
    c = _boost(w)
    K = torch.randn(b, hk, T, d, generator=g, device=device)
    heavy = torch.rand(b, hk, T, generator=g, device=device) < HEAVY_FRACTION
    heavy[:, :, 0] = True
    K += heavy.unsqueeze(-1) * (c * ul)[None, :, None, :]
    K = K.to(w.torch_dtype)
    V = torch.randn(b, hk, T, d, generator=g, device=device).to(w.torch_dtype)
    Qw = torch.randn(b, hq, W, d, generator=g, device=device)
    Qw += (c * ul).repeat_interleave(w.group, dim=0)[None, :, None, :]
    return K, V, Qw.to(w.torch_dtype)


def decode_inputs(w: Workload, step: int, device="cpu", u: Optional[torch.Tensor] = None):
    """One decode step for every layer: q [L, batch, n_q_heads, d] and k_new,
    v_new [L, batch, n_kv_heads, d] in the storage dtype."""
    if u is None:
        u = directions(w, device)
    u = u.to(device)
    g = _gen(device, w.seed * 1_000_003 + 104_729 * (step + 1) + 2)
    L, b, hk, hq, d = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim
    c = _boost(w)
    q = torch.randn(L, b, hq, d, generator=g, device=device)
    q += (c * u).repeat_interleave(w.group, dim=1)[:, None, :, :]
    k = torch.randn(L, b, hk, d, generator=g, device=device)
    heavy = torch.rand(L, b, hk, generator=g, device=device) < HEAVY_FRACTION
    k += heavy.unsqueeze(-1) * (c * u)[:, None, :, :]
    v = torch.randn(L, b, hk, d, generator=g, device=device)
    dt = w.torch_dtype
    return q.to(dt), k.to(dt), v.to(dt)
