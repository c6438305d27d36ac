"""Seeded synthetic KV caches shaped like the paper's workloads.

This module only draws inputs: random bf16 tensors with the shapes of the
models the paper evaluates (Section 3.1: Llama-3.1-8B, Llama-3-8B-ProLong-512k,
Qwen2.5-7B) and with a planted sparsity structure standing in for the attention
sparsity the paper observes on real prompts.  It contains none of the method's
arithmetic, imports neither the CUDA binding nor the CPU oracle, and serves
both: whatever tensor it returns is the single source of truth for a test (the
oracle reads a host copy of the very same bits).

Structure of a layer (per batch element, per KV head g):
  K, V ~ N(0,1) rounded to bf16; q_last ~ N(0,1).
  "Heavy" tokens: positions in the eviction region whose key is
  4*q_hat + N(0, sigma=0.5), q_hat the unit-normalised last-token query of one
  of the KV head's G query heads (planted token number j uses head g*G + j%G),
  so that head's logit there is about 4*|q|/sqrt(d) ~ 4 above the background.
  Placement by `structure`:
    "count"      a fixed number per KV head, uniform without replacement
    "fraction"   a fixed fraction of the eviction region, uniform
    "varfrac"    a fraction drawn per KV head from U(lo, hi)
    "spans"      the fraction is laid out as n_spans contiguous runs
    "dups"       "fraction" plus near-duplicate key pairs: for a share of the
                 positions K[i'] := K[i] (exact ties); for an equal share K[i']
                 is K[i] with one lane moved by one bf16 ulp (near ties).  Half
                 of the pairs copy a heavy token so ties straddle the k-th score.
"""

from __future__ import annotations

from dataclasses import dataclass, field, replace

import torch

__all__ = ["Workload", "WORKLOADS", "workload", "make_layer", "make_decode_inputs"]


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    n_ctx: int            # N, the last token included
    budget: int           # B = S + G*k_q + R
    n_init: int           # S
    n_recent_min: int     # R before the non-divisible remainder is added
    decode_steps: int
    structure: str
    heavy: tuple = ()     # parameters of `structure`
    seed: int = 0x5A6E0000

    @property
    def G(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def k_q(self) -> int:
        """Tokens kept per query head: the selected slots of a KV head divided
        evenly among its G query heads (Appendix A.2 fixes k per query head)."""
        return (self.budget - self.n_init - self.n_recent_min) // self.G

    @property
    def n_sel(self) -> int:
        return self.G * self.k_q

    @property
    def n_recent(self) -> int:
        """Slots left over by a non-divisible split go to the recent window,
        as in the appendix's Qwen example."""
        return self.budget - self.n_init - self.n_sel

    @property
    def E(self) -> int:
        return self.n_ctx - 1 - self.n_init - self.n_recent

    @property
    def L(self) -> int:
        return self.budget + 1

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    # one layer, Llama-3.1-8B head shape, 4K context, budget 512
    "C1": Workload("C1", 1, 32, 8, 128, 1, 4096, 512, 4, 64, 16, "count", (32,), 0x5A6E0001),
    # Llama-3.1-8B stack, 32K context, budget 2048
    "C2": Workload("C2", 32, 32, 8, 128, 1, 32768, 2048, 4, 128, 256, "fraction", (0.01,), 0x5A6E0002),
    # Llama-3.1-8B stack, 128K context, budgets 1024 / 2048 / 4096
    "C3-1024": Workload("C3-1024", 32, 32, 8, 128, 1, 131072, 1024, 4, 128, 512, "varfrac", (0.001, 0.02), 0x5A6E0003),
    "C3-2048": Workload("C3-2048", 32, 32, 8, 128, 1, 131072, 2048, 4, 128, 512, "varfrac", (0.001, 0.02), 0x5A6E0003),
    "C3-4096": Workload("C3-4096", 32, 32, 8, 128, 1, 131072, 4096, 4, 128, 512, "varfrac", (0.001, 0.02), 0x5A6E0003),
    # Qwen2.5-7B stack (G = 7), 128K context, budget 2048, batch 1 and 4
    "C4-b1": Workload("C4-b1", 28, 28, 4, 128, 1, 131072, 2048, 4, 128, 256, "dups", (0.01, 0.005), 0x5A6E0004),
    "C4-b4": Workload("C4-b4", 28, 28, 4, 128, 4, 131072, 2048, 4, 128, 256, "dups", (0.01, 0.005), 0x5A6E0004),
    # ProLong-512K-style Llama-3-8B stack, 512K context, budgets 4096 / 8192
    "C5-4096": Workload("C5-4096", 32, 32, 8, 128, 1, 524288, 4096, 4, 256, 512, "spans", (0.01, 8), 0x5A6E0005),
    "C5-8192": Workload("C5-8192", 32, 32, 8, 128, 1, 524288, 8192, 4, 256, 512, "spans", (0.01, 8), 0x5A6E0005),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


def _gen(device, *keys: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in keys:
        s = (s ^ (int(k) + 0x9E3779B97F4A7C15 + ((s << 6) & (2**64 - 1)) + (s >> 2))) & (2**63 - 1)
    g.manual_seed(s)
    return g


def _heavy_positions(w: Workload, gen: torch.Generator, device) -> list:
    """Planted positions per KV head (1-D int64 tensors, absolute, in the eviction region)."""
    S, E = w.n_init, w.E
    out = []
    for _ in range(w.n_kv_heads):
        if E <= 0:
            out.append(torch.zeros(0, dtype=torch.int64, device=device))
            continue
        if w.structure == "count":
            n = min(int(w.heavy[0]), E)
            pos = torch.randperm(E, generator=gen, device=device)[:n]
        elif w.structure in ("fraction", "dups"):
            n = max(1, int(round(w.heavy[0] * E)))
            pos = torch.randperm(E, generator=gen, device=device)[:n]
        elif w.structure == "varfrac":
            lo, hi = w.heavy
            u = torch.rand(1, generator=gen, device=device).item()
            n = max(1, int(round((lo + (hi - lo) * u) * E)))
            pos = torch.randperm(E, generator=gen, device=device)[:n]
        elif w.structure == "spans":
            frac, n_spans = w.heavy
            span = max(1, int(round(frac * E / n_spans)))
            starts = torch.randint(0, max(1, E - span), (int(n_spans),), generator=gen, device=device)
            pos = (starts[:, None] + torch.arange(span, device=device)[None, :]).reshape(-1)
            pos = torch.unique(pos.clamp_(max=E - 1))
        else:
            raise ValueError(w.structure)
        out.append(pos.to(torch.int64) + S)
    return out


def make_layer(w: Workload, layer: int, device="cpu") -> dict:
    """One layer's prefilled cache and last-token query.

    Returns {"q_last": bf16 [B, H_q, d], "K": bf16 [B, H_kv, N, d], "V": same,
    "heavy": list over batch of lists over KV heads of planted positions}.
    """
    device = torch.device(device)
    gen = _gen(device, w.seed, layer, 1)
    B, Hq, Hkv, N, d, G = w.batch, w.n_q_heads, w.n_kv_heads, w.n_ctx, w.head_dim, w.G
    q = torch.randn(B, Hq, d, generator=gen, device=device, dtype=torch.float32)
    K = torch.empty(B, Hkv, N, d, device=device, dtype=torch.bfloat16)
    V = torch.empty(B, Hkv, N, d, device=device, dtype=torch.bfloat16)
    for b in range(B):
        for g in range(Hkv):
            K[b, g] = torch.randn(N, d, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
            V[b, g] = torch.randn(N, d, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    q_bf = q.to(torch.bfloat16)
    q_hat = q_bf.float()
    q_hat = q_hat / q_hat.norm(dim=-1, keepdim=True)
    heavy_all = []
    for b in range(B):
        heavy = _heavy_positions(w, gen, device)
        heavy_all.append(heavy)
        for g in range(Hkv):
            pos = heavy[g]
            n = pos.numel()
            if n == 0:
                continue
            owner = g * G + (torch.arange(n, device=device) % G)
            noise = torch.randn(n, d, generator=gen, device=device, dtype=torch.float32) * 0.5
            K[b, g, pos] = (4.0 * q_hat[b, owner] + noise).to(torch.bfloat16)
        if w.structure == "dups" and w.E > 4:
            S, E = w.n_init, w.E
            n_pairs = max(2, int(round(w.heavy[1] * E)))
            for g in range(Hkv):
                src_bg = torch.randint(0, E, (n_pairs,), generator=gen, device=device) + S
                hv = heavy[g]
                pick = torch.randint(0, max(1, hv.numel()), (n_pairs,), generator=gen, device=device)
                src_hv = hv[pick] if hv.numel() else src_bg
                use_hv = (torch.arange(n_pairs, device=device) % 2) == 0
                src = torch.where(use_hv, src_hv, src_bg)
                dst = torch.randint(0, E, (n_pairs,), generator=gen, device=device) + S
                rows = K[b, g, src].clone()
                near = (torch.arange(n_pairs, device=device) % 4) >= 2
                lane = torch.randint(0, d, (n_pairs,), generator=gen, device=device)
                bits = rows.view(torch.int16)
                bump = torch.zeros_like(bits)
                bump[torch.arange(n_pairs, device=device), lane] = near.to(torch.int16)
                rows = (bits + bump).view(torch.bfloat16)
                K[b, g, dst] = rows
    return {"q_last": q_bf, "K": K, "V": V, "heavy": heavy_all}


def make_decode_inputs(w: Workload, layer: int, step: int, device="cpu") -> dict:
    """Random q / k_new / v_new ~ N(0,1) for decode step `step` of `layer`."""
    device = torch.device(device)
    gen = _gen(device, w.seed, layer, 2, step)
    B, Hq, Hkv, d = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    mk = lambda h: torch.randn(B, h, d, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    return {"q": mk(Hq), "k_new": mk(Hkv), "v_new": mk(Hkv)}
