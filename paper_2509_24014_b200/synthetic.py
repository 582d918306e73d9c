"""Seeded synthetic inputs shaped like the attention layers of LLaDA-8B / Dream-7B.

This module only draws random tensors and plants per-head structure in them. It holds
none of the method's arithmetic (no softmax, pooling, selection or attention), so both
the CUDA path and the CPU oracle can be fed from it without sharing any method code.

The planted structures mimic the head families the paper describes in its
"Observations" section (column-wise heads, sliding-window heads, mixed heads):

* ``band(w)``    - tokens are grouped in cells of ``w`` tokens; one random direction of
                   norm 3 per cell is added to the query rows and key rows of that cell,
                   which makes queries attend to keys of their own cell (a local band).
* ``sink(n)``    - one direction of norm 3 per head is added to every query row and to
                   the first ``n`` key rows (attention sinks = leading vertical stripe).
* ``stripes(m)`` - the same per-head direction is added to ``m`` seeded key rows
                   (single-token vertical stripes).
* ``diffuse``    - nothing planted: near-uniform attention, the near-tie stress case.

With grouped-query attention the key-side vectors of all query heads of a group are
summed into the shared key head.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class AttnConfig:
    name: str
    batch: int
    heads_q: int
    heads_kv: int
    seq_len: int
    head_dim: int
    block_size: int
    keep_ratio: float
    prefill_len: int = 0
    seed: int = 0
    total_steps: int = 1
    skip: float = 0.0
    layers: int = 1
    step_noise: float = 0.0
    hidden: int = 0  # > 0: Q/K/V come from random projections of a hidden state of this width
    fixed_heads: Optional[Tuple[Tuple[str, ...], ...]] = None
    plant_norm: float = 3.0  # L2 norm of the planted vectors: logit boost plant_norm^2 / sqrt(head_dim)

    @property
    def num_blocks(self) -> int:
        return self.seq_len // self.block_size

    def with_(self, **kw) -> "AttnConfig":
        return dataclasses.replace(self, **kw)


# The five workloads. c1 is the small exhaustive case, c2/c3 the LLaDA / Dream shapes,
# c4 the 64k pattern-reuse loop, c5 the 4-layer denoising schedule.
CONFIGS: Dict[str, AttnConfig] = {
    "c1": AttnConfig("c1", 1, 2, 2, 1024, 128, 64, 0.3, 0, seed=0,
                     fixed_heads=(("band", "128"), ("sink+stripes", "32", "4"))),
    "c2": AttnConfig("c2", 1, 32, 32, 8192, 128, 128, 0.2, 4096, seed=2),
    "c3": AttnConfig("c3", 1, 28, 4, 16384, 128, 128, 0.15, 0, seed=3),
    "c4": AttnConfig("c4", 1, 32, 32, 65536, 128, 128, 0.1, 0, seed=4, total_steps=64, skip=0.2,
                     step_noise=0.05),
    "c5": AttnConfig("c5", 1, 32, 32, 32768, 128, 128, 0.1, 16384, seed=5, total_steps=256, skip=0.25,
                     layers=4, hidden=4096),
}

def _gen(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for v in key:
        s = (s * 6364136223846793005 + int(v) + 1442695040888963407) % (1 << 63)
    g.manual_seed(s)
    return g


def head_kinds(cfg: AttnConfig, layer: int = 0) -> List[Tuple]:
    """Planted structure of each query head: a list of (kind, params...) tuples."""
    if cfg.fixed_heads is not None:
        out = []
        for spec in cfg.fixed_heads:
            if spec[0] == "band":
                out.append(("band", int(spec[1])))
            elif spec[0] == "sink+stripes":
                out.append(("sink+stripes", int(spec[1]), int(spec[2])))
            else:
                out.append(("diffuse",))
        return out
    g = _gen("cpu", cfg.seed, 101, layer)
    kinds = []
    for _ in range(cfg.heads_q):
        r = int(torch.randint(0, 4, (1,), generator=g))
        if r == 0:
            kinds.append(("band", int(torch.randint(64, 513, (1,), generator=g))))
        elif r == 1:
            kinds.append(("sink", int(torch.randint(16, 65, (1,), generator=g))))
        elif r == 2:
            kinds.append(("stripes", int(torch.randint(2, 17, (1,), generator=g))))
        else:
            kinds.append(("diffuse",))
    return kinds


def _direction(g: torch.Generator, shape, device, norm: float) -> torch.Tensor:
    u = torch.randn(*shape, generator=g, device=device, dtype=torch.float32)
    return u * (norm / u.norm(dim=-1, keepdim=True))


def _plant(cfg: AttnConfig, q: torch.Tensor, k: torch.Tensor, layer: int) -> None:
    """Adds the planted vectors in place to fp32 q [B,Hq,L,D] and k [B,Hkv,L,D]."""
    device = q.device
    group = cfg.heads_q // cfg.heads_kv
    L, D = cfg.seq_len, cfg.head_dim
    for h, kind in enumerate(head_kinds(cfg, layer)):
        g = _gen(device, cfg.seed, 202, layer, h)
        gc = _gen("cpu", cfg.seed, 203, layer, h)
        hk = h // group
        if kind[0] == "band":
            w = kind[1]
            cells = (L + w - 1) // w
            u = _direction(g, (cells, D), device, cfg.plant_norm)
            cell = torch.arange(L, device=device) // w
            q[:, h] += u[cell]
            k[:, hk] += u[cell]
        elif kind[0] in ("sink", "sink+stripes", "stripes"):
            a = _direction(g, (D,), device, cfg.plant_norm)
            q[:, h] += a
            if kind[0] != "stripes":
                k[:, hk, : kind[1]] += a
            m = kind[2] if kind[0] == "sink+stripes" else (kind[1] if kind[0] == "stripes" else 0)
            if m:
                pos = torch.randperm(L, generator=gc)[:m].to(device)
                k[:, hk, pos] += a


def make_base(cfg: AttnConfig, device="cpu", layer: int = 0):
    """fp32 base tensors (q [B,Hq,L,D], k, v [B,Hkv,L,D]) before rounding to bf16."""
    B, Hq, Hkv, L, D = cfg.batch, cfg.heads_q, cfg.heads_kv, cfg.seq_len, cfg.head_dim
    if cfg.hidden:
        # Q/K/V as seeded random projections of a seeded N(0,1) hidden state; the weight
        # variances make Q,K ~ N(0,1/D) and V ~ N(0,1) elementwise.
        W = cfg.hidden
        gx = _gen(device, cfg.seed, 301)
        x = torch.randn(B, L, W, generator=gx, device=device, dtype=torch.float32)
        gw = _gen(device, cfg.seed, 302, layer)
        wq = torch.randn(W, Hq * D, generator=gw, device=device, dtype=torch.float32) / math.sqrt(W * D)
        wk = torch.randn(W, Hkv * D, generator=gw, device=device, dtype=torch.float32) / math.sqrt(W * D)
        wv = torch.randn(W, Hkv * D, generator=gw, device=device, dtype=torch.float32) / math.sqrt(W)
        q = (x @ wq).view(B, L, Hq, D).transpose(1, 2).contiguous()
        k = (x @ wk).view(B, L, Hkv, D).transpose(1, 2).contiguous()
        v = (x @ wv).view(B, L, Hkv, D).transpose(1, 2).contiguous()
        del x, wq, wk, wv
    else:
        g = _gen(device, cfg.seed, 401, layer)
        q = torch.randn(B, Hq, L, D, generator=g, device=device, dtype=torch.float32) / math.sqrt(D)
        k = torch.randn(B, Hkv, L, D, generator=g, device=device, dtype=torch.float32) / math.sqrt(D)
        v = torch.randn(B, Hkv, L, D, generator=g, device=device, dtype=torch.float32)
    _plant(cfg, q, k, layer)
    return q, k, v


def make_qkv(cfg: AttnConfig, device="cpu", layer: int = 0, step: Optional[int] = None, base=None):
    """bf16 (q, k, v) for one layer. With ``cfg.step_noise`` > 0 and a ``step`` given, step t
    sees ``bf16(base + N(0, step_noise^2))`` with fresh noise keyed by t (not cumulative)."""
    if base is None:
        base = make_base(cfg, device, layer)
    out = []
    for i, t in enumerate(base):
        if cfg.step_noise > 0 and step is not None:
            g = _gen(t.device, cfg.seed, 501 + i, layer, step)
            # noise is drawn per head slice to bound the fp32 temporary at long sequences
            r = torch.empty_like(t, dtype=torch.bfloat16)
            for h in range(t.shape[1]):
                n = torch.randn(t[:, h].shape, generator=g, device=t.device, dtype=torch.float32)
                r[:, h] = (t[:, h] + cfg.step_noise * n).to(torch.bfloat16)
            out.append(r)
        else:
            out.append(t.to(torch.bfloat16))
    return tuple(out)


def random_scores(rows: int, nb: int, seed: int, device="cpu", ties: bool = False) -> torch.Tensor:
    """fp32 [rows, nb] positive pseudo block scores for exercising selection alone.
    With ``ties`` the values are quantised to a few levels so that many compare equal."""
    g = _gen(device, seed, 601)
    s = torch.rand(rows, nb, generator=g, device=device, dtype=torch.float32)
    if ties:
        s = torch.floor(s * 8) / 8
    return s
