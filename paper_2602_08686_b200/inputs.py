"""Seeded synthetic inputs for the retention pass (shared by the oracle tests and the CUDA tests).

This module only *builds inputs*: random Q/K/V with an attention sink and planted
needle keys, and random tables.  It contains none of the method's arithmetic
(no softmax, pooling, budgets, selection) and imports neither the oracle nor the
CUDA binding.

The inputs stand in for the long-context workloads the paper evaluates on
(needle-at-depth retrieval, 8k-128k prompts, a 512-row budget at 32k and the
fixed 512/32k ratio beyond): only their shapes and structure are taken.
Every unit (one sequence x layer pair) is drawn from its own generator seeded
with ``1000 * config_id + unit``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2


@dataclass(frozen=True)
class Config:
    name: str
    config_id: int
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    seq_len: int
    window: int
    pool_kind: int
    pool_size: int
    budget_per_head: int
    floor_per_head: int
    n_needles: int
    dtype: str = "bf16"           # "bf16" | "f32"
    head_dim: int = 128
    n_buckets: int = 16
    heavy_tail: bool = False      # Student-t(3) key scales
    stratified: bool = False      # needles spread uniformly in depth
    low_rel_group: bool = False   # one KV group per layer has reliability near 0.1

    @property
    def n_units(self) -> int:
        return self.n_layers * self.batch

    @property
    def n(self) -> int:
        return self.seq_len - self.window


# The five workload shapes (single layer fp32; Llama-3-8B shape at 32k; the same at
# batch 16; Llama-3.1-8B shape at 128k with heavy-tailed keys; Qwen2.5-7B shape).
CONFIGS = {
    "c1": Config("c1", 1, 1, 1, 8, 2, 2048, 32, POOL_MAX, 7, 512, 1, 8, dtype="f32"),
    "c2": Config("c2", 2, 32, 1, 32, 8, 32768, 32, POOL_MAX, 7, 512, 1, 32),
    "c3": Config("c3", 3, 32, 16, 32, 8, 32768, 32, POOL_MAX, 7, 512, 1, 32),
    "c4": Config("c4", 4, 32, 1, 32, 8, 131072, 32, POOL_MAX, 7, 2048, 1, 64, heavy_tail=True, stratified=True),
    "c5": Config("c5", 5, 28, 4, 28, 4, 4096, 64, POOL_AVG, 5, 128, 8, 8, low_rel_group=True),
}


def c5_point(seq_len: int, budget: int) -> Config:
    """One (L, B) point of the Qwen-shaped sweep: L in {4096, 16384, 65536}, B in {128, 512, 2048}."""
    return replace(CONFIGS["c5"], seq_len=seq_len, budget_per_head=budget)


def shrink(cfg: Config, **kw) -> Config:
    """A smaller case with the same structure (used by the parity tests)."""
    return replace(cfg, **kw)


def _needle_positions(cfg: Config, gen: torch.Generator, device) -> torch.Tensor:
    """[Hkv, n_needles] distinct positions in [1, n), at least pool_size apart."""
    n, nn, s = cfg.n, cfg.n_needles, max(cfg.pool_size, 1)
    out = []
    for _ in range(cfg.n_kv_heads):
        if cfg.stratified:
            # one needle per depth stratum; the draw stays away from the stratum edges
            u = 0.1 + 0.8 * torch.rand(nn, generator=gen, device=device)
            r = torch.arange(nn, device=device)
            p = ((r + u) * (n / nn)).floor().long().clamp_(1, n - 1)
        else:
            m = (n - 1) - (nn - 1) * (s - 1)
            if m < nn:
                raise ValueError("prefix too short for the requested needles")
            y = torch.randperm(m, generator=gen, device=device)[:nn].sort().values
            p = 1 + y + torch.arange(nn, device=device) * (s - 1)
        out.append(p)
    return torch.stack(out)


def make_unit(cfg: Config, unit: int, device="cpu"):
    """Q_win [H,W,d], K, V [Hkv,L,d] (cfg dtype), head_w [H] fp32, needle positions [Hkv,Nn] of one unit."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1000 * cfg.config_id + unit)
    H, Hkv, L, W, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.seq_len, cfg.window, cfg.head_dim
    G = H // Hkv
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    q = torch.randn(H, W, d, generator=gen, device=dev).to(tdt)
    k = torch.randn(Hkv, L, d, generator=gen, device=dev)
    v = torch.randn(Hkv, L, d, generator=gen, device=dev).to(tdt)
    qf = q.float().view(Hkv, G * W, d)

    if cfg.heavy_tail:
        z = torch.randn(Hkv, L, generator=gen, device=dev)
        chi = torch.randn(Hkv, L, 3, generator=gen, device=dev).pow(2).sum(-1) / 3.0
        x = z / chi.sqrt()
        scale = (x.abs() / (2.0 * math.sqrt(3.0) / math.pi)).clamp_(max=6.0)
        k = k * scale.unsqueeze(-1)

    # attention sink: key 0 points along the mean window query with 4x the typical norm
    qbar = qf.mean(1)
    k[:, 0, :] = 4.0 * math.sqrt(d) * qbar / qbar.norm(dim=-1, keepdim=True)

    # needles: cosine 0.9 to one window query of the group, norm sqrt(d).  The query is drawn from the half of the
    # group's rows that point least along the sink direction (a row that points along it hands the sink nearly all
    # of its attention, and a key planted for that row would not stand out), each row at most once where the group
    # has enough of them, so that two needles never split one row's attention.
    pos = _needle_positions(cfg, gen, dev)
    nn = cfg.n_needles
    along = (qf * (qbar / qbar.norm(dim=-1, keepdim=True)).unsqueeze(1)).sum(-1)
    eligible = along.argsort(dim=1)[:, :(G * W + 1) // 2]
    m = eligible.shape[1]
    if nn <= m:
        sel = torch.rand(Hkv, m, generator=gen, device=dev).argsort(dim=1)[:, :nn]
    else:
        sel = torch.randint(0, m, (Hkv, nn), generator=gen, device=dev)
    pick = torch.gather(eligible, 1, sel)
    qsel = torch.gather(qf, 1, pick.unsqueeze(-1).expand(Hkv, nn, d))
    qhat = qsel / qsel.norm(dim=-1, keepdim=True)
    z = torch.randn(Hkv, nn, d, generator=gen, device=dev)
    z = z - (z * qhat).sum(-1, keepdim=True) * qhat
    z = z / z.norm(dim=-1, keepdim=True)
    needle = math.sqrt(d) * (0.9 * qhat + math.sqrt(0.19) * z)
    k.scatter_(1, pos.unsqueeze(-1).expand(Hkv, nn, d), needle)
    k = k.to(tdt)

    head_w = 0.5 + torch.rand(H, generator=gen, device=dev)
    if cfg.low_rel_group:
        g_low = int(torch.randint(0, Hkv, (1,), generator=gen, device=dev).item())
        head_w[g_low * G:(g_low + 1) * G] = 0.05 + 0.1 * torch.rand(G, generator=gen, device=dev)
    return q, k, v, head_w.float(), pos


def make_sens(cfg: Config, device="cpu") -> torch.Tensor:
    """The threshold table shared by all units: [n_buckets] fp32 in U(0.8, 1.2)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1000 * cfg.config_id + 999)
    return (0.8 + 0.4 * torch.rand(cfg.n_buckets, generator=gen)).float().to(device)


def make_batch(cfg: Config, device="cpu", units=None):
    """Stacked inputs for ``units`` (default: all): dict with q [Nu,H,W,d], k, v [Nu,Hkv,L,d],
    head_w [Nu,H], sens [n_buckets], needles [Nu,Hkv,Nn]."""
    units = list(range(cfg.n_units)) if units is None else list(units)
    dev = torch.device(device)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    Nu = len(units)
    q = torch.empty(Nu, cfg.n_q_heads, cfg.window, cfg.head_dim, dtype=tdt, device=dev)
    k = torch.empty(Nu, cfg.n_kv_heads, cfg.seq_len, cfg.head_dim, dtype=tdt, device=dev)
    v = torch.empty_like(k)
    head_w = torch.empty(Nu, cfg.n_q_heads, dtype=torch.float32, device=dev)
    needles = torch.empty(Nu, cfg.n_kv_heads, cfg.n_needles, dtype=torch.long, device=dev)
    for j, u in enumerate(units):
        q[j], k[j], v[j], head_w[j], needles[j] = make_unit(cfg, u, dev)
    return dict(q=q, k=k, v=v, head_w=head_w, sens=make_sens(cfg, dev), needles=needles, units=units)


def as_numpy(t: torch.Tensor):
    """Host numpy view of a tensor; bf16 comes back as its uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
