"""Seeded synthetic inputs for the CaDDTree hot path (draft logits, cost models, target logits).

This module only *draws inputs*: it contains none of the method's arithmetic (no softmax,
no top-K, no tree logic).  Both the CUDA path and the CPU oracle are fed the identical
bits produced here.  The shapes follow the paper's workloads (block size L=16, bf16,
Qwen3-sized vocabulary V=151936, node caps up to 1024; Section 5 "Setup" and Table 2);
the values are Gaussian noise plus one planted ("confident") token per draft position.

Recipe, per request b and position index d = 0..L-1 (depth d+1 in the tree):
    x[b,d,:]          = sigma[b,d] * N(0,1)            (fp32)
    planted[b,d]      ~ U{0..V-1}
    x[b,d,planted]   += boost[b,d] * decay**d
    cast to the config dtype (round to nearest even)
Target logits for a built tree, per row j with depth e = depth[b,j] (padding rows use e=0):
    y[b,j,:]          = sigma[b,min(e,L-1)] * N(0,1)
    if e < l_eff[b]:  with probability `agreement` boost planted[b,e] (the drafter's token
                      for the next position), otherwise boost a uniformly drawn other token;
                      boost = target_boost (if given) else boost[b,e] * decay**e
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import torch

COST_QUADRATIC = 0
COST_TABLE = 1
COST_TABLE_INTERP = 2


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    index: int                 # 1-based position in the list of benchmark configurations
    batch: int
    L: int
    V: int
    dtype: str                 # "bf16" | "fp32"
    K: int
    B_max: int
    sigma: Tuple[float, float]           # sigma ~ U[lo, hi] per (b, d); lo == hi -> constant
    boost: Tuple[float, float]           # boost ~ U[lo, hi] per (b, d)
    decay: float
    t_draft: float
    cost_abc: Tuple[float, float, float]  # C_v(B) = a + b*B + c*B^2
    agreement: float
    target_boost: Optional[float] = None  # fixed target boost (config 1) or None = "same generator"
    regimes: Optional[Tuple[Tuple[float, float], ...]] = None   # per-request boost ranges, b mod len
    cost_step: Optional[Tuple[int, float]] = None   # (B0, step): +step for B >= B0, convexified
    l_eff_range: Optional[Tuple[int, int]] = None   # L_eff ~ U{lo..hi} per request
    cost_jitter: float = 0.0                        # each of a,b,c times U[1-j, 1+j] per request
    fixed_budget: bool = False                      # expansion ignores the stopping rule

    @property
    def R(self) -> int:
        """Row capacity of the per-request node arrays: root row + B_max draft nodes."""
        return self.B_max + 1

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4


_V_QWEN = 151936

CONFIGS = {
    "c1": WorkloadConfig("c1", 1, batch=1, L=8, V=1024, dtype="fp32", K=4, B_max=32,
                         sigma=(1.0, 1.0), boost=(6.0, 6.0), decay=0.8, t_draft=1.0,
                         cost_abc=(2.0, 0.01, 0.0005), agreement=0.7, target_boost=5.0),
    "c2": WorkloadConfig("c2", 2, batch=32, L=16, V=_V_QWEN, dtype="bf16", K=8, B_max=256,
                         sigma=(1.0, 4.0), boost=(2.0, 10.0), decay=0.85, t_draft=0.3,
                         cost_abc=(1.0, 0.002, 0.00002), agreement=0.6),
    "c3": WorkloadConfig("c3", 3, batch=128, L=16, V=_V_QWEN, dtype="bf16", K=16, B_max=512,
                         sigma=(1.0, 4.0), boost=(0.0, 0.0), decay=0.85, t_draft=0.25,
                         cost_abc=(1.0, 0.0015, 0.00001), agreement=0.6,
                         regimes=((8.0, 12.0), (3.0, 6.0), (0.0, 0.0)), cost_step=(256, 0.5)),
    "c4": WorkloadConfig("c4", 4, batch=64, L=32, V=_V_QWEN, dtype="bf16", K=32, B_max=1024,
                         sigma=(1.0, 1.0), boost=(0.0, 2.0), decay=1.0, t_draft=0.2,
                         cost_abc=(1.0, 0.0005, 0.000002), agreement=0.6),
    "c4_stress": WorkloadConfig("c4_stress", 4, batch=64, L=32, V=_V_QWEN, dtype="bf16", K=32,
                                B_max=1024, sigma=(1.0, 1.0), boost=(0.0, 2.0), decay=1.0,
                                t_draft=0.2, cost_abc=(1.0, 0.0005, 0.000002), agreement=0.6,
                                fixed_budget=True),
    "c5": WorkloadConfig("c5", 5, batch=256, L=16, V=_V_QWEN, dtype="bf16", K=8, B_max=384,
                         sigma=(1.0, 1.0), boost=(0.0, 12.0), decay=0.9, t_draft=0.3,
                         cost_abc=(1.0, 0.002, 0.00002), agreement=0.6,
                         l_eff_range=(4, 16), cost_jitter=0.2),
}


def scaled(cfg: WorkloadConfig, **kw) -> WorkloadConfig:
    """A copy of a config with some fields replaced (used for reduced-size test cases)."""
    d = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    d.update(kw)
    return WorkloadConfig(**d)


def config_seed(cfg: WorkloadConfig, round_idx: int = 0) -> int:
    """seed = 1000 * config + round; config 1 uses seed 0 as the benchmark list states."""
    return 0 if (cfg.index == 1 and round_idx == 0) else 1000 * cfg.index + round_idx


@dataclass
class DraftInputs:
    logits: torch.Tensor      # [batch, L, V], cfg dtype
    planted: torch.Tensor     # [batch, L] int64 (cpu)
    sigma: torch.Tensor       # [batch, L] float64 (cpu)
    boost: torch.Tensor       # [batch, L] float64 (cpu), already multiplied by decay**d
    l_eff: torch.Tensor       # [batch] int32 (cpu)
    bonus_token: torch.Tensor  # [batch] int32 (cpu)
    ctx_len: torch.Tensor     # [batch] int32 (cpu)


@dataclass
class CostInputs:
    kind: int
    coef: Optional[torch.Tensor] = None       # [batch, 4] float64: t_draft, a, b, c
    table: Optional[torch.Tensor] = None      # [n_tables, B_max+1] float64
    table_idx: Optional[torch.Tensor] = None  # [batch] int32
    t_draft: Optional[torch.Tensor] = None    # [batch] float64


def _uniform(g: torch.Generator, shape, lo: float, hi: float) -> torch.Tensor:
    u = torch.rand(shape, generator=g, dtype=torch.float64)
    return lo + (hi - lo) * u


def make_draft_inputs(cfg: WorkloadConfig, seed: int, device: str = "cpu") -> DraftInputs:
    """Draft logits [batch, L, V] and the parameters they were drawn from."""
    gp = torch.Generator(device="cpu").manual_seed(seed)          # parameters (tiny, always CPU)
    gn = torch.Generator(device=device).manual_seed(seed + 7919)  # noise (on the target device)
    B, L, V = cfg.batch, cfg.L, cfg.V
    sigma = _uniform(gp, (B, L), *cfg.sigma)
    if cfg.regimes is not None:
        boost = torch.empty(B, L, dtype=torch.float64)
        for b in range(B):
            lo, hi = cfg.regimes[b % len(cfg.regimes)]
            boost[b] = _uniform(gp, (L,), lo, hi)
    else:
        boost = _uniform(gp, (B, L), *cfg.boost)
    d = torch.arange(L, dtype=torch.float64)
    boost = boost * (cfg.decay ** d)[None, :]
    planted = torch.randint(0, V, (B, L), generator=gp, dtype=torch.int64)
    if cfg.l_eff_range is not None:
        lo, hi = cfg.l_eff_range
        l_eff = torch.randint(lo, hi + 1, (B,), generator=gp, dtype=torch.int64).to(torch.int32)
    else:
        l_eff = torch.full((B,), L, dtype=torch.int32)
    bonus = torch.randint(0, V, (B,), generator=gp, dtype=torch.int64).to(torch.int32)
    ctx = torch.randint(0, 8192, (B,), generator=gp, dtype=torch.int64).to(torch.int32)

    logits = torch.empty(B, L, V, dtype=cfg.torch_dtype, device=device)
    sig_dev = sigma.to(device=device, dtype=torch.float32)
    boost_dev = boost.to(device=device, dtype=torch.float32)
    planted_dev = planted.to(device)
    rows = torch.arange(L, device=device)
    for b in range(B):
        x = torch.randn(L, V, generator=gn, dtype=torch.float32, device=device)
        x *= sig_dev[b][:, None]
        x[rows, planted_dev[b]] += boost_dev[b]
        logits[b] = x.to(cfg.torch_dtype)
    return DraftInputs(logits, planted, sigma, boost, l_eff, bonus, ctx)


def convex_step_table(abc: Tuple[float, float, float], B0: int, step: float, B_max: int) -> torch.Tensor:
    """C_v(B) = max(c0(B), g(B)) for B = 0..B_max, with c0 the quadratic, g = c0 + step for
    B >= B0 and, left of B0, the tangent of c0 + step at B0 (a maximum of convex functions)."""
    a, b, c = abc
    n = torch.arange(B_max + 1, dtype=torch.float64)
    c0 = a + b * n + c * n * n
    c0_B0 = a + b * B0 + c * B0 * B0
    slope = b + 2.0 * c * B0
    g = torch.where(n >= B0, c0 + step, c0_B0 + step + slope * (n - B0))
    return torch.maximum(c0, g)


def make_cost_inputs(cfg: WorkloadConfig, seed: int) -> CostInputs:
    g = torch.Generator(device="cpu").manual_seed(seed + 104729)
    B = cfg.batch
    if cfg.cost_step is not None:
        table = convex_step_table(cfg.cost_abc, cfg.cost_step[0], cfg.cost_step[1], cfg.B_max)[None, :]
        return CostInputs(COST_TABLE, table=table.contiguous(),
                          table_idx=torch.zeros(B, dtype=torch.int32),
                          t_draft=torch.full((B,), cfg.t_draft, dtype=torch.float64))
    coef = torch.empty(B, 4, dtype=torch.float64)
    coef[:, 0] = cfg.t_draft
    abc = torch.tensor(cfg.cost_abc, dtype=torch.float64)
    if cfg.cost_jitter > 0.0:
        j = _uniform(g, (B, 3), 1.0 - cfg.cost_jitter, 1.0 + cfg.cost_jitter)
        coef[:, 1:] = abc[None, :] * j
    else:
        coef[:, 1:] = abc[None, :]
    return CostInputs(COST_QUADRATIC, coef=coef)


def make_target_logits(cfg: WorkloadConfig, seed: int, draft: DraftInputs, depth: torch.Tensor,
                       device: str = "cpu", out: Optional[torch.Tensor] = None,
                       row_chunk: int = 128) -> torch.Tensor:
    """Target logits [batch, R, V] for a built tree whose per-row depths are `depth` [batch, R]."""
    B, L, V = cfg.batch, cfg.L, cfg.V
    R = depth.shape[1]
    gp = torch.Generator(device="cpu").manual_seed(seed + 15485863)
    gn = torch.Generator(device=device).manual_seed(seed + 32452843)
    depth = depth.to("cpu", torch.int64).clamp(min=0)
    e = depth.clamp(max=L - 1)
    agree = torch.rand((B, R), generator=gp, dtype=torch.float64) < cfg.agreement
    other = torch.randint(0, V - 1, (B, R), generator=gp, dtype=torch.int64)
    bidx = torch.arange(B)[:, None].expand(B, R)
    plant_e = draft.planted[bidx, e]
    other = other + (other >= plant_e).to(torch.int64)       # uniform over tokens != planted
    tok = torch.where(agree, plant_e, other)
    live = depth < draft.l_eff.to(torch.int64)[:, None]
    if cfg.target_boost is not None:
        bst = torch.full((B, R), float(cfg.target_boost), dtype=torch.float64)
    else:
        bst = draft.boost[bidx, e]
    bst = torch.where(live, bst, torch.zeros_like(bst))
    sig = draft.sigma[bidx, e]

    if out is None:
        out = torch.empty(B, R, V, dtype=cfg.torch_dtype, device=device)
    for b in range(B):
        for r0 in range(0, R, row_chunk):
            r1 = min(R, r0 + row_chunk)
            y = torch.randn(r1 - r0, V, generator=gn, dtype=torch.float32, device=device)
            y *= sig[b, r0:r1].to(device=device, dtype=torch.float32)[:, None]
            y[torch.arange(r1 - r0, device=device), tok[b, r0:r1].to(device)] += \
                bst[b, r0:r1].to(device=device, dtype=torch.float32)
            out[b, r0:r1] = y.to(cfg.torch_dtype)
    return out


def make_context_cost_tables(B_max: int, grid=(0, 1024, 2048, 3072, 4096, 5120, 6144, 7168, 8192),
                             abc: Tuple[float, float, float] = (1.0, 0.002, 0.00002)):
    """Verification-cost tables at a grid of context lengths, shaped like the paper's profile (Figure 3:
    convex and increasing in the node count; longer contexts shift the curve up and steepen it).
    Returns (tables [len(grid), B_max+1] float64, grid int32)."""
    a, b, c = abc
    n = torch.arange(B_max + 1, dtype=torch.float64)
    rows = []
    for j, _ in enumerate(grid):
        rows.append(a * (1.0 + 0.10 * j) + b * (1.0 + 0.15 * j) * n + c * (1.0 + 0.10 * j) * n * n)
    return torch.stack(rows), torch.tensor(grid, dtype=torch.int32)
