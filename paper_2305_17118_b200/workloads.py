"""Seeded synthetic input streams for the compressed decode-attention path.

This module only draws random tensors.  It contains none of the method's
arithmetic (no attention, no record, no eviction) and imports neither the CUDA
binding nor the CPU oracle, so both sides of a parity test can be fed from it.

The paper evaluates on OPT checkpoints running over text corpora; none of that
is available here, so the streams below stand in for it.  They are shaped like
the per-head tensors of OPT decoder layers and are built to show the two
properties the paper states for attention scores (Sections 3.1 and 3.2): a
heavy-tailed score distribution, and a small set of "pivotal" tokens that keep
receiving high scores from later queries.

Recipe, per unit (one (sequence, head) pair):
  * a fixed unit vector ``u`` (normalised N(0, I_d));
  * query at every step  ``q_t = rho * u + eps_t``, ``eps_t ~ N(0, I_d)``;
  * value ``v_t ~ N(0, I_d)``;
  * key   ``k_t = g_t + boost_t * u`` with ``g_t ~ N(0, I_d)`` and a
    kind-specific ``boost_t`` (see ``WorkloadConfig.kind``).
All tensors are rounded to the storage dtype here, before either
implementation sees them.  Each step is drawn from a generator seeded by
``(seed, step)``, so any step can be regenerated on its own; a given
(seed, step, device type) always gives the same bits, and parity tests move the
very same tensors to the other side instead of regenerating them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import torch

_TORCH_DTYPE = {
    "f32": torch.float32,
    "f16": torch.float16,
    "bf16": torch.bfloat16,
    "int4": torch.float16,  # int4 stores take fp16 inputs and quantise on append
}


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    """One synthetic workload: shapes, the method's parameters and the recipe.

    ``units`` is the number of independent (sequence, head) pairs handled by
    one handle (batch x heads).  ``layers`` handles of that size make up one
    "step" of the workload.  ``B, r, w, m`` are the paper's budget, recent
    window, history window and drop amount (Algorithms 1 and 2).
    """

    name: str
    units: int
    head_dim: int
    dtype: str  # "f32" | "f16" | "bf16" | "int4"
    B: int
    r: int
    w: int
    m: int
    prompt: int
    decode: int
    seed: int
    kind: str  # "pivot" | "heavy" | "zipf"
    layers: int = 1
    batch: int = 1
    heads: int = 1

    @property
    def torch_dtype(self) -> torch.dtype:
        return _TORCH_DTYPE[self.dtype]

    @property
    def total_steps(self) -> int:
        return self.prompt + self.decode

    def scaled(self, **kw) -> "WorkloadConfig":
        return dataclasses.replace(self, **kw)


# The five workloads of the benchmark definition.  Index 0 is the tiny case the
# oracle finishes at once; index 3 (OPT-66B-shaped, max batch) is the one the
# headline metric is quoted on.
CONFIGS = {
    "tiny": WorkloadConfig("tiny", units=2, head_dim=64, dtype="f32", B=64, r=8, w=16, m=16,
                           prompt=32, decode=224, seed=0, kind="pivot", batch=1, heads=2),
    "opt6b": WorkloadConfig("opt6b", units=8 * 32, head_dim=128, dtype="f16", B=410, r=64, w=128, m=64,
                            prompt=1024, decode=1024, seed=2000, kind="heavy", batch=8, heads=32),
    "opt13b": WorkloadConfig("opt13b", units=32 * 40, head_dim=128, dtype="bf16", B=512, r=128, w=256,
                             m=128, prompt=1536, decode=512, seed=3000, kind="zipf", layers=40,
                             batch=32, heads=40),
    "opt66b": WorkloadConfig("opt66b", units=128 * 72, head_dim=128, dtype="f16", B=410, r=64, w=128,
                             m=64, prompt=2048, decode=256, seed=4000, kind="heavy", batch=128, heads=72),
    "opt6b_int4": WorkloadConfig("opt6b_int4", units=8 * 32, head_dim=128, dtype="int4", B=410, r=64,
                                 w=128, m=64, prompt=1024, decode=1024, seed=2000, kind="heavy",
                                 batch=8, heads=32),
}
CONFIG_ORDER = ["tiny", "opt6b", "opt13b", "opt66b", "opt6b_int4"]

PIVOT_POSITIONS = (5, 11, 19, 27)  # 1-based stream positions of the "tiny" pivots
HEAVY_PROB = 0.02
ZIPF_A = 1.1
ZIPF_CAP = 10_000


def _zipf_cdf(device) -> torch.Tensor:
    """CDF of Zipf(a) on 1..ZIPF_CAP-1; mass beyond is clipped onto ZIPF_CAP."""
    k = torch.arange(1, ZIPF_CAP, dtype=torch.float64)
    pmf = k.pow(-ZIPF_A)
    # zeta(a) = sum_{k>=1} k^-a : partial sum plus the Euler-Maclaurin tail.
    n = float(ZIPF_CAP)
    tail = n ** (1 - ZIPF_A) / (ZIPF_A - 1) + 0.5 * n ** (-ZIPF_A) + ZIPF_A * n ** (-ZIPF_A - 1) / 12.0
    zeta = float(pmf.sum()) + tail
    return (pmf.cumsum(0) / zeta).to(device)


class Stream:
    """Input stream of one handle (one layer) of a workload."""

    def __init__(self, cfg: WorkloadConfig, device="cpu", layer: int = 0):
        self.cfg = cfg
        self.device = torch.device(device)
        self.layer = layer
        self.seed = cfg.seed + layer
        g = self._gen(0)
        u = torch.randn(cfg.units, cfg.head_dim, generator=g, device=self.device, dtype=torch.float32)
        self.u = u / u.norm(dim=1, keepdim=True)
        d = cfg.head_dim
        self.rho = d ** 0.25 if cfg.kind == "pivot" else 1.0
        self.scale = 1.0 / math.sqrt(d)
        self._cdf = _zipf_cdf(self.device) if cfg.kind == "zipf" else None

    def _gen(self, step: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed((self.seed * 1_000_003 + step) & 0x7FFFFFFFFFFF)
        return g

    def step(self, t: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """(q, k, v) of 1-based stream position ``t``; each ``[units, head_dim]``
        in the storage dtype, on ``self.device``."""
        cfg = self.cfg
        U, d = cfg.units, cfg.head_dim
        g = self._gen(t)
        eps = torch.randn(3, U, d, generator=g, device=self.device, dtype=torch.float32)
        q = self.rho * self.u + eps[0]
        k = eps[1]
        v = eps[2]
        if cfg.kind == "pivot":
            if t in PIVOT_POSITIONS:
                k = k + 3.0 * self.rho * self.u
        elif cfg.kind == "heavy":
            hit = torch.rand(U, 1, generator=g, device=self.device) < HEAVY_PROB
            k = k + hit.to(torch.float32) * (4.0 * math.sqrt(d)) * self.u
        elif cfg.kind == "zipf":
            x = torch.rand(U, generator=g, device=self.device, dtype=torch.float64)
            z = torch.searchsorted(self._cdf, x).to(torch.float32) + 1.0  # 1..ZIPF_CAP
            k = k + (torch.log(z) * math.sqrt(d) / self.rho).unsqueeze(1) * self.u
        else:
            raise ValueError(cfg.kind)
        dt = cfg.torch_dtype
        return q.to(dt).contiguous(), k.to(dt).contiguous(), v.to(dt).contiguous()

    def block(self, t0: int, t1: int):
        """Steps ``t0 .. t1-1`` stacked time-major: three ``[t1-t0, units, head_dim]``."""
        qs, ks, vs = zip(*(self.step(t) for t in range(t0, t1)))
        return torch.stack(qs), torch.stack(ks), torch.stack(vs)


def sample_units(cfg: WorkloadConfig, count: int, seed: int = 12345) -> torch.Tensor:
    """A fixed, sorted sample of unit indices that always contains the first
    and the last unit (units are independent, so any subset can be checked)."""
    U = cfg.units
    if count >= U:
        return torch.arange(U)
    g = torch.Generator()
    g.manual_seed(seed)
    perm = torch.randperm(U - 2, generator=g)[: max(count - 2, 0)] + 1
    return torch.cat([torch.tensor([0, U - 1]), perm]).sort().values


def random_stream(units: int, head_dim: int, steps: int, seed: int, dtype: str = "f32",
                  peaked: float = 0.0, device="cpu"):
    """Plain N(0,1) q, k, v for small tests: three ``[steps, units, head_dim]``
    tensors in the storage dtype.  ``peaked`` > 0 adds ``peaked * u`` to every
    query and to a random 10 % of keys so the scores are not flat."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    x = torch.randn(3, steps, units, head_dim, generator=g, device=device, dtype=torch.float32)
    q, k, v = x[0], x[1], x[2]
    if peaked:
        u = torch.randn(units, head_dim, generator=g, device=device)
        u = u / u.norm(dim=1, keepdim=True)
        hit = (torch.rand(steps, units, 1, generator=g, device=device) < 0.1).to(torch.float32)
        q = q + peaked * u
        k = k + hit * peaked * math.sqrt(head_dim) * u
    dt = _TORCH_DTYPE[dtype]
    return q.to(dt).contiguous(), k.to(dt).contiguous(), v.to(dt).contiguous()
