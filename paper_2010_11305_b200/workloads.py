"""Seeded synthetic workloads shaped like the paper's DLRM index streams.

This module only draws inputs (table sizes, bag lengths, bounded-Zipf row
indices, output gradients).  It holds none of the method's arithmetic and is
the one piece shared by the GPU path's tests/benchmark and the CPU oracle's
tests.  The streams stand in for the Criteo-Kaggle and internal datasets of
the paper (Section 4, Section 5), which skew heavily toward a few rows
(Figure 3: fewer than 20% of the rows take more than 80% of the accesses).

Recipe: rank k in 1..N is drawn with P(k) proportional to k^-a by inverse
transform on a float64 cumulative table; ranks map to row ids through a seeded
affine bijection so that hot rows are scattered over the table; "uniform"
streams draw rows directly.  Bag lengths are fixed, Poisson, or capped
Poisson.  Output gradients are i.i.d. Normal(0, 1e-2).  All draws come from a
torch.Generator seeded from (config seed, table, step), on whichever device
the stream lives (CPU and CUDA generators give different, equally valid,
streams; a test that compares two implementations draws once and copies).
"""
from dataclasses import dataclass, field, replace
from math import gcd
from typing import List, Optional, Tuple

import numpy as np
import torch

LRU, LFU = 0, 1
SGD, ROWWISE_ADAGRAD = 0, 1


@dataclass
class Config:
    name: str
    num_rows: List[int]
    dim: int
    bits: int
    cache_fraction: float
    ways: int
    policy: int
    optimizer: int
    lr: float
    batch: int
    bag: Tuple                      # ("fixed", k) | ("poisson", mean) | ("poisson_cap", mean, cap)
    zipf: List[Optional[float]]     # per-table exponent; None = uniform
    steps: int
    eps: float = 1e-8
    init_lo: float = -0.05
    init_hi: float = 0.05
    seed: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def num_tables(self):
        return len(self.num_rows)


def _cfg2_rows(seed=0, lo=3, hi=10_000_000, n=26, target=33_000_000, tol=0.05):
    rng = np.random.Generator(np.random.Philox(seed))
    while True:
        rows = np.exp(rng.uniform(np.log(lo), np.log(hi), n)).astype(np.int64)
        rows = np.clip(rows, lo, hi)
        if abs(int(rows.sum()) - target) <= tol * target:
            return [int(r) for r in rows]


def config(i: int) -> Config:
    """The five benchmark configurations (1-based)."""
    if i == 1:
        return Config("cfg1", [10_000], 16, 8, 0.05, 8, LRU, SGD, 0.01, 128, ("fixed", 4), [1.05], 10, seed=0)
    if i == 2:
        rows = _cfg2_rows(0)
        return Config("cfg2", rows, 16, 8, 0.05, 32, LFU, SGD, 0.1, 2048, ("fixed", 1), [1.1] * 26, 100, seed=2)
    if i == 3:
        return Config("cfg3", [20_000_000] * 8, 64, 4, 0.01, 16, LRU, ROWWISE_ADAGRAD, 0.05, 4096,
                      ("poisson", 20.0), [1.2] * 8, 50, seed=3)
    if i == 4:
        rng = np.random.Generator(np.random.Philox(4))
        alphas = [float(a) for a in rng.uniform(1.0, 1.3, 64)]
        return Config("cfg4", [5_000_000] * 64, 128, 4, 0.01, 32, LFU, SGD, 0.05, 16384,
                      ("poisson_cap", 30.0, 100), alphas, 20, seed=4)
    if i == 5:  # one point of the sweep; sweep() enumerates the rest
        return Config("cfg5", [10_000_000] * 4, 64, 8, 0.01, 32, LRU, SGD, 0.05, 8192, ("fixed", 10),
                      [1.05] * 4, 100, seed=5)
    raise ValueError(i)


def sweep5():
    """Every point of the policy/skew sweep (configuration 5)."""
    base = config(5)
    for bits in (8, 4):
        for frac in (0.005, 0.01, 0.05, 0.10):
            for policy in (LRU, LFU):
                for a in (None, 0.8, 1.05, 1.4):
                    name = f"cfg5-int{bits}-c{frac:g}-{'lru' if policy == LRU else 'lfu'}-{'uniform' if a is None else 'z%g' % a}"
                    yield replace(base, name=name, bits=bits, cache_fraction=frac, policy=policy, zipf=[a] * 4)


def scaled(cfg: Config, rows_div: int = 1, batch_div: int = 1, tables: Optional[int] = None, steps: Optional[int] = None) -> Config:
    """A smaller instance of a configuration with the same shape parameters (for CPU-sized parity cases)."""
    nt = cfg.num_tables if tables is None else min(tables, cfg.num_tables)
    rows = [max(3, r // rows_div) for r in cfg.num_rows[:nt]]
    return replace(cfg, name=f"{cfg.name}/r{rows_div}b{batch_div}t{nt}", num_rows=rows, zipf=cfg.zipf[:nt],
                   batch=max(1, cfg.batch // batch_div), steps=cfg.steps if steps is None else steps)


class Stream:
    """Index/gradient stream of one configuration on one torch device."""

    def __init__(self, cfg: Config, device="cpu"):
        self.cfg = cfg
        self.device = torch.device(device)
        self.cdf = []
        self.affine = []
        rng = np.random.Generator(np.random.Philox(cfg.seed * 1000 + 7))
        cache = {}
        for t, (n, a) in enumerate(zip(cfg.num_rows, cfg.zipf)):
            if a is None:
                self.cdf.append(None)
            else:
                key = (n, a)
                if key not in cache:
                    k = torch.arange(1, n + 1, dtype=torch.float64, device=self.device)
                    c = torch.cumsum(k.pow_(-a), 0)
                    c /= c[-1].clone()
                    cache[key] = c
                self.cdf.append(cache[key])
            mult = int(rng.integers(1, max(2, n)))
            while gcd(mult, n) != 1:
                mult += 1
            self.affine.append((mult, int(rng.integers(0, n))))

    def _gen(self, step, t, salt):
        g = torch.Generator(device=self.device)
        g.manual_seed(((self.cfg.seed * 1_000_003 + step) * 1009 + t) * 17 + salt)
        return g

    def bag_lengths(self, step, t):
        cfg, kind = self.cfg, self.cfg.bag[0]
        if kind == "fixed":
            return torch.full((cfg.batch,), int(cfg.bag[1]), dtype=torch.int64, device=self.device)
        lam = torch.full((cfg.batch,), float(cfg.bag[1]), dtype=torch.float32, device=self.device)
        n = torch.poisson(lam, generator=self._gen(step, t, 1)).to(torch.int64)
        if kind == "poisson_cap":
            n.clamp_(max=int(cfg.bag[2]))
        return n

    def batch(self, step):
        """-> (indices int32 [L], offsets int32 [T*B+1], grad_out float32 [B, T*dim]); table-major bags."""
        cfg = self.cfg
        idx, lens = [], []
        for t, n in enumerate(cfg.num_rows):
            ln = self.bag_lengths(step, t)
            total = int(ln.sum().item())
            g = self._gen(step, t, 2)
            if self.cdf[t] is None:
                rows = torch.randint(0, n, (total,), generator=g, device=self.device, dtype=torch.int64)
            else:
                u = torch.rand(total, generator=g, device=self.device, dtype=torch.float64)
                rank = torch.searchsorted(self.cdf[t], u, right=True).clamp_(max=n - 1)
                mult, add = self.affine[t]
                rows = (rank * mult + add) % n
            idx.append(rows.to(torch.int32))
            lens.append(ln)
        indices = torch.cat(idx) if idx else torch.zeros(0, dtype=torch.int32, device=self.device)
        offsets = torch.zeros(cfg.num_tables * cfg.batch + 1, dtype=torch.int64, device=self.device)
        torch.cumsum(torch.cat(lens), 0, out=offsets[1:])
        grad = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, dtype=torch.float32, device=self.device)
        grad.normal_(0.0, 1e-2, generator=self._gen(step, 0, 3))
        return indices.contiguous(), offsets.to(torch.int32).contiguous(), grad
