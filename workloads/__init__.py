"""Seeded synthetic inputs for the TT-embedding gather: table shapes, TT-cores, index streams, bags.

This module holds no arithmetic of the method (no digit decomposition, no contraction, no pooling).
It only draws random numbers.  Both the CPU oracle's tests and the CUDA path's tests/benchmark take
their inputs from here, so the two sides always see the same arrays.

Conventions
-----------
* A table has N rows, row factors n = (n_1..n_K) with prod(n) >= N, dim factors d = (d_1..d_K) with
  prod(d) = D, ranks r = (r_0=1, r_1, .., r_K=1).
* Cores are returned in the index order G_k[r_{k-1}, n_k, d_k, r_k] (C-contiguous fp32).  Values are
  drawn in fp64 and rounded to fp32 once; the fp32 values are the ground truth for everyone.
* `indices` is int64[L], table-major (all bags of table 0, then table 1, ...); `offsets` is
  int64[T*B+1] with offsets[0] = 0 and offsets[T*B] = L (CSR over (table, bag)).
* The index stream of a table is a bounded Zipf law: P(rank = k) proportional to k**(-alpha) for
  k = 1..N, sampled by inverse CDF on an fp64 cumulative table.  rank -> row is either the identity
  (row = k-1) or "scattered" (row = a*(k-1) mod N with a coprime to N).
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

BASE_SEED = 260903459


@dataclass
class TableSpec:
    N: int
    n: Tuple[int, ...]
    d: Tuple[int, ...]
    r: Tuple[int, ...]
    alpha: float
    core_dist: str  # "uniform" (half-width = core_scale) or "normal" (std = core_scale)
    core_scale: float

    @property
    def K(self) -> int:
        return len(self.n)

    @property
    def D(self) -> int:
        return int(np.prod(self.d))


@dataclass
class Workload:
    name: str
    tables: List[TableSpec]
    B: int
    indices: np.ndarray  # int64 [L]
    offsets: np.ndarray  # int64 [T*B+1]
    cores: List[List[np.ndarray]]  # [T][K] fp32, shape (r_{k-1}, n_k, d_k, r_k)
    grad_out: Optional[np.ndarray] = None  # fp32 [B, T*D] for the training configuration
    lr: float = 0.01
    mapping: str = "identity"
    meta: dict = field(default_factory=dict)

    @property
    def T(self) -> int:
        return len(self.tables)

    @property
    def L(self) -> int:
        return int(self.indices.shape[0])

    @property
    def D(self) -> int:
        return self.tables[0].D

    def table_slice(self, t: int) -> Tuple[np.ndarray, np.ndarray]:
        """(indices, offsets rebased to 0) of table t alone."""
        o = self.offsets[t * self.B:(t + 1) * self.B + 1]
        return self.indices[o[0]:o[-1]], o - o[0]


def _scatter_multiplier(N: int) -> int:
    a = 2654435761 % N
    if a < 2:
        a = 2
    while math.gcd(a, N) != 1:
        a += 1
    return a


def zipf_rows(rng: np.random.Generator, N: int, alpha: float, size: int, mapping: str = "identity") -> np.ndarray:
    """`size` row ids in [0, N) whose popularity rank follows a bounded Zipf(alpha) law."""
    cdf = np.arange(1, N + 1, dtype=np.float64)
    np.power(cdf, -float(alpha), out=cdf)
    np.cumsum(cdf, out=cdf)
    cdf /= cdf[-1]
    u = rng.random(size)
    rank0 = np.searchsorted(cdf, u, side="left").astype(np.int64)
    np.minimum(rank0, N - 1, out=rank0)
    if mapping == "identity":
        return rank0
    if mapping == "scattered":
        a = _scatter_multiplier(N)
        return (rank0 * a) % N
    raise ValueError(f"unknown mapping {mapping!r}")


def make_cores(rng: np.random.Generator, spec: TableSpec) -> List[np.ndarray]:
    cores = []
    for k in range(spec.K):
        shape = (spec.r[k], spec.n[k], spec.d[k], spec.r[k + 1])
        if spec.core_dist == "uniform":
            g = rng.uniform(-spec.core_scale, spec.core_scale, size=shape)
        elif spec.core_dist == "normal":
            g = rng.normal(0.0, spec.core_scale, size=shape)
        else:
            raise ValueError(spec.core_dist)
        cores.append(np.ascontiguousarray(g.astype(np.float32)))
    return cores


def near_equal_factors3(N: int) -> Tuple[int, int, int]:
    """n = smallest integer with n**3 >= N; (ceil(N / n**2), n, n)."""
    n = max(1, int(round(N ** (1.0 / 3.0))))
    while n ** 3 < N:
        n += 1
    while n > 1 and (n - 1) ** 3 >= N:
        n -= 1
    n1 = -(-N // (n * n))
    return (n1, n, n)


def _assemble(name, tables, B, pooling, seed0, mapping, with_grad, meta=None, batch_seed0=None) -> Workload:
    """pooling: int (fixed) or (lo, hi) inclusive uniform per (table, bag); a list gives one of these per table.
    batch_seed0: draw the batch (bag lengths, indices, grad_out) from another stream while the cores stay
    those of seed0 (used for the per-rank batches of a multi-GPU run)."""
    T = len(tables)

    def one_table(t):
        # every table has its own generator, so the result does not depend on thread scheduling
        spec = tables[t]
        rng = np.random.default_rng(seed0 + t)
        tc = make_cores(rng, spec)
        if batch_seed0 is not None:
            rng = np.random.default_rng(batch_seed0 + t)
        pool_t = pooling[t] if isinstance(pooling, list) else pooling
        if isinstance(pool_t, tuple):
            lens = rng.integers(pool_t[0], pool_t[1] + 1, size=B, dtype=np.int64)
        else:
            lens = np.full(B, int(pool_t), dtype=np.int64)
        return tc, lens, zipf_rows(rng, spec.N, spec.alpha, int(lens.sum()), mapping)

    if T > 1 and sum(s.N for s in tables) > 1_000_000:
        with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
            parts = list(ex.map(one_table, range(T)))
    else:
        parts = [one_table(t) for t in range(T)]
    cores = [p[0] for p in parts]
    len_parts = [p[1] for p in parts]
    idx_parts = [p[2] for p in parts]
    lens = np.concatenate(len_parts)
    offsets = np.zeros(T * B + 1, dtype=np.int64)
    np.cumsum(lens, out=offsets[1:])
    indices = np.concatenate(idx_parts).astype(np.int64) if idx_parts else np.zeros(0, np.int64)
    grad = None
    if with_grad:
        rng = np.random.default_rng((seed0 if batch_seed0 is None else batch_seed0) + 999)
        D = tables[0].D
        grad = rng.standard_normal(size=(B, T * D)).astype(np.float32)
    return Workload(name=name, tables=tables, B=B, indices=indices, offsets=offsets, cores=cores,
                    grad_out=grad, mapping=mapping, meta=meta or {})


def _cfg3_tables(rng: np.random.Generator, T: int, n_cap: Optional[int] = None) -> List[TableSpec]:
    tables = []
    for _ in range(T):
        N = int(round(10.0 ** rng.uniform(4.0, math.log10(4e7))))
        if n_cap is not None:
            N = max(2, N % (n_cap ** 3 - 1) + 1)
        n = near_equal_factors3(N)
        r1 = int(rng.choice([16, 32]))
        r2 = int(rng.choice([16, 32]))
        alpha = float(rng.uniform(0.8, 1.2))
        tables.append(TableSpec(N=N, n=n, d=(4, 4, 4), r=(1, r1, r2, 1), alpha=alpha,
                                core_dist="normal", core_scale=0.05))
    return tables


def make(config: int, *, tiny: bool = False, mapping: str = "identity", seed: Optional[int] = None,
         batch: Optional[int] = None, num_tables: Optional[int] = None, batch_seed: Optional[int] = None) -> Workload:
    """Build one of the five benchmark configurations (1..5).

    tiny=True keeps the structure (K, dim factors, skew, pooling law) but shrinks row factors to <= 6
    and the batch to <= 16 so that a dense materialisation of the table is affordable.
    `batch` / `num_tables` override B / T (used for reduced-size parity cases and bounded CPU timing).
    `batch_seed` draws another batch (bag lengths, indices, grad_out) for the same tables and cores.
    """
    seed0 = (BASE_SEED if seed is None else seed) + 1000 * config
    bs0 = None if batch_seed is None else batch_seed + 1000 * config
    if config == 1:
        n = (5, 6, 4) if tiny else (100, 100, 100)
        N = int(np.prod(n)) - (3 if tiny else 0)
        spec = TableSpec(N=N, n=n, d=(4, 4, 4), r=(1, 8, 8, 1), alpha=1.05, core_dist="uniform", core_scale=0.1)
        B = batch or (16 if tiny else 1024)
        return _assemble("cfg1" + ("-tiny" if tiny else ""), [spec], B, 1, seed0, mapping, False, batch_seed0=bs0)
    if config == 2:
        n = (4, 5, 6) if tiny else (200, 250, 200)
        N = int(np.prod(n))
        r = (1, 5, 3, 1) if tiny else (1, 32, 32, 1)
        spec = TableSpec(N=N, n=n, d=(4, 8, 4), r=r, alpha=1.1, core_dist="normal", core_scale=0.05)
        B = batch or (12 if tiny else 32768)
        return _assemble("cfg2" + ("-tiny" if tiny else ""), [spec], B, 20, seed0, mapping, False, batch_seed0=bs0)
    if config in (3, 5):
        # tables are drawn from the config-3 stream for both 3 and 5 so that 5 trains on 3's tables
        seed3 = (BASE_SEED if seed is None else seed) + 1000 * 3
        T = num_tables or (4 if tiny else 60)
        trng = np.random.default_rng(seed3 + 500)
        tables = _cfg3_tables(trng, T, n_cap=5 if tiny else None)
        if tiny:
            tables = [TableSpec(N=s.N, n=s.n, d=s.d, r=(1, 3 + (i % 2), 2 + (i % 3), 1), alpha=s.alpha,
                                core_dist=s.core_dist, core_scale=s.core_scale) for i, s in enumerate(tables)]
        B = batch or (16 if tiny else 32768)
        pooling = (1, 9) if tiny else (1, 100)
        return _assemble(f"cfg{config}" + ("-tiny" if tiny else ""), tables, B, pooling, seed3, mapping,
                         with_grad=(config == 5), batch_seed0=None if batch_seed is None else batch_seed + 3000)
    if config == 4:
        n = (3, 4, 3, 4) if tiny else (64, 64, 64, 64)
        N = int(np.prod(n))
        r = (1, 3, 4, 2, 1) if tiny else (1, 64, 64, 64, 1)
        spec = TableSpec(N=N, n=n, d=(2, 4, 4, 4), r=r, alpha=1.2, core_dist="normal", core_scale=0.02)
        B = batch or (16 if tiny else 65536)
        return _assemble("cfg4" + ("-tiny" if tiny else ""), [spec], B, 8, seed0, mapping, False, batch_seed0=bs0)
    raise ValueError("config must be 1..5")


def custom(tables: Sequence[TableSpec], B: int, pooling, *, seed: int = 1234, mapping: str = "identity",
           with_grad: bool = False, name: str = "custom") -> Workload:
    """Arbitrary shapes for unit tests (pooling: int or (lo, hi); lo may be 0 to get empty bags)."""
    return _assemble(name, list(tables), B, pooling, seed, mapping, with_grad)


SWEEP_DIM_FACTORS = {16: (2, 2, 4), 32: (2, 4, 4), 64: (4, 4, 4), 128: (4, 8, 4)}


def sweep_point(D: int, rank: int, batch: int, *, num_tables: int = 8, with_grad: bool = False,
                mapping: str = "identity", seed: Optional[int] = None) -> Workload:
    """One point of the embedding-dimension / TT-rank / batch-size sweep (3 cores).

    Tables: the first `num_tables` row counts and Zipf exponents of the config-3 stream (row counts
    log-uniform in [1e4, 4e7], three near-equal row factors), every table with dim factors
    SWEEP_DIM_FACTORS[D] and ranks (1, rank, rank, 1); cores N(0, 0.05); pooling factor uniform in
    [1, 100] per (table, bag).  The same tables serve every (D, rank, batch), so points differ only in
    the swept quantity.
    """
    if D not in SWEEP_DIM_FACTORS:
        raise ValueError(f"D must be one of {sorted(SWEEP_DIM_FACTORS)}")
    seed3 = (BASE_SEED if seed is None else seed) + 1000 * 3
    base = _cfg3_tables(np.random.default_rng(seed3 + 500), num_tables)
    tables = [TableSpec(N=s.N, n=s.n, d=SWEEP_DIM_FACTORS[D], r=(1, rank, rank, 1), alpha=s.alpha,
                        core_dist="normal", core_scale=0.05) for s in base]
    return _assemble(f"sweep-D{D}-r{rank}-B{batch}", tables, batch, (1, 100), seed3 + 7 * D + rank, mapping,
                     with_grad=with_grad)


def generic_point(batch: int = 32768, *, num_tables: int = 8, with_grad: bool = True, mapping: str = "identity",
                  seed: Optional[int] = None) -> Workload:
    """A shape that none of the register-tiled kernel variants covers: dim factors (3, 3, 5) (D = 45, not a multiple
    of four) and ranks (1, 6, 4, 1), on the first `num_tables` row counts and Zipf exponents of the config-3 stream,
    pooling factor uniform in [1, 100].  It exercises the any-shape path end to end (scalar pooling and dE included)."""
    seed3 = (BASE_SEED if seed is None else seed) + 1000 * 3
    base = _cfg3_tables(np.random.default_rng(seed3 + 500), num_tables)
    tables = [TableSpec(N=s.N, n=s.n, d=(3, 3, 5), r=(1, 6, 4, 1), alpha=s.alpha, core_dist="normal", core_scale=0.05)
              for s in base]
    return _assemble(f"generic-d3x3x5-r6x4-B{batch}", tables, batch, (1, 100), seed3 + 4500, mapping, with_grad=with_grad)


def many_tables_point(batch: int = 32768, *, num_tables: int = 240, with_grad: bool = True, mapping: str = "identity",
                      seed: Optional[int] = None) -> Workload:
    """The operating point of the paper's evaluation (Sec. 4.1): hundreds of tables, three cores, D = 32 (dim factors
    2 x 4 x 4), ranks (1, 32, 32, 1), batch 32768.  The paper's tables and index streams are a public benchmark that
    is not available here and whose pooling factors the paper does not state, so this is a stand-in: row counts and
    Zipf exponents from the config-3 recipe (log-uniform in [1e4, 4e7], exponent uniform in [0.8, 1.2]); every table
    has its own largest bag length P_t, log-uniform in [1, 64] (a quarter of the tables come out with at most three
    lookups per bag, a fifth with up to 32 or more), bag lengths uniform in [1, P_t]."""
    seed6 = (BASE_SEED if seed is None else seed) + 1000 * 6
    trng = np.random.default_rng(seed6 + 500)
    base = _cfg3_tables(trng, num_tables)
    tables = [TableSpec(N=s.N, n=s.n, d=(2, 4, 4), r=(1, 32, 32, 1), alpha=s.alpha, core_dist="normal", core_scale=0.05)
              for s in base]
    pooling = [(1, int(round(64.0 ** trng.uniform(0.0, 1.0)))) for _ in range(num_tables)]
    return _assemble(f"many-tables-T{num_tables}-D32-r32-B{batch}", tables, batch, pooling, seed6, mapping,
                     with_grad=with_grad, meta={"max_bag": [p[1] for p in pooling]})
