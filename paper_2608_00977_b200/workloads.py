"""Seeded synthetic templates (inputs only: no residual, gradient or update arithmetic).

The same arrays are handed to the CPU oracle and to the CUDA library, so this
module is imported by tests and by the bench, never by either implementation.

Recipes (stand-ins for the paper's recommender and synthetic matrices, Sec. 6.1):
  * positions: uniform without replacement, an independent Bernoulli mask, or a
    "Zipf product law" (row and column popularity ranks drawn independently from a
    bounded power law, scattered over the ids by a fixed affine bijection,
    de-duplicated, trimmed to exactly nnz by a keyed hash);
  * values: low-rank signal p*_i . q*_j from random factors plus Gaussian noise,
    optionally mapped to integer 1..5 ratings: clamp(round(3 + signal + noise), 1, 5);
  * initial factors: a different draw from the data-generating factors.
`N(0, v)` is read as mean 0, VARIANCE v everywhere (so N(0, 1/sqrt(k)) has standard
deviation k**-0.25 and p.q has unit variance).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

CLIP_NONE, CLIP_ASYM_STEP, CLIP_ASYM_GRAD, CLIP_ASYM_ENTRY = 0, 1, 2, 3
NORM_NONE, NORM_COUNT = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    m: int
    n: int
    k: int
    nnz: int                 # target |Omega| (bernoulli: expected value, actual count differs)
    positions: str           # "uniform" | "zipf" | "bernoulli"
    zipf_s: float = 0.0
    density: float = 0.0     # bernoulli only
    values: str = "lowrank"  # "lowrank" (signal + noise) | "ratings" (1..5 integers)
    noise_var: float = 1e-4
    signal_rank: int = 0     # 0 -> k
    precision: str = "f32"   # "f32" | "bf16"
    eta: float = 0.01
    lam: float = 0.0
    xi: float = 0.1
    clip: int = CLIP_NONE
    norm_p: int = NORM_NONE
    norm_q: int = NORM_NONE
    epochs: int = 20
    seed: int = 20260800


# The five benchmark configurations (C1..C5) and their step parameters.
C1 = Workload("C1-tiny-2000x1500-k16", 2000, 1500, 16, 150_000, "uniform",
              values="lowrank", noise_var=1e-4, precision="f32", eta=0.01, lam=0.0,
              clip=CLIP_NONE, norm_p=NORM_NONE, norm_q=NORM_NONE, epochs=20, seed=20260801)
C2 = Workload("C2-50000x20000-k32-zipf1.1", 50_000, 20_000, 32, 10_000_000, "zipf", zipf_s=1.1,
              values="ratings", noise_var=0.25, precision="f32", eta=0.05, lam=0.03, xi=0.1,
              clip=CLIP_ASYM_STEP, norm_p=NORM_COUNT, norm_q=NORM_COUNT, epochs=50, seed=20260802)
C3 = Workload("C3-200000x100000-k64-zipf1.1-bf16", 200_000, 100_000, 64, 100_000_000, "zipf",
              zipf_s=1.1, values="ratings", noise_var=0.25, precision="bf16", eta=0.05, lam=0.03,
              xi=0.1, clip=CLIP_ASYM_STEP, norm_p=NORM_COUNT, norm_q=NORM_COUNT, epochs=10,
              seed=20260803)
C4 = Workload("C4-16384x16384-k128-bernoulli0.30", 16_384, 16_384, 128, int(0.30 * 16_384 * 16_384),
              "bernoulli", density=0.30, values="lowrank", noise_var=1e-4, precision="bf16",
              eta=0.2, lam=0.0, clip=CLIP_NONE, norm_p=NORM_COUNT, norm_q=NORM_COUNT, epochs=10,
              seed=20260804)
C5 = Workload("C5-2000000x1000000-k128-zipf1.05-bf16", 2_000_000, 1_000_000, 128, 1_000_000_000,
              "zipf", zipf_s=1.05, values="ratings", noise_var=0.25, signal_rank=16,
              precision="bf16", eta=0.05, lam=0.03, xi=0.1, clip=CLIP_ASYM_STEP,
              norm_p=NORM_COUNT, norm_q=NORM_COUNT, epochs=3, seed=20260805)

CONFIGS = {"C1": C1, "C2": C2, "C3": C3, "C4": C4, "C5": C5}


def scaled(w: Workload, name: str, m: int, n: int, nnz: int, **kw) -> Workload:
    """A smaller template with the same recipe and step parameters (parity-test sizes)."""
    return replace(w, name=name, m=m, n=n, nnz=nnz, **kw)


# C5 at 1/16 of its entries (same recipe, k and skew; both bf16 shadows still exceed L2): the case
# small enough for multi-pass profiler captures
CONFIGS["C5S"] = scaled(C5, "C5S-500000x250000-k128-zipf1.05-bf16", 500_000, 250_000, 62_500_000)


@dataclass
class Template:
    w: Workload
    rows: torch.Tensor   # int32 (nnz)
    cols: torch.Tensor   # int32 (nnz)
    vals: torch.Tensor   # float32 (nnz)
    P0: torch.Tensor     # float32 (m, k) initial factors
    Q0: torch.Tensor     # float32 (n, k)

    @property
    def nnz(self) -> int:
        return int(self.rows.numel())


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _coprime_near(x: int, N: int) -> int:
    x = max(1, x % N) if N > 1 else 1
    while math.gcd(x, N) != 1:
        x += 1
    return x


def _mix64(x: torch.Tensor, seed: int) -> torch.Tensor:
    """Keyed 63-bit hash of int64 keys (wrapping int64 arithmetic; logical shifts by masking)."""
    def lsr(v, s):
        return (v >> s) & ((1 << (64 - s)) - 1)
    c1 = 0xBF58476D1CE4E5B9 - (1 << 64)
    c2 = 0x94D049BB133111EB - (1 << 64)
    x = x + ((seed * 0x9E3779B97F4A7C15) & ((1 << 63) - 1))
    x = (x ^ lsr(x, 30)) * c1
    x = (x ^ lsr(x, 27)) * c2
    x = x ^ lsr(x, 31)
    return x & ((1 << 63) - 1)


def zipf_ranks(N: int, s: float, count: int, g: torch.Generator, device) -> torch.Tensor:
    """0-based popularity ranks from the bounded power law with exponent s (inverse CDF)."""
    u = torch.rand(count, generator=g, device=device, dtype=torch.float64)
    a = 1.0 - s
    base = 1.0 + u * ((N + 1.0) ** a - 1.0)
    r = torch.floor(base ** (1.0 / a)).to(torch.int64)
    return torch.clamp(r, 1, N) - 1


def positions_zipf(m, n, nnz, s, seed, device) -> torch.Tensor:
    """Sorted unique int64 keys row*n+col, exactly nnz of them."""
    if nnz > m * n:
        raise ValueError("nnz exceeds the number of cells")
    g = _gen(seed, device)
    Ar, Br = _coprime_near(int(0.6180339887 * m), m), (seed * 7919) % m
    Ac, Bc = _coprime_near(int(0.7548776662 * n), n), (seed * 104729) % n
    uniq = torch.empty(0, dtype=torch.int64, device=device)
    draws = 0
    while uniq.numel() < nnz:
        deficit = nnz - uniq.numel()
        batch = int(min(max(2 * deficit, 1 << 16), 1 << 30))
        rr = (zipf_ranks(m, s, batch, g, device) * Ar + Br) % m
        cc = (zipf_ranks(n, s, batch, g, device) * Ac + Bc) % n
        key = rr * n + cc
        del rr, cc
        uniq = torch.unique(torch.cat([uniq, key]))
        del key
        draws += batch
        if draws > 400 * nnz:
            raise RuntimeError("zipf generator cannot reach the requested nnz")
    if uniq.numel() > nnz:
        h = _mix64(uniq, seed)
        thr = torch.sort(h).values[nnz - 1]
        keep = h <= thr
        del h
        uniq = uniq[keep][:nnz]
    return uniq


def positions_uniform(m, n, nnz, seed, device) -> torch.Tensor:
    g = _gen(seed, device)
    cells = m * n
    if cells <= (1 << 27):
        ids = torch.randperm(cells, generator=g, device=device)[:nnz]
        return torch.sort(ids).values.to(torch.int64)
    uniq = torch.empty(0, dtype=torch.int64, device=device)
    while uniq.numel() < nnz:
        extra = torch.randint(0, cells, (int(1.2 * (nnz - uniq.numel())) + 1024,), generator=g,
                              device=device, dtype=torch.int64)
        uniq = torch.unique(torch.cat([uniq, extra]))
    if uniq.numel() > nnz:
        h = _mix64(uniq, seed)
        thr = torch.sort(h).values[nnz - 1]
        uniq = uniq[h <= thr][:nnz]
    return uniq


def positions_bernoulli(m, n, density, seed, device) -> torch.Tensor:
    g = _gen(seed, device)
    out = []
    rows_per = max(1, (1 << 26) // n)
    for r0 in range(0, m, rows_per):
        r1 = min(m, r0 + rows_per)
        mask = torch.rand((r1 - r0) * n, generator=g, device=device) < density
        out.append(torch.nonzero(mask).flatten() + r0 * n)
    return torch.cat(out) if out else torch.empty(0, dtype=torch.int64, device=device)


def _factors(nrow, k, var, g, device) -> torch.Tensor:
    return torch.randn(nrow, k, generator=g, device=device, dtype=torch.float32) * math.sqrt(var)


def make_template(w: Workload, device="cpu", order: str = "sorted") -> Template:
    """Builds the COO triples and the initial factors of workload `w` on `device`.

    order = "sorted": COO sorted by (row, col); "shuffled": a seeded random permutation.
    """
    device = torch.device(device)
    if w.positions == "uniform":
        keys = positions_uniform(w.m, w.n, w.nnz, w.seed, device)
    elif w.positions == "zipf":
        keys = positions_zipf(w.m, w.n, w.nnz, w.zipf_s, w.seed, device)
    elif w.positions == "bernoulli":
        keys = positions_bernoulli(w.m, w.n, w.density, w.seed, device)
    else:
        raise ValueError(w.positions)
    nnz = keys.numel()
    rows = (keys // w.n).to(torch.int32)
    cols = (keys % w.n).to(torch.int32)
    del keys

    g = _gen(w.seed + 1000003, device)
    r = w.signal_rank or w.k
    Ps = _factors(w.m, r, 1.0 / math.sqrt(r), g, device)
    Qs = _factors(w.n, r, 1.0 / math.sqrt(r), g, device)
    vals = torch.empty(nnz, dtype=torch.float32, device=device)
    chunk = max(1, (1 << 28) // max(r, 1))
    for a in range(0, nnz, chunk):
        b = min(nnz, a + chunk)
        sig = (Ps[rows[a:b].long()] * Qs[cols[a:b].long()]).sum(dim=1)
        noise = torch.randn(b - a, generator=g, device=device, dtype=torch.float32) * math.sqrt(w.noise_var)
        if w.values == "ratings":
            vals[a:b] = torch.clamp(torch.round(3.0 + sig + noise), 1.0, 5.0)
        else:
            vals[a:b] = sig + noise
    del Ps, Qs

    if order == "shuffled" and nnz > 0:
        gp = _gen(w.seed + 77, device)
        p = torch.randperm(nnz, generator=gp, device=device)
        rows, cols, vals = rows[p].contiguous(), cols[p].contiguous(), vals[p].contiguous()

    g0 = _gen(w.seed + 1, device)
    P0 = _factors(w.m, w.k, 1.0 / math.sqrt(w.k), g0, device)
    Q0 = _factors(w.n, w.k, 1.0 / math.sqrt(w.k), g0, device)
    return Template(w, rows, cols, vals, P0, Q0)
