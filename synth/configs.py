"""Seeded synthetic stand-ins for the paper's workloads (SuiteSparse matrices, FROSTT / BIGtensor
3-order tensors), in the five shapes the benchmark configuration names.

Each generator returns a `Case`: COO coordinates (one int32 tensor per mode, arbitrary order, all
cells distinct), fp64 values U(-1,1), the dense operands, and the realised statistics. Nothing here
computes a contraction or a packed format: this module only makes inputs, for the CPU oracle and for
the CUDA library alike.

Discrete laws are sampled by inverse CDF: the cumulative table is built once on the host in fp64,
then binary-searched with uniforms from the counter-based generator (`synth.rng`), so a case is a
pure function of (config, scale, seed) on any device.

`scale` s multiplies nnz by s and every extent by s**(1/order), which keeps density and mean segment
lengths roughly constant; s = 1 is the only scale that is reported.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

from . import rng

BASE_SEED = 20210205


@dataclass
class Case:
    name: str
    op: str                      # "spmv" | "spmm" | "ttv" | "ttm" | "mttkrp"
    dims: tuple
    coords: list                 # order x int32[nnz], COO, shuffled
    val: torch.Tensor            # float64[nnz]
    dense: dict                  # operand name -> float64 tensor
    R: int = 1
    mode: int = 0                # contracted (ttv/ttm) or output (mttkrp) tensor mode, 0-based
    seed: int = 0
    stats: dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.val.numel())

    @property
    def order(self) -> int:
        return len(self.dims)

    def to(self, device) -> "Case":
        return Case(self.name, self.op, self.dims, [c.to(device) for c in self.coords],
                    self.val.to(device), {k: v.to(device) for k, v in self.dense.items()},
                    self.R, self.mode, self.seed, dict(self.stats))


# ----------------------------------------------------------------------------- helpers

def _scaled(extent: int, scale: float, order: int, floor: int = 4) -> int:
    return max(floor, int(round(extent * scale ** (1.0 / order))))


def _inverse_cdf(cdf: np.ndarray, u: torch.Tensor) -> torch.Tensor:
    """Smallest k with cdf[k] > u (0-based), clamped to the table."""
    t = torch.from_numpy(cdf).to(u.device)
    k = torch.searchsorted(t, u, right=True)
    return torch.clamp(k, max=len(cdf) - 1)


def _redraw_duplicates(keys_of, draw, n: int, max_rounds: int = 64):
    """Make n draws whose keys are pairwise distinct.

    `draw(idx, round)` returns fresh raw draws for positions idx; `keys_of(idx, raw)` maps them to
    int64 keys. A position whose key equals that of an earlier position (in sorted order) is redrawn
    with the next round's counters until no duplicate is left.
    """
    device = draw.device
    idx = torch.arange(n, dtype=torch.int64, device=device)
    raw = draw(idx, 0)
    key = keys_of(idx, raw)
    for rnd in range(1, max_rounds + 1):
        order = torch.sort(key, stable=True).indices
        sk = key[order]
        dup = torch.zeros(n, dtype=torch.bool, device=device)
        dup[1:] = sk[1:] == sk[:-1]
        bad = order[dup]
        if bad.numel() == 0:
            return raw
        new = draw(bad, rnd)
        raw[bad] = new
        key[bad] = keys_of(bad, new)
    raise RuntimeError("could not make the draws distinct")


class _Draw:
    """Uniform integer draws in [0, bound) addressed by (position, round)."""

    def __init__(self, seed, stream, bound, n, device):
        self.seed, self.stream, self.bound, self.n, self.device = seed, stream, bound, n, device

    def __call__(self, idx, rnd):
        return rng.below_at(self.seed, self.stream, idx + rnd * self.n, self.bound)


def _distinct_subset(keys: torch.Tensor, n: int, seed: int, stream: int) -> torch.Tensor:
    """n distinct keys chosen uniformly among the distinct values of `keys` (returned unordered)."""
    uniq = torch.unique(keys)
    if uniq.numel() < n:
        raise RuntimeError(f"only {uniq.numel()} distinct keys for {n} wanted")
    rank = rng.bits64(seed, stream, uniq)
    keep = torch.sort(rank, stable=True).indices[:n]
    return uniq[keep]


def _shuffle(seed, stream, tensors):
    p = rng.permutation(seed, stream, tensors[0].numel(), tensors[0].device)
    return [t[p] for t in tensors]


def _i32(t):
    return t.to(torch.int32).contiguous()


# ----------------------------------------------------------------------------- config 1: SpMV

def spmv_uniform(scale: float = 1.0, seed: int | None = None, device="cpu") -> Case:
    """4096 x 4096 fp64 matrix, 65,536 nnz at uniform-random distinct cells; dense x of length 4096."""
    seed = BASE_SEED + 1 if seed is None else seed
    I = J = _scaled(4096, scale, 2)
    n = min(max(1, int(round(65536 * scale))), I * J)
    cells = rng.below(seed, 1, int(n * 1.05) + 1024, I * J, device)
    while torch.unique(cells).numel() < n:
        cells = torch.cat([cells, rng.below(seed, 1, n, I * J, device, offset=cells.numel())])
    cells = _distinct_subset(cells, n, seed, 2)
    i, j = cells // J, cells % J
    val = rng.symmetric(seed, 3, n, device)
    i, j, val = _shuffle(seed, 4, [i, j, val])
    x = rng.symmetric(seed, 5, J, device)
    return Case("C1-spmv-uniform", "spmv", (I, J), [_i32(i), _i32(j)], val, {"x": x}, seed=seed,
                stats={"nnz": n, "mean_row": n / I})


# ----------------------------------------------------------------------------- config 2: SpMM

def zipf_clipped_cdf(s: float, cap: int) -> np.ndarray:
    """CDF over k = 1..cap of P(k) = k^-s / zeta(s), with the whole tail mass k >= cap lumped on cap."""
    k = np.arange(1, cap, dtype=np.float64)
    zeta = float(np.sum(np.arange(1, 2_000_000, dtype=np.float64) ** -s)) + \
        (2_000_000.0 ** (1.0 - s)) / (s - 1.0)          # Euler-Maclaurin tail
    cdf = np.cumsum(k ** -s) / zeta
    return np.concatenate([cdf, [1.0]])


def spmm_zipf(scale: float = 1.0, seed: int | None = None, device="cpu", R: int = 64) -> Case:
    """1,048,576^2 fp64 matrix, row lengths min(Zipf(1.8), 10,000), uniform distinct columns per row;
    dense B of 1,048,576 x 64."""
    seed = BASE_SEED + 2 if seed is None else seed
    I = J = max(4, int(round((1 << 20) * scale)))      # nnz follows the row count, so rows scale by s
    cap = max(1, min(10_000, J // 4))
    cdf = zipf_clipped_cdf(1.8, cap)
    length = _inverse_cdf(cdf, rng.uniform(seed, 1, I, device)) + 1            # 1..cap
    n = int(length.sum().item())
    row = torch.repeat_interleave(torch.arange(I, dtype=torch.int64, device=device), length)
    draw = _Draw(seed, 2, J, n, device)
    col = _redraw_duplicates(lambda idx, raw: row[idx] * J + raw, draw, n)
    val = rng.symmetric(seed, 3, n, device)
    row, col, val = _shuffle(seed, 4, [row, col, val])
    B = rng.symmetric(seed, 5, J * R, device).reshape(J, R)
    return Case("C2-spmm-zipf", "spmm", (I, J), [_i32(row), _i32(col)], val, {"B": B}, R=R, seed=seed,
                stats={"nnz": n, "mean_row": n / I, "max_row": int(length.max().item()),
                       "rows_len1": int((length == 1).sum().item())})


# ----------------------------------------------------------------------------- config 3: TTV

def _largest_remainder(weights: np.ndarray, total: int) -> np.ndarray:
    w = weights / weights.sum() * total
    base = np.floor(w).astype(np.int64)
    rest = int(total - base.sum())
    if rest > 0:
        frac = w - base
        top = np.argsort(-frac, kind="stable")[:rest]
        base[top] += 1
    return base


def ttv_powerlaw_slices(scale: float = 1.0, seed: int | None = None, device="cpu") -> Case:
    """20,000^3 tensor, 50M nnz, mode-1 slice sizes ~ rank^-2, uniform distinct (j,k) inside a slice;
    dense vector over mode 3."""
    seed = BASE_SEED + 3 if seed is None else seed
    I = _scaled(20_000, scale, 3)
    J = _scaled(20_000, scale, 3)
    K = _scaled(20_000, scale, 3)
    n = max(1, int(round(50_000_000 * scale)))
    sizes = _largest_remainder(np.arange(1, I + 1, dtype=np.float64) ** -2.0, n)
    sizes = np.minimum(sizes, (J * K) // 2)          # never ask a slice for more cells than it can hold
    n = int(sizes.sum())
    size_t = torch.from_numpy(sizes).to(device)
    relabel = rng.permutation(seed, 6, I, device)
    rank = torch.repeat_interleave(torch.arange(I, dtype=torch.int64, device=device), size_t)
    draw = _Draw(seed, 2, J * K, n, device)
    cell = _redraw_duplicates(lambda idx, raw: rank[idx] * (J * K) + raw, draw, n)
    i = relabel[rank]
    j, k = cell // K, cell % K
    val = rng.symmetric(seed, 3, n, device)
    i, j, k, val = _shuffle(seed, 4, [i, j, k, val])
    v = rng.symmetric(seed, 5, K, device)
    return Case("C3-ttv-powerlaw", "ttv", (I, J, K), [_i32(i), _i32(j), _i32(k)], val, {"v": v}, mode=2,
                seed=seed, stats={"nnz": n, "slices": int((sizes > 0).sum()), "top_slice": int(sizes.max())})


# ----------------------------------------------------------------------------- config 4: TTM

def ttm_geometric_fibers(scale: float = 1.0, seed: int | None = None, device="cpu", R: int = 16) -> Case:
    """100,000 x 50,000 x 20,000 tensor, 30M nnz, fiber lengths geometric (mean 8) on {1,2,...},
    fibers at uniform distinct (i,j), uniform distinct k inside a fiber; dense U of 20,000 x 16."""
    seed = BASE_SEED + 4 if seed is None else seed
    I = _scaled(100_000, scale, 3)
    J = _scaled(50_000, scale, 3)
    K = _scaled(20_000, scale, 3)
    n = max(1, int(round(30_000_000 * scale)))
    p = 1.0 / 8.0
    nf = int(n / 8 * 1.05) + 64
    nf = min(nf, (I * J) // 2)
    while True:
        u = rng.uniform(seed, 1, nf, device)
        length = torch.floor(torch.log1p(-u) / math.log1p(-p)).to(torch.int64) + 1
        length = torch.clamp(length, max=max(1, K // 2))
        csum = torch.cumsum(length, 0)
        if int(csum[-1].item()) >= n or nf >= (I * J) // 2:
            break
        nf = min(nf * 2, (I * J) // 2)
    n = min(n, int(csum[-1].item()))
    f_last = int(torch.searchsorted(csum, torch.tensor([n], device=device)).item())
    length = length[: f_last + 1].clone()
    length[f_last] -= int(csum[f_last].item()) - n
    F = f_last + 1
    cells = rng.below(seed, 7, int(F * 1.02) + 1024, I * J, device)
    while torch.unique(cells).numel() < F:
        cells = torch.cat([cells, rng.below(seed, 7, F, I * J, device, offset=cells.numel())])
    cells = _distinct_subset(cells, F, seed, 8)
    cells = cells[rng.permutation(seed, 9, F, device)]       # fiber lengths independent of position
    fib = torch.repeat_interleave(torch.arange(F, dtype=torch.int64, device=device), length)
    draw = _Draw(seed, 2, K, n, device)
    k = _redraw_duplicates(lambda idx, raw: fib[idx] * K + raw, draw, n)
    cell = cells[fib]
    i, j = cell // J, cell % J
    val = rng.symmetric(seed, 3, n, device)
    i, j, k, val = _shuffle(seed, 4, [i, j, k, val])
    U = rng.symmetric(seed, 5, K * R, device).reshape(K, R)
    return Case("C4-ttm-geometric", "ttm", (I, J, K), [_i32(i), _i32(j), _i32(k)], val, {"U": U}, R=R, mode=2,
                seed=seed, stats={"nnz": n, "fibers": F, "max_fiber": int(length.max().item())})


# ----------------------------------------------------------------------------- config 5: MTTKRP

def zipf_mandelbrot_cdf(dim: int, alpha: float, q: float) -> np.ndarray:
    k = np.arange(1, dim + 1, dtype=np.float64)
    w = (k + q) ** -alpha
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    cdf[-1] = 1.0
    return cdf


def mttkrp_powerlaw(scale: float = 1.0, seed: int | None = None, device="cpu", R: int = 32,
                    q: float = 100.0) -> Case:
    """1,000,000 x 500,000 x 200,000 tensor, 100M nnz, independent per-mode power-law index frequencies
    p(k) ~ (k+q)^-1.5 (q = 100 so that the draws are mostly distinct cells), ids relabelled by a seeded
    permutation; dense factors B (500,000 x 32) and C (200,000 x 32)."""
    seed = BASE_SEED + 5 if seed is None else seed
    dims = (_scaled(1_000_000, scale, 3), _scaled(500_000, scale, 3), _scaled(200_000, scale, 3))
    n = max(1, int(round(100_000_000 * scale)))
    tables = [zipf_mandelbrot_cdf(d, 1.5, q) for d in dims]
    draws = int(n * 1.08) + 4096
    key = None
    for attempt in range(8):
        key = torch.zeros(draws, dtype=torch.int64, device=device)
        for m, d in enumerate(dims):
            idx = _inverse_cdf(tables[m], rng.uniform(seed, 10 + m, draws, device))
            key = key * d + idx
            del idx
        if torch.unique(key).numel() >= n:
            break
        draws = int(draws * 1.3)
    key = _distinct_subset(key, n, seed, 2)
    coords = []
    for m in (2, 1, 0):
        coords.append(key % dims[m])
        key = key // dims[m]
    k, j, i = coords
    i = rng.permutation(seed, 20, dims[0], device)[i]
    j = rng.permutation(seed, 21, dims[1], device)[j]
    k = rng.permutation(seed, 22, dims[2], device)[k]
    val = rng.symmetric(seed, 3, n, device)
    i, j, k, val = _shuffle(seed, 4, [i, j, k, val])
    B = rng.symmetric(seed, 5, dims[1] * R, device).reshape(dims[1], R)
    C = rng.symmetric(seed, 6, dims[2] * R, device).reshape(dims[2], R)
    return Case("C5-mttkrp-powerlaw", "mttkrp", dims, [_i32(i), _i32(j), _i32(k)], val, {"B": B, "C": C},
                R=R, mode=0, seed=seed, stats={"nnz": n, "q": q})


CONFIGS = {
    1: spmv_uniform,
    2: spmm_zipf,
    3: ttv_powerlaw_slices,
    4: ttm_geometric_fibers,
    5: mttkrp_powerlaw,
}


def make(config: int, scale: float = 1.0, seed: int | None = None, device="cpu", **kw) -> Case:
    return CONFIGS[config](scale=scale, seed=seed, device=device, **kw)


# ----------------------------------------------------------------------------- small random cases for tests

def random_coo(dims, nnz: int, seed: int, device="cpu", integer_values: bool = False):
    """nnz distinct uniform cells of a tensor with the given extents, shuffled; values U(-1,1) or small
    integers in {-3..3} (zero excluded) when `integer_values` (then every partial sum is exact)."""
    total = 1
    for d in dims:
        total *= d
    nnz = min(nnz, total)
    if nnz == 0:
        return [torch.zeros(0, dtype=torch.int32, device=device) for _ in dims], \
            torch.zeros(0, dtype=torch.float64, device=device)
    if total <= 4 * nnz + 64:
        cells = rng.permutation(seed, 1, total, device)[:nnz]
    else:
        cells = rng.below(seed, 1, 2 * nnz + 64, total, device)
        while torch.unique(cells).numel() < nnz:
            cells = torch.cat([cells, rng.below(seed, 1, nnz, total, device, offset=cells.numel())])
        cells = _distinct_subset(cells, nnz, seed, 2)
        cells = cells[rng.permutation(seed, 4, nnz, device)]
    coords = []
    for d in reversed(dims):
        coords.append(_i32(cells % d))
        cells = cells // d
    coords.reverse()
    if integer_values:
        v = rng.below(seed, 3, nnz, 6, device) - 3
        v = torch.where(v >= 0, v + 1, v).to(torch.float64)
    else:
        v = rng.symmetric(seed, 3, nnz, device)
    return coords, v


def random_dense(shape, seed: int, stream: int = 50, device="cpu", integer_values: bool = False):
    n = 1
    for d in shape:
        n *= d
    if integer_values:
        t = (rng.below(seed, stream, n, 7, device) - 3).to(torch.float64)
    else:
        t = rng.symmetric(seed, stream, n, device)
    return t.reshape(shape)
