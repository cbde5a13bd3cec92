"""Seeded synthetic workloads shaped like the paper's GLM experiments (Table 1 shapes; Sec. 5.1 set-up).

This module only draws inputs. It contains none of the training method's arithmetic and is the one module
that both the GPU library's callers and the CPU checker's callers may use, so that both sides see the
very same arrays. All draws come from a ``torch.Generator`` seeded by the caller, so a workload is a pure
function of (config, scale, seed) for a given torch build.

Five configurations (``scale`` divides the number of rows and columns, keeping the non-zeros per row):

1. ``hinge_dense``     n=10 000, d=100 dense N(0,1); noisy linear labels; lambda = 1/n; K=4.
2. ``hinge_csr``       n=1 000 000, d=100 000, Poisson(50) distinct Zipf(1.1) ids per row, unit-norm rows,
                       5 % label flips; lambda=1e-5; K=16.
3. ``logistic_dense``  n=11 000 000, d=28 standardised N(0,1) (the shape of Higgs); Bernoulli(sigmoid) labels;
                       lambda=1e-6; K=32.
4. ``hinge_hashed``    n=45 000 000, d=1 000 000, exactly 39 distinct Zipf(1.05) ids per row (the shape of
                       hashed Criteo), 25 % positives; lambda=1e-7; K=64 for 10 rounds, then K=16.
5. ``ridge_csc``       n=350 000, d=16 000 000, Poisson(3700) distinct uniform ids per row, U(0,1] values,
                       unit-norm rows, targets X w* + noise; lambda=1e-4; K=128 feature partitions; CSC.

No record of any real dataset is used or reproduced.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np
import torch


@dataclass
class Phase:
    """From round ``start`` on, use ``K`` partitions drawn with ``seed`` and the given sigma'."""
    start: int
    K: int
    seed: int
    sigma_prime: float


@dataclass
class Workload:
    name: str
    loss: str                 # "hinge" | "logistic" | "ridge"
    fmt: str                  # "dense" | "csr" | "csc"
    n_rows: int
    n_cols: int
    values: np.ndarray        # fp32: nnz, or n_rows*n_cols row-major for dense
    labels: np.ndarray        # fp32, one per row (example)
    lam: float
    rounds: int
    phases: List[Phase]
    indptr: Optional[np.ndarray] = None    # int64
    indices: Optional[np.ndarray] = None   # int32, sorted and unique inside a row / column
    H: int = 0                # 0 = one local epoch per round
    meta: dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.values.size)

    @property
    def n_coord(self) -> int:
        return self.n_cols if self.loss == "ridge" else self.n_rows

    def phase_at(self, rnd: int) -> Phase:
        cur = self.phases[0]
        for p in self.phases:
            if rnd >= p.start:
                cur = p
        return cur


_DEVICE = "cpu"   # where make() draws; "cuda" makes the two largest configurations practical (other random stream)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device=_DEVICE)
    g.manual_seed(int(seed))
    return g


def _sign_pm1(t: torch.Tensor) -> torch.Tensor:
    return torch.where(t >= 0, torch.ones_like(t), -torch.ones_like(t))


def _zipf_cdf(d: int, s: float) -> torch.Tensor:
    w = torch.arange(1, d + 1, dtype=torch.float64).pow(-s)
    c = torch.cumsum(w, 0)
    return c / c[-1]


def _distinct_ids(counts: torch.Tensor, d: int, g: torch.Generator, cdf: Optional[torch.Tensor],
                  rank_to_id: Optional[torch.Tensor], chunk_elems: int = 1 << 24) -> Tuple[torch.Tensor, torch.Tensor]:
    """For every row r draws ids with replacement from the given distribution over [0, d) (inverse CDF of
    ``cdf``, or uniform when ``cdf`` is None) and keeps the first ``counts[r]`` distinct ones in draw order
    (i.e. duplicates are redrawn). Ranks are mapped through ``rank_to_id`` when given. Returns
    (indptr int64, ids int32 sorted inside each row)."""
    n = counts.numel()
    counts = counts.to(torch.int64)
    indptr = torch.zeros(n + 1, dtype=torch.int64)
    indptr[1:] = torch.cumsum(counts, 0)
    out = torch.empty(int(indptr[-1]), dtype=torch.int32)
    cmax = int(counts.max())
    base_m = cmax + 16 if cdf is None else int(cmax * 2.0) + 32
    rows_per_chunk = max(1, chunk_elems // base_m)
    big = torch.iinfo(torch.int64).max
    for r0 in range(0, n, rows_per_chunk):
        r1 = min(n, r0 + rows_per_chunk)
        cnt = counts[r0:r1]
        todo = torch.arange(r1 - r0)
        m = base_m
        chosen = torch.full((r1 - r0, cmax), d, dtype=torch.int64)      # padded with d (sorts last)
        while todo.numel() > 0:
            u = torch.rand((todo.numel(), m), generator=g, dtype=torch.float64)
            if cdf is None:
                ranks = torch.clamp((u * d).to(torch.int64), max=d - 1)
            else:
                ranks = torch.clamp(torch.searchsorted(cdf, u), max=d - 1)
            pos = torch.arange(m, dtype=torch.int64).expand_as(ranks)
            key, _ = torch.sort(ranks * m + pos, dim=1)                  # by rank, then by draw position
            rk, ps = key // m, key % m
            first = torch.ones_like(rk, dtype=torch.bool)
            first[:, 1:] = rk[:, 1:] != rk[:, :-1]
            order_key = torch.where(first, ps * d + rk, torch.full_like(ps, big))
            order_key, _ = torch.sort(order_key, dim=1)                  # distinct ranks by first draw position
            ndist = first.sum(1)
            need = cnt[todo]
            ok = ndist >= need
            take = order_key[:, :cmax] if m >= cmax else torch.nn.functional.pad(order_key, (0, cmax - m), value=big)
            ids = take % d
            col = torch.arange(cmax).expand(todo.numel(), cmax)
            ids = torch.where((col < need[:, None]) & (take != big), ids, torch.full_like(ids, d))
            chosen[todo[ok]] = ids[ok]
            todo = todo[~ok]
            m *= 2                                                       # rare: a row ran out of distinct draws
        if rank_to_id is not None:
            valid = chosen < d
            chosen = torch.where(valid, rank_to_id[torch.clamp(chosen, max=d - 1)], chosen)
        chosen, _ = torch.sort(chosen, dim=1)
        mask = torch.arange(cmax).expand(r1 - r0, cmax) < cnt[:, None]
        out[int(indptr[r0]):int(indptr[r1])] = chosen[mask].to(torch.int32)
    return indptr, out


def _row_of_nnz(indptr: torch.Tensor) -> torch.Tensor:
    n = indptr.numel() - 1
    return torch.repeat_interleave(torch.arange(n, dtype=torch.int64), indptr[1:] - indptr[:-1])


def _row_sums(indptr: torch.Tensor, per_nnz: torch.Tensor) -> torch.Tensor:
    n = indptr.numel() - 1
    out = torch.zeros(n, dtype=per_nnz.dtype)
    out.index_add_(0, _row_of_nnz(indptr), per_nnz)
    return out


def _sparse_truth(d: int, density: float, g: torch.Generator) -> torch.Tensor:
    w = torch.zeros(d, dtype=torch.float64)
    nz = max(1, int(round(d * density)))
    idx = torch.randperm(d, generator=g)[:nz]
    w[idx] = torch.randn(nz, generator=g, dtype=torch.float64)
    return w


def hinge_dense(scale: int = 1, seed: int = 0) -> Workload:
    n, d = max(8, 10_000 // scale), 100
    g = _gen(seed)
    X = torch.randn((n, d), generator=g, dtype=torch.float32)
    w = torch.randn(d, generator=g, dtype=torch.float64)
    y = _sign_pm1(X.double() @ w + 0.1 * torch.randn(n, generator=g, dtype=torch.float64)).float()
    K = 4
    return Workload("hinge_dense", "hinge", "dense", n, d, X.reshape(-1).cpu().numpy(), y.cpu().numpy(), 1.0 / n, 10,
                    [Phase(0, K, seed, float(K))])


def hinge_csr(scale: int = 1, seed: int = 0, mean_nnz: float = 50.0, zipf_s: float = 1.1, K: int = 16,
              name: str = "hinge_csr", n_full: int = 1_000_000, d_full: int = 100_000, lam: float = 1e-5,
              rounds: int = 20) -> Workload:
    n, d = max(64, n_full // scale), max(256, d_full // scale)
    g = _gen(seed)
    counts = torch.clamp(torch.poisson(torch.full((n,), mean_nnz, dtype=torch.float64), generator=g), 1, d).to(torch.int64)
    rank_to_id = torch.randperm(d, generator=g)
    indptr, idx = _distinct_ids(counts, d, g, _zipf_cdf(d, zipf_s), rank_to_id)
    vals = torch.repeat_interleave(counts.double().rsqrt(), counts).float()
    w = _sparse_truth(d, 0.01, g)
    score = _row_sums(indptr, vals.double() * w[idx.long()])
    y = _sign_pm1(score)
    flip = torch.rand(n, generator=g, dtype=torch.float64) < 0.05
    y = torch.where(flip, -y, y).float()
    return Workload(name, "hinge", "csr", n, d, vals.cpu().numpy(), y.cpu().numpy(), lam * scale, rounds,
                    [Phase(0, K, seed, float(K))], indptr.cpu().numpy(), idx.cpu().numpy(),
                    meta={"lambda_note": "lambda*n kept constant when scaled"})


def logistic_dense(scale: int = 1, seed: int = 0) -> Workload:
    n, d = max(64, 11_000_000 // scale), 28
    g = _gen(seed)
    X = torch.randn((n, d), generator=g, dtype=torch.float32)
    mu = X.double().mean(0)
    sd = X.double().std(0, unbiased=False)
    X = ((X.double() - mu) / sd).float()
    w = torch.randn(d, generator=g, dtype=torch.float64)
    p = torch.sigmoid(X.double() @ w)
    y = torch.where(torch.rand(n, generator=g, dtype=torch.float64) < p, 1.0, -1.0).float()
    K = 32
    return Workload("logistic_dense", "logistic", "dense", n, d, X.reshape(-1).cpu().numpy(), y.cpu().numpy(), 1e-6 * scale, 20,
                    [Phase(0, K, seed, float(K))], meta={"lambda_note": "lambda*n kept at 11 when scaled"})


def hinge_hashed(scale: int = 1, seed: int = 0) -> Workload:
    n, d = max(256, 45_000_000 // scale), max(1024, 1_000_000 // scale)
    g = _gen(seed)
    nnz_row = 39
    counts = torch.full((n,), nnz_row, dtype=torch.int64)
    rank_to_id = torch.randperm(d, generator=g)
    indptr, idx = _distinct_ids(counts, d, g, _zipf_cdf(d, 1.05), rank_to_id)
    vals = torch.full((n * nnz_row,), 1.0 / math.sqrt(nnz_row), dtype=torch.float32)
    w = _sparse_truth(d, 0.01, g)
    score = _row_sums(indptr, vals.double() * w[idx.long()])
    score = score + 0.1 * torch.randn(n, generator=g, dtype=torch.float64)
    head = score[: min(n, 1_000_000)]
    thr = torch.quantile(head[: min(head.numel(), 1 << 24)], 0.75)
    y = torch.where(score > thr, 1.0, -1.0).float()
    return Workload("hinge_hashed", "hinge", "csr", n, d, vals.cpu().numpy(), y.cpu().numpy(), 1e-7 * scale, 30,
                    [Phase(0, 64, seed, 64.0), Phase(10, 16, seed + 1, 16.0)], indptr.cpu().numpy(), idx.cpu().numpy(),
                    meta={"lambda_note": "lambda*n kept at 4.5 when scaled"})


def ridge_csc(scale: int = 1, seed: int = 0, mean_nnz: float = 3700.0) -> Workload:
    n, d = max(32, 350_000 // scale), max(1024, 16_000_000 // scale)
    g = _gen(seed)
    counts = torch.clamp(torch.poisson(torch.full((n,), mean_nnz, dtype=torch.float64), generator=g), 1, d).to(torch.int64)
    indptr, idx = _distinct_ids(counts, d, g, None, None)
    vals = 1.0 - torch.rand(int(indptr[-1]), generator=g, dtype=torch.float64)        # U(0,1]
    norm = _row_sums(indptr, vals * vals).sqrt()
    rows = _row_of_nnz(indptr)
    vals = (vals / norm[rows]).float()
    w = _sparse_truth(d, 0.01, g)
    y = _row_sums(indptr, vals.double() * w[idx.long()]) + 0.01 * torch.randn(n, generator=g, dtype=torch.float64)
    # transpose to CSC: stable sort by column keeps rows ascending inside a column
    order = torch.sort(idx.long(), stable=True).indices
    col_counts = torch.bincount(idx.long(), minlength=d)
    colptr = torch.zeros(d + 1, dtype=torch.int64)
    colptr[1:] = torch.cumsum(col_counts, 0)
    K = 128
    return Workload("ridge_csc", "ridge", "csc", n, d, vals[order].cpu().numpy(), y.float().cpu().numpy(), 1e-4 * scale, 15,
                    [Phase(0, K, seed, float(K))], colptr.cpu().numpy(), rows[order].to(torch.int32).cpu().numpy())


CONFIGS = {
    "hinge_dense": hinge_dense,
    "hinge_csr": hinge_csr,
    "logistic_dense": logistic_dense,
    "hinge_hashed": hinge_hashed,
    "ridge_csc": ridge_csc,
}


def make(name: str, scale: int = 1, seed: int = 0, device: str = "cpu") -> Workload:
    """Draws a workload. ``device="cuda"`` draws with torch on the GPU (needed in practice for the two largest
    configurations at full size; the random stream differs from the CPU one) and returns host arrays all the same."""
    global _DEVICE
    prev = _DEVICE
    _DEVICE = device
    try:
        with torch.device(device):
            return CONFIGS[name](scale=scale, seed=seed)
    finally:
        _DEVICE = prev
