"""Seeded synthetic workloads for WP-SGD (shared by the CPU oracle's tests and the CUDA path).

This module only *generates inputs*: feature matrices, labels, shard offsets, per-node
step counts and the hyper-parameters of each workload.  It contains none of the method's
arithmetic (no SGD step, no sample draw, no combination weights), so that the oracle and
the CUDA library can both consume exactly the same arrays without sharing any code.

Workloads follow the shapes of the paper's experiments (Section "Numerical experiments":
k simulated nodes with unequal amounts of consumed data; sparse binary-like rows with a
few tens of features, unit-normalised rows) and the five benchmark configurations:

  1  k=4     dense fp32  d=64      hinge     steps 1000/800/500/250
  2  k=16    dense fp32  d=1024    logistic  steps 20000 x (1, .5, .25) cycling
  3  k=128   dense bf16  d=4096    squared   steps uniform in [5000, 50000]
  4  k=64    CSR d=2^20 ~40 nnz/row hinge    eta0/sqrt(n), steps 65536 x (1,.7,.4,.1) cycling
  5  k=1024  dense fp32  d=256     logistic  2^24 steps split by a speed ratio rho

Everything is a pure function of the integer data seed (1000 + config number) and of the
requested sizes; the sample-draw seed handed to the library is (config number - 1).
Generation uses torch ops so the large cases can be produced directly in device memory;
a CPU-generated and a CUDA-generated workload differ in values (different torch
generators) but not in distribution, and whoever consumes a workload must hand the *same*
tensors to both sides.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np
import torch

LOSS_HINGE, LOSS_LOGISTIC, LOSS_SQUARED = 0, 1, 2
LR_CONST, LR_INV_SQRT = 0, 1
X_F32, X_BF16 = 0, 1


@dataclasses.dataclass
class Workload:
    """One problem instance. Dense: X is [N, d] row-major (fp32 or bf16). Sparse: CSR."""

    name: str
    k: int
    d: int
    shard_off: np.ndarray  # int64 [k+1]; node j owns rows [off[j], off[j+1])
    n_steps: np.ndarray  # int64 [k]; steps node j runs
    eta0: float
    sched: int
    lam: float
    loss: int
    seed: int  # seed of the sample-index stream
    y: torch.Tensor  # float32 [N]
    X: Optional[torch.Tensor] = None  # dense features
    row_ptr: Optional[torch.Tensor] = None  # int64 [N+1]
    col_idx: Optional[torch.Tensor] = None  # int32 [nnz]
    val: Optional[torch.Tensor] = None  # float32 [nnz]
    w0: Optional[torch.Tensor] = None  # float32 [d] shared start or None (zeros)

    @property
    def sparse(self) -> bool:
        return self.row_ptr is not None

    @property
    def xtype(self) -> int:
        return X_BF16 if (self.X is not None and self.X.dtype == torch.bfloat16) else X_F32

    @property
    def total_steps(self) -> int:
        return int(self.n_steps.sum())

    def to(self, device) -> "Workload":
        def mv(t):
            return None if t is None else t.to(device)

        return dataclasses.replace(
            self, y=mv(self.y), X=mv(self.X), row_ptr=mv(self.row_ptr), col_idx=mv(self.col_idx),
            val=mv(self.val), w0=mv(self.w0))


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _equal_shards(k: int, m: int) -> np.ndarray:
    return (np.arange(k + 1, dtype=np.int64) * int(m)).astype(np.int64)


def _randn_rows(n_rows: int, d: int, std: float, g: torch.Generator, device, dtype=torch.float32,
                chunk_rows: int = 1 << 16) -> torch.Tensor:
    """N(0, std^2) rows, generated chunk by chunk in fp32 and converted once to `dtype`."""
    out = torch.empty((n_rows, d), dtype=dtype, device=device)
    for r0 in range(0, n_rows, chunk_rows):
        r1 = min(n_rows, r0 + chunk_rows)
        blk = torch.randn((r1 - r0, d), generator=g, device=device, dtype=torch.float32)
        if std != 1.0:
            blk.mul_(std)
        out[r0:r1] = blk.to(dtype)  # round-to-nearest-even for bf16
    return out


def _matvec_rows(X: torch.Tensor, w: torch.Tensor, chunk_rows: int = 1 << 16) -> torch.Tensor:
    """X @ w in fp32 by row chunks (label generation only)."""
    out = torch.empty(X.shape[0], dtype=torch.float32, device=X.device)
    for r0 in range(0, X.shape[0], chunk_rows):
        r1 = min(X.shape[0], r0 + chunk_rows)
        out[r0:r1] = X[r0:r1].float() @ w
    return out


def speed_split(k: int, total: int, rho: float) -> np.ndarray:
    """Split `total` steps over k nodes with linearly decreasing speeds, max/min = rho.

    s_j = 1 - (1 - 1/rho) j/(k-1); n_j = floor(total s_j / sum s); the remainder goes,
    one step each, to the lowest-numbered nodes.
    """
    j = np.arange(k, dtype=np.float64)
    s = 1.0 - (1.0 - 1.0 / float(rho)) * (j / max(k - 1, 1))
    n = np.floor(total * s / s.sum()).astype(np.int64)
    left = int(total - n.sum())
    n[:left] += 1
    return n


def config1(k=4, d=64, m=4096, n_steps=(1000, 800, 500, 250), device="cpu", data_seed=1001) -> Workload:
    g = _gen(device, data_seed)
    w_star = torch.randn(d, generator=g, device=device)
    X = _randn_rows(k * m, d, 1.0, g, device)
    s = _matvec_rows(X, w_star)
    y = torch.where(s >= 0, 1.0, -1.0).float()
    flip = torch.rand(k * m, generator=g, device=device) < 0.05
    y = torch.where(flip, -y, y).contiguous()
    n = np.asarray(list(n_steps)[:k] if len(n_steps) >= k else [n_steps[i % len(n_steps)] for i in range(k)],
                   dtype=np.int64)
    return Workload("config1", k, d, _equal_shards(k, m), n, 0.01, LR_CONST, 1e-3, LOSS_HINGE, 0, y, X=X)


def config2(k=16, d=1024, m=8192, base_steps=20000, device="cpu", data_seed=1002) -> Workload:
    g = _gen(device, data_seed)
    w_star = torch.randn(d, generator=g, device=device)
    X = _randn_rows(k * m, d, 1.0 / math.sqrt(d), g, device)
    p = torch.sigmoid(_matvec_rows(X, w_star))
    y = torch.where(torch.rand(k * m, generator=g, device=device) < p, 1.0, -1.0).float().contiguous()
    speeds = np.array([1.0, 0.5, 0.25])
    n = np.floor(base_steps * speeds[np.arange(k) % 3]).astype(np.int64)
    return Workload("config2", k, d, _equal_shards(k, m), n, 0.05, LR_CONST, 1e-4, LOSS_LOGISTIC, 1, y, X=X)


def config3(k=128, d=4096, m=32768, n_lo=5000, n_hi=50000, device="cpu", data_seed=1003) -> Workload:
    g = _gen(device, data_seed)
    w_star = torch.randn(d, generator=g, device=device)
    X = _randn_rows(k * m, d, 1.0 / math.sqrt(d), g, device, dtype=torch.bfloat16)
    y = _matvec_rows(X, w_star) + 0.1 * torch.randn(k * m, generator=g, device=device)
    u = np.random.default_rng(data_seed).random(k)
    n = (n_lo + np.floor(u * (n_hi - n_lo + 1))).astype(np.int64)
    return Workload("config3", k, d, _equal_shards(k, m), n, 0.01, LR_CONST, 1e-4, LOSS_SQUARED, 2,
                    y.float().contiguous(), X=X)


def _zipf_cdf(n: int, a: float, device) -> torch.Tensor:
    r = torch.arange(1, n + 1, dtype=torch.float64, device=device)
    c = torch.cumsum(r.pow(-a), 0)
    return c / c[-1]


def _zipf_draw(cdf: torch.Tensor, shape, g: torch.Generator) -> torch.Tensor:
    u = torch.rand(shape, generator=g, device=cdf.device, dtype=torch.float64)
    return torch.searchsorted(cdf, u).clamp_(max=cdf.numel() - 1)  # 0-based rank


def config4(k=64, d=1 << 20, m=65536, base_steps=65536, mean_nnz=40.0, max_nnz=128, device="cpu",
            data_seed=1004, chunk_rows: int = 1 << 18) -> Workload:
    """Sparse stand-in for the paper's KDD-Cup-like rows (a few tens of features, unit norm)."""
    g = _gen(device, data_seed)
    max_nnz = int(min(max_nnz, d))
    cdf = _zipf_cdf(d, 1.1, device)
    perm = torch.randperm(d, generator=g, device=device)  # rank -> column (hot columns scattered)
    # sparse w*: ceil(0.01 d) nonzeros on columns drawn from the same law
    n_star = max(1, math.ceil(0.01 * d))
    star_cols = perm[_zipf_draw(cdf, (n_star,), g)]
    star_vals = torch.randn(n_star, generator=g, device=device)
    # the hot columns are drawn more than once: the last draw of a column stands (written out on the host, in order,
    # because a device scatter with repeated indices keeps whichever write lands last)
    w_host = np.zeros(d, dtype=np.float32)
    w_host[star_cols.cpu().numpy()] = star_vals.cpu().numpy()
    w_star = torch.from_numpy(w_host).to(device)

    N = k * m
    nnz_all, cols_all, y_all = [], [], []
    lane = torch.arange(max_nnz, device=device)
    for r0 in range(0, N, chunk_rows):
        R = min(N, r0 + chunk_rows) - r0
        nnz = torch.poisson(torch.full((R,), float(mean_nnz), device=device), generator=g).long()
        nnz = nnz.clamp_(1, max_nnz)
        valid = lane[None, :] < nnz[:, None]
        ranks = _zipf_draw(cdf, (R, max_nnz), g)
        sentinel = d + lane[None, :].expand(R, -1)  # distinct padding, sorts after every rank
        ranks = torch.where(valid, ranks, sentinel)
        for _ in range(200):
            srt, order = torch.sort(ranks, dim=1)
            dup_sorted = torch.zeros_like(srt, dtype=torch.bool)
            dup_sorted[:, 1:] = (srt[:, 1:] == srt[:, :-1]) & (srt[:, 1:] < d)
            if not bool(dup_sorted.any()):
                break
            dup = torch.zeros_like(dup_sorted).scatter_(1, order, dup_sorted)
            fresh = _zipf_draw(cdf, (int(dup.sum()),), g)
            ranks[dup] = fresh
        else:  # pragma: no cover
            raise RuntimeError("could not make row features distinct")
        cols = torch.where(ranks < d, perm[ranks.clamp(max=d - 1)], torch.full_like(ranks, 1 << 40))
        cols, _ = torch.sort(cols, dim=1)  # valid columns first, ascending
        keep = lane[None, :] < nnz[:, None]
        flat_cols = cols[keep]
        vals_row = nnz.float().rsqrt()
        # label = sign(w* . x)
        contrib = torch.where(keep, w_star[cols.clamp(max=d - 1)], torch.zeros((), device=device))
        s = contrib.sum(1) * vals_row
        y_all.append(torch.where(s >= 0, 1.0, -1.0).float())
        nnz_all.append(nnz)
        cols_all.append(flat_cols.to(torch.int32))
    nnz = torch.cat(nnz_all)
    row_ptr = torch.zeros(N + 1, dtype=torch.int64, device=device)
    row_ptr[1:] = torch.cumsum(nnz, 0)
    col_idx = torch.cat(cols_all).contiguous()
    val = torch.repeat_interleave(nnz.float().rsqrt(), nnz).contiguous()
    speeds = np.array([1.0, 0.7, 0.4, 0.1])
    n = np.floor(base_steps * speeds[np.arange(k) % 4] + 1e-9).astype(np.int64)
    return Workload("config4", k, d, _equal_shards(k, m), n, 0.1, LR_INV_SQRT, 1e-5, LOSS_HINGE, 3,
                    torch.cat(y_all).contiguous(), row_ptr=row_ptr, col_idx=col_idx, val=val)


def config5(k=1024, d=256, m=2048, total_steps=1 << 24, rho=4.0, device="cpu", data_seed=1005) -> Workload:
    g = _gen(device, data_seed)
    w_star = torch.randn(d, generator=g, device=device)
    X = _randn_rows(k * m, d, 1.0 / math.sqrt(d), g, device)
    p = torch.sigmoid(_matvec_rows(X, w_star))
    y = torch.where(torch.rand(k * m, generator=g, device=device) < p, 1.0, -1.0).float().contiguous()
    n = speed_split(k, total_steps, rho)
    wl = Workload("config5", k, d, _equal_shards(k, m), n, 0.02, LR_CONST, 1e-3, LOSS_LOGISTIC, 4, y, X=X)
    wl.name = f"config5_rho{rho:g}"
    return wl


def densify(wl: Workload) -> Workload:
    """Dense fp32 copy of a (small) CSR workload, for sparse-vs-dense cross checks."""
    assert wl.sparse
    N = wl.row_ptr.numel() - 1
    X = torch.zeros((N, wl.d), dtype=torch.float32, device=wl.y.device)
    counts = (wl.row_ptr[1:] - wl.row_ptr[:-1])
    rows = torch.repeat_interleave(torch.arange(N, device=X.device), counts)
    X[rows, wl.col_idx.long()] = wl.val
    return dataclasses.replace(wl, X=X, row_ptr=None, col_idx=None, val=None, name=wl.name + "_dense")


def analog_rows(n_rows: int, d: int = 100000, device="cpu", data_seed=2001):
    """Rows after the paper's 'analog data' recipe (Section "Analog data"): 5-10 random
    features per row at random positions with random values, label 1 when
    sum_i x_i (i mod 4) (-1)^i > 0 else 0 (mapped here to +1/-1), rows scaled to unit length.
    Feature numbering i is 1-based as in the paper. Returns CSR (row_ptr, col_idx, val, y)."""
    g = _gen(device, data_seed)
    nnz = torch.randint(5, 11, (n_rows,), generator=g, device=device)
    L = 10
    lane = torch.arange(L, device=device)
    keep = lane[None, :] < nnz[:, None]
    cols = torch.randint(0, d, (n_rows, L), generator=g, device=device)
    for _ in range(100):
        pad = torch.where(keep, cols, d + lane[None, :].expand(n_rows, -1))
        srt, order = torch.sort(pad, dim=1)
        dup_s = torch.zeros_like(srt, dtype=torch.bool)
        dup_s[:, 1:] = (srt[:, 1:] == srt[:, :-1]) & (srt[:, 1:] < d)
        if not bool(dup_s.any()):
            break
        dup = torch.zeros_like(dup_s).scatter_(1, order, dup_s)
        cols[dup] = torch.randint(0, d, (int(dup.sum()),), generator=g, device=device)
    pad = torch.where(keep, cols, torch.full_like(cols, 1 << 40))
    cols, _ = torch.sort(pad, dim=1)
    vals = torch.rand((n_rows, L), generator=g, device=device) + 0.05
    vals = torch.where(keep, vals, torch.zeros((), device=device))
    i1 = cols.clamp(max=d - 1) + 1
    coef = (i1 % 4).float() * torch.where(i1 % 2 == 0, 1.0, -1.0)
    s = (vals * coef).sum(1)
    y = torch.where(s > 0, 1.0, -1.0).float()
    vals = vals / vals.pow(2).sum(1, keepdim=True).sqrt()
    row_ptr = torch.zeros(n_rows + 1, dtype=torch.int64, device=device)
    row_ptr[1:] = torch.cumsum(nnz, 0)
    return row_ptr, cols[keep].to(torch.int32).contiguous(), vals[keep].contiguous(), y


FULL = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def small(cfg: int, device="cpu") -> Workload:
    """Scaled-down copies the oracle finishes in seconds; sizes still span several tiles of
    the kernels and leave ragged tails (d not a multiple of the vector width where allowed)."""
    if cfg == 1:
        return config1(device=device)
    if cfg == 2:
        return config2(k=7, d=1024, m=512, base_steps=1500, device=device)
    if cfg == 3:
        return config3(k=9, d=4096, m=256, n_lo=200, n_hi=1200, device=device)
    if cfg == 4:
        return config4(k=8, d=1 << 14, m=2048, base_steps=3000, device=device)
    if cfg == 5:
        return config5(k=40, d=256, m=256, total_steps=40 * 700, rho=4.0, device=device)
    raise ValueError(cfg)
