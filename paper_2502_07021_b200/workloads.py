"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NO Sinkhorn arithmetic: it only draws point clouds and histograms and
forms the dense cost / Gibbs-kernel matrices that are the *inputs* of the method
(C_il = ||x_i - y_l||^2 as in the paper's embedding-cost experiment, K = exp(-C/eps) as in
Section 1).  Both the CUDA path and the CPU checker are fed from here, so that they see
bit-identical fp32 arrays.

Recipe (all draws numpy ``default_rng(seed)`` = PCG64, everything computed in fp64 on the
host and rounded ONCE to fp32):
  points X seed 1000+cfg, points Y seed 2000+cfg, a seed 3000+cfg (+p for problem p of a
  batch), b seed 4000+cfg (+p);  Dirichlet(1) = i.i.d. Exp(1) normalised to sum 1;
  equal row blocks offsets[j] = j*n // c.

The five configurations (``n`` may be overridden to get a scaled-down copy of the same recipe):
  1  n=512    X,Y ~ U[0,1]^2 independent, raw cost, eps=0.05, a=b=1/n, c=4, scaling, 200 it
  2  n=4096   X ~ N(0,I_16), Y ~ N(0.5*1,I_16), cost / max, eps=0.1, Dirichlet a,b, c=8, 1000 it
  3  n=16384  X,Y ~ U[0,1]^8, raw cost, eps=0.01, Dirichlet a,b, c=16, LOG domain, 500 it,
              error trace every 10
  4  n=32768  X,Y ~ U[0,1]^32, cost / max, eps=0.2, a=b=1/n, c=32, scaling, 300 it
  5  n=8192   one cloud X ~ N(0,I_16) (symmetric cost), cost / max, eps=0.1,
              N=128 Dirichlet (a,b) pairs, c=1, scaling, 200 it
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

DOMAIN_SCALING = 0
DOMAIN_LOG = 1
KIND_KERNEL = 0
KIND_COST = 1

_SPECS = {
    1: dict(n=512, dim=2, cloud="uniform", two_clouds=True, normalize=False, eps=0.05, marg="uniform",
            c=4, domain=DOMAIN_SCALING, iters=200, nbatch=1, check_every=0),
    2: dict(n=4096, dim=16, cloud="gauss_shift", two_clouds=True, normalize=True, eps=0.1, marg="dirichlet",
            c=8, domain=DOMAIN_SCALING, iters=1000, nbatch=1, check_every=0),
    3: dict(n=16384, dim=8, cloud="uniform", two_clouds=True, normalize=False, eps=0.01, marg="dirichlet",
            c=16, domain=DOMAIN_LOG, iters=500, nbatch=1, check_every=10),
    4: dict(n=32768, dim=32, cloud="uniform", two_clouds=True, normalize=True, eps=0.2, marg="uniform",
            c=32, domain=DOMAIN_SCALING, iters=300, nbatch=1, check_every=0),
    5: dict(n=8192, dim=16, cloud="gauss", two_clouds=False, normalize=True, eps=0.1, marg="dirichlet",
            c=1, domain=DOMAIN_SCALING, iters=200, nbatch=128, check_every=0),
}


@dataclass
class Workload:
    cfg: int
    name: str
    n: int
    c: int
    offsets: np.ndarray          # int64 [c+1]
    eps: float
    domain: int
    iters: int
    nbatch: int
    check_every: int
    a: np.ndarray                # float32 [n] or [nbatch][n]
    b: np.ndarray
    K: np.ndarray | None = None  # float32 [n][n] Gibbs kernel (scaling-domain configs)
    C: np.ndarray | None = None  # float32 [n][n] cost
    X: np.ndarray | None = None  # float32 [n][dim] points of the first cloud (only with fp32_points)
    Y: np.ndarray | None = None  # float32 [n][dim] points of the second cloud (X itself for one cloud)
    cost_scale: float = 1.0      # C_il = cost_scale * |x_i - y_l|^2 (1 / largest squared distance, or 1)
    meta: dict = field(default_factory=dict)

    @property
    def matrix(self) -> np.ndarray:
        """The matrix the solver is given: C in the log domain, K otherwise."""
        return self.C if self.domain == DOMAIN_LOG else self.K

    @property
    def kind(self) -> int:
        return KIND_COST if self.domain == DOMAIN_LOG else KIND_KERNEL


def equal_offsets(n: int, c: int) -> np.ndarray:
    return np.array([j * n // c for j in range(c + 1)], dtype=np.int64)


def dirichlet1(rng: np.random.Generator, n: int) -> np.ndarray:
    e = rng.exponential(1.0, size=n)
    return e / e.sum()


def _points(kind: str, rng: np.random.Generator, n: int, dim: int, shifted: bool) -> np.ndarray:
    if kind == "uniform":
        return rng.random((n, dim))
    x = rng.standard_normal((n, dim))
    if kind == "gauss_shift" and shifted:
        x = x + 0.5
    return x


def _sqdist_rows(X: np.ndarray, Y: np.ndarray, ynorm: np.ndarray, r0: int, r1: int) -> np.ndarray:
    xb = X[r0:r1]
    d = (xb * xb).sum(1)[:, None] + ynorm[None, :] - 2.0 * (xb @ Y.T)
    np.maximum(d, 0.0, out=d)
    return d


def cost_and_kernel(X, Y, eps, normalize, want_cost=True, want_kernel=True, chunk=2048, rows=None):
    """Dense C_il = max(0, |x_i|^2 + |y_l|^2 - 2 x_i.y_l) (optionally divided by its maximum)
    and K = exp(-C/eps), built in fp64 row chunks and rounded once to fp32.  With rows = (lo, hi) only
    that row block is materialised (the maximum is still taken over the whole matrix)."""
    n = X.shape[0]
    ynorm = (Y * Y).sum(1)
    scale = 1.0
    cmax = 0.0
    for r0 in range(0, n, chunk):
        cmax = max(cmax, float(_sqdist_rows(X, Y, ynorm, r0, min(n, r0 + chunk)).max()))
    if normalize:
        scale = 1.0 / cmax
    lo, hi = (0, n) if rows is None else rows
    C32 = np.empty((hi - lo, n), dtype=np.float32) if want_cost else None
    K32 = np.empty((hi - lo, n), dtype=np.float32) if want_kernel else None
    for r0 in range(lo, hi, chunk):
        r1 = min(hi, r0 + chunk)
        d = _sqdist_rows(X, Y, ynorm, r0, r1)
        if normalize:
            d *= scale
        if want_cost:
            C32[r0 - lo:r1 - lo] = d
        if want_kernel:
            d *= -1.0 / eps
            np.exp(d, out=d)
            K32[r0 - lo:r1 - lo] = d
    return C32, K32, dict(raw_cost_max=cmax, cost_scale=scale)


def make(cfg: int, n: int | None = None, nbatch: int | None = None, c: int | None = None,
         offsets=None, want_cost: bool | None = None, want_kernel: bool | None = None, rows=None,
         fp32_points: bool = False) -> Workload:
    """Build configuration `cfg` (1..5).  `n`, `nbatch`, `c`/`offsets` override the stated sizes
    to get a smaller or differently partitioned copy of the same recipe.  `rows = (lo, hi)` materialises
    only that row block of the matrices (a, b stay whole): what one shard of a row partition holds.
    With `fp32_points` the clouds are rounded to fp32 BEFORE the cost is formed and are returned as X, Y
    together with cost_scale: the inputs of the implicit-kernel path (the matrices, if asked for, are then
    those of the rounded points, so that both paths describe the same problem)."""
    s = dict(_SPECS[cfg])
    n = int(s["n"] if n is None else n)
    nb = int(s["nbatch"] if nbatch is None else nbatch)
    if offsets is not None:
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        cc = off.size - 1
    else:
        cc = int(s["c"] if c is None else c)
        cc = max(1, min(cc, n))
        off = equal_offsets(n, cc)
    X = _points(s["cloud"], np.random.default_rng(1000 + cfg), n, s["dim"], shifted=False)
    Y = _points(s["cloud"], np.random.default_rng(2000 + cfg), n, s["dim"], shifted=True) if s["two_clouds"] else X
    if fp32_points:
        X32 = X.astype(np.float32)
        Y32 = X32 if Y is X else Y.astype(np.float32)
        X = X32.astype(np.float64)
        Y = X if Y32 is X32 else Y32.astype(np.float64)
    log = s["domain"] == DOMAIN_LOG
    if want_cost is None:
        want_cost = True if log else n <= 8192
    if want_kernel is None:
        want_kernel = not log
    C32, K32, meta = cost_and_kernel(X, Y, s["eps"], s["normalize"], want_cost, want_kernel, rows=rows)

    def marg(seed):
        if s["marg"] == "uniform":
            return np.full(n, 1.0 / n)
        return dirichlet1(np.random.default_rng(seed), n)

    if nb == 1:
        a = marg(3000 + cfg).astype(np.float32)
        b = marg(4000 + cfg).astype(np.float32)
    else:
        a = np.stack([marg(3000 + cfg + p) for p in range(nb)]).astype(np.float32)
        b = np.stack([marg(4000 + cfg + p) for p in range(nb)]).astype(np.float32)
    name = f"cfg{cfg}_n{n}" + (f"_N{nb}" if nb > 1 else "") + ("_log" if log else "_scaling") + f"_c{cc}"
    return Workload(cfg=cfg, name=name, n=n, c=cc, offsets=off, eps=float(s["eps"]), domain=s["domain"],
                    iters=int(s["iters"]), nbatch=nb, check_every=int(s["check_every"]), a=a, b=b,
                    K=K32, C=C32, meta=meta, X=X32 if fp32_points else None, Y=Y32 if fp32_points else None,
                    cost_scale=float(meta["cost_scale"]))


def additive_cost(n: int, seed: int = 7):
    """C_il = x_i + y_l (rank-one Gibbs kernel): the closed-form test instance.  Returns
    fp32 C and the fp64 vectors x, y that C was rounded from."""
    rng = np.random.default_rng(seed)
    x = rng.random(n)
    y = rng.random(n)
    return (x[:, None] + y[None, :]).astype(np.float32), x, y
