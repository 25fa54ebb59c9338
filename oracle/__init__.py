"""fp64 CPU oracle for the Sinkhorn hot path -- TEST INFRASTRUCTURE, not the product.

Thin ctypes wrapper around ``fs_oracle.c`` (plain C, fp64, ascending-index sums; see the
header of that file for what is computed and which passage of the paper each part
follows).  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library never does, and this package never imports it.

All functions take the fp32 arrays the GPU path receives (matrix, a, b) and return float64
numpy arrays.  ``kind`` is 0 when the matrix holds the Gibbs kernel K and 1 when it holds the
cost C (then K = exp(-C/eps) is evaluated in fp64).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

KIND_KERNEL = 0
KIND_COST = 1
DOMAIN_SCALING = 0
DOMAIN_LOG = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fs_oracle.c")
_LIB = os.path.join(_HERE, "_fs_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile fs_oracle.c into oracle/_fs_oracle.so with gcc (fp64, no contraction, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-Wall", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i64p = ctypes.POINTER(ctypes.c_int64)
_i64 = ctypes.c_int64
_i32 = ctypes.c_int32
_dbl = ctypes.c_double
_int = ctypes.c_int


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            sig = {
                "or_matvec_rows": [_i64, _f32p, _i64, _int, _dbl, _f64p, _i64, _i64, _f64p],
                "or_matvec_cols": [_i64, _f32p, _i64, _int, _dbl, _f64p, _i64, _i64, _f64p],
                "or_row_pass": [_i64, _f32p, _i64, _int, _dbl, _f32p, _f64p, _f64p, _f64p],
                "or_col_pass": [_i64, _f32p, _i64, _int, _dbl, _f32p, _f64p, _f64p, _f64p],
                "or_sinkhorn_scaling": [_i64, _f32p, _i64, _int, _dbl, _f32p, _f32p, _i64, _f64p, _f64p],
                "or_sinkhorn_damped": [_i64, _f32p, _i64, _int, _dbl, _f32p, _f32p, _dbl, _i64, _f64p, _f64p],
                "or_sinkhorn_protocol": [_i64, _i32, _i64p, _f32p, _i64, _int, _dbl, _f32p, _f32p, _i64,
                                         _f64p, _f64p, ctypes.POINTER(_i32)],
                "or_sinkhorn_rowpartition": [_i64, _i32, _i64p, _f32p, _i64, _int, _dbl, _f32p, _f32p,
                                             _i64, _f64p, _f64p],
                "or_lse_rows": [_i64, _f32p, _i64, _dbl, _f64p, _f64p],
                "or_lse_cols": [_i64, _f32p, _i64, _dbl, _f64p, _f64p],
                "or_log_row_pass": [_i64, _f32p, _i64, _dbl, _f32p, _f64p, _f64p],
                "or_log_col_pass": [_i64, _f32p, _i64, _dbl, _f32p, _f64p, _f64p],
                "or_sinkhorn_log": [_i64, _f32p, _i64, _dbl, _f32p, _f32p, _i64, _f64p, _f64p],
                "or_marginals_scaling": [_i64, _f32p, _i64, _int, _dbl, _f64p, _f64p, _f64p, _f64p],
                "or_marginals_log": [_i64, _f32p, _i64, _dbl, _f64p, _f64p, _f64p, _f64p],
                "or_marginal_errors": [_i64, _f64p, _f64p, _f32p, _f32p, _f64p],
                "or_cost_from_points": [_i64, _i64, _f32p, _f32p, _dbl, _f64p],
                "or_sinkhorn_points": [_i64, _i64, _f32p, _f32p, _dbl, _dbl, _f32p, _f32p, _i64, _f64p, _f64p],
                "or_marginals_points": [_i64, _i64, _f32p, _f32p, _dbl, _dbl, _f64p, _f64p, _f64p, _f64p],
                "or_plan": [_i64, _f32p, _i64, _int, _dbl, _int, _f64p, _f64p, _f64p],
                "or_objectives": [_i64, _f32p, _i64, _int, _dbl, _int, _f64p, _f64p, _f32p, _i64, _f64p],
            }
            for name, args in sig.items():
                fn = getattr(lib, name)
                fn.argtypes = args
                fn.restype = None
            _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS, else the visible cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        try:
            return max(1, int(env.split(",")[0]))
        except ValueError:
            pass
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _mat(M):
    M = np.asarray(M)
    if M.dtype != np.float32 or M.ndim != 2 or M.shape[0] != M.shape[1] or M.strides[1] != 4:
        raise ValueError("matrix must be a square float32 array with unit column stride")
    if M.strides[0] % 4:
        raise ValueError("row stride must be a multiple of 4 bytes")
    return M, M.shape[0], M.strides[0] // 4


def _f32(x, n):
    x = np.ascontiguousarray(x, dtype=np.float32)
    if x.shape != (n,):
        raise ValueError(f"expected a float32 vector of length {n}")
    return x


def _f64(x, n):
    x = np.array(x, dtype=np.float64, copy=True, order="C")
    if x.shape != (n,):
        raise ValueError(f"expected a vector of length {n}")
    return x


def _p32(x):
    return x.ctypes.data_as(_f32p)


def _p64(x):
    return x.ctypes.data_as(_f64p)


# ----------------------------------------------------------------------------- scaling domain

def row_pass(M, kind, eps, a, v):
    """(u, q) with q = K v and u = a / q."""
    M, n, ld = _mat(M)
    a = _f32(a, n)
    v = _f64(v, n)
    u = np.empty(n)
    q = np.empty(n)
    _load().or_row_pass(n, _p32(M), ld, kind, float(eps), _p32(a), _p64(v), _p64(u), _p64(q))
    return u, q


def col_pass(M, kind, eps, b, u):
    """(v, r) with r = K^T u and v = b / r."""
    M, n, ld = _mat(M)
    b = _f32(b, n)
    u = _f64(u, n)
    v = np.empty(n)
    r = np.empty(n)
    _load().or_col_pass(n, _p32(M), ld, kind, float(eps), _p32(b), _p64(u), _p64(v), _p64(r))
    return v, r


def sinkhorn_scaling(M, kind, eps, a, b, iters, u0=None, v0=None):
    """Centralized Sinkhorn-Knopp, `iters` full iterations from u0, v0 (default ones)."""
    M, n, ld = _mat(M)
    a, b = _f32(a, n), _f32(b, n)
    u = _f64(np.ones(n) if u0 is None else u0, n)
    v = _f64(np.ones(n) if v0 is None else v0, n)
    _load().or_sinkhorn_scaling(n, _p32(M), ld, kind, float(eps), _p32(a), _p32(b), int(iters),
                                _p64(u), _p64(v))
    return u, v


def sinkhorn_damped(M, kind, eps, a, b, eta, iters, u0=None, v0=None):
    """Relaxed iteration u <- (1-eta) u + eta a/(Kv), v <- (1-eta) v + eta b/(K^T u) from u0, v0 (default ones)."""
    M, n, ld = _mat(M)
    a, b = _f32(a, n), _f32(b, n)
    u = _f64(np.ones(n) if u0 is None else u0, n)
    v = _f64(np.ones(n) if v0 is None else v0, n)
    _load().or_sinkhorn_damped(n, _p32(M), ld, kind, float(eps), _p32(a), _p32(b), float(eta), int(iters),
                               _p64(u), _p64(v))
    return u, v


def _offsets(offsets, n):
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    if off.ndim != 1 or off.size < 2 or off[0] != 0 or off[-1] != n or np.any(np.diff(off) <= 0):
        raise ValueError("offsets must be strictly increasing from 0 to n")
    return off


def sinkhorn_protocol(M, kind, eps, a, b, offsets, iters, u0=None, v0=None):
    """Algorithm 1 with c logical clients; returns (u, v, all_clients_agree)."""
    M, n, ld = _mat(M)
    a, b = _f32(a, n), _f32(b, n)
    off = _offsets(offsets, n)
    u = _f64(np.ones(n) if u0 is None else u0, n)
    v = _f64(np.ones(n) if v0 is None else v0, n)
    agree = _i32(0)
    _load().or_sinkhorn_protocol(n, off.size - 1, off.ctypes.data_as(_i64p), _p32(M), ld, kind,
                                 float(eps), _p32(a), _p32(b), int(iters), _p64(u), _p64(v),
                                 ctypes.byref(agree))
    return u, v, bool(agree.value)


def sinkhorn_rowpartition(M, kind, eps, a, b, offsets, iters, u0=None, v0=None):
    """Strict row partition: r assembled as the sum of per-block partial transpose products."""
    M, n, ld = _mat(M)
    a, b = _f32(a, n), _f32(b, n)
    off = _offsets(offsets, n)
    u = _f64(np.ones(n) if u0 is None else u0, n)
    v = _f64(np.ones(n) if v0 is None else v0, n)
    _load().or_sinkhorn_rowpartition(n, off.size - 1, off.ctypes.data_as(_i64p), _p32(M), ld, kind,
                                     float(eps), _p32(a), _p32(b), int(iters), _p64(u), _p64(v))
    return u, v


def sinkhorn_batched(M, kind, eps, A, B, iters):
    """Shared-K multi-problem Sinkhorn: the centralized iteration applied to each (a, b) pair
    on its own; A, B are [N][n].  Returns U, V of the same shape."""
    A = np.asarray(A, dtype=np.float32)
    B = np.asarray(B, dtype=np.float32)
    U = np.empty(A.shape)
    V = np.empty(B.shape)
    for p in range(A.shape[0]):
        U[p], V[p] = sinkhorn_scaling(M, kind, eps, A[p], B[p], iters)
    return U, V


# ----------------------------------------------------------------------------- log domain

def lse_rows(C, eps, g):
    C, n, ld = _mat(C)
    g = _f64(g, n)
    L = np.empty(n)
    _load().or_lse_rows(n, _p32(C), ld, float(eps), _p64(g), _p64(L))
    return L


def lse_cols(C, eps, f):
    C, n, ld = _mat(C)
    f = _f64(f, n)
    L = np.empty(n)
    _load().or_lse_cols(n, _p32(C), ld, float(eps), _p64(f), _p64(L))
    return L


def log_row_pass(C, eps, a, g):
    C, n, ld = _mat(C)
    a = _f32(a, n)
    g = _f64(g, n)
    f = np.empty(n)
    _load().or_log_row_pass(n, _p32(C), ld, float(eps), _p32(a), _p64(g), _p64(f))
    return f


def log_col_pass(C, eps, b, f):
    C, n, ld = _mat(C)
    b = _f32(b, n)
    f = _f64(f, n)
    g = np.empty(n)
    _load().or_log_col_pass(n, _p32(C), ld, float(eps), _p32(b), _p64(f), _p64(g))
    return g


def sinkhorn_log(C, eps, a, b, iters, f0=None, g0=None):
    """Log-domain Sinkhorn, `iters` full iterations from f0, g0 (default zeros)."""
    C, n, ld = _mat(C)
    a, b = _f32(a, n), _f32(b, n)
    f = _f64(np.zeros(n) if f0 is None else f0, n)
    g = _f64(np.zeros(n) if g0 is None else g0, n)
    _load().or_sinkhorn_log(n, _p32(C), ld, float(eps), _p32(a), _p32(b), int(iters), _p64(f), _p64(g))
    return f, g


# ----------------------------------------------------------------------------- implicit kernel from points

def _points(X, Y):
    X = np.ascontiguousarray(X, dtype=np.float32)
    Y = np.ascontiguousarray(Y, dtype=np.float32)
    if X.ndim != 2 or X.shape != Y.shape:
        raise ValueError("X and Y must be float32 arrays of the same shape [n][d]")
    return X, Y, X.shape[0], X.shape[1]


def cost_from_points(X, Y, scale=1.0):
    """C_il = scale * |x_i - y_l|^2 as an n x n float64 array (X, Y: [n][d] float32)."""
    X, Y, n, d = _points(X, Y)
    C = np.empty((n, n))
    _load().or_cost_from_points(n, d, _p32(X), _p32(Y), float(scale), _p64(C))
    return C


def sinkhorn_points(X, Y, scale, eps, a, b, iters, u0=None, v0=None):
    """Sinkhorn-Knopp with K_il = exp(-scale |x_i - y_l|^2 / eps) evaluated on the fly; `iters` full
    iterations from u0, v0 (default ones)."""
    X, Y, n, d = _points(X, Y)
    a, b = _f32(a, n), _f32(b, n)
    u = _f64(np.ones(n) if u0 is None else u0, n)
    v = _f64(np.ones(n) if v0 is None else v0, n)
    _load().or_sinkhorn_points(n, d, _p32(X), _p32(Y), float(scale), float(eps), _p32(a), _p32(b), int(iters),
                               _p64(u), _p64(v))
    return u, v


def marginal_errors_points(X, Y, scale, eps, u, v, a, b):
    """dict(row_l1, row_l2, col_l1, col_l2) of the implicit-kernel plan's marginals against a and b."""
    X, Y, n, d = _points(X, Y)
    u, v = _f64(u, n), _f64(v, n)
    row, col = np.empty(n), np.empty(n)
    _load().or_marginals_points(n, d, _p32(X), _p32(Y), float(scale), float(eps), _p64(u), _p64(v), _p64(row), _p64(col))
    return marginal_error_norms(row, col, a, b)


# ----------------------------------------------------------------------------- errors, objectives

def marginals(M, kind, eps, domain, x, y):
    """(row, col) marginals of the plan defined by scalings (domain 0) or duals (domain 1)."""
    M, n, ld = _mat(M)
    x, y = _f64(x, n), _f64(y, n)
    row, col = np.empty(n), np.empty(n)
    if domain == DOMAIN_SCALING:
        _load().or_marginals_scaling(n, _p32(M), ld, kind, float(eps), _p64(x), _p64(y), _p64(row), _p64(col))
    else:
        if kind != KIND_COST:
            raise ValueError("the log domain needs the cost matrix")
        _load().or_marginals_log(n, _p32(M), ld, float(eps), _p64(x), _p64(y), _p64(row), _p64(col))
    return row, col


def marginal_error_norms(row, col, a, b):
    """dict(row_l1, row_l2, col_l1, col_l2): 1-norm and 2-norm of row - a and of col - b for given marginals."""
    n = np.asarray(row).size
    row, col = _f64(row, n), _f64(col, n)
    a, b = _f32(a, n), _f32(b, n)
    err = np.empty(4)
    _load().or_marginal_errors(n, _p64(row), _p64(col), _p32(a), _p32(b), _p64(err))
    return dict(row_l1=err[0], row_l2=err[1], col_l1=err[2], col_l2=err[3])


def marginal_errors(M, kind, eps, domain, x, y, a, b):
    """dict(row_l1, row_l2, col_l1, col_l2) of the plan's marginals against a and b."""
    row, col = marginals(M, kind, eps, domain, x, y)
    return marginal_error_norms(row, col, a, b)


def plan(M, kind, eps, domain, x, y):
    """Dense transport plan P (n x n float64)."""
    M, n, ld = _mat(M)
    x, y = _f64(x, n), _f64(y, n)
    P = np.empty((n, n))
    _load().or_plan(n, _p32(M), ld, kind, float(eps), domain, _p64(x), _p64(y), _p64(P))
    return P


def objectives(M, kind, eps, domain, x, y, C):
    """dict(cost=<P,C>, primal=Eq. 1 objective, mass=sum P)."""
    M, n, ld = _mat(M)
    C, n2, ldc = _mat(C)
    if n2 != n:
        raise ValueError("C and M sizes differ")
    x, y = _f64(x, n), _f64(y, n)
    out = np.empty(3)
    _load().or_objectives(n, _p32(M), ld, kind, float(eps), domain, _p64(x), _p64(y), _p32(C), ldc, _p64(out))
    return dict(cost=out[0], primal=out[1], mass=out[2])


def dual_value(eps, f, g, a, b, mass):
    """Dual objective of Eq. 1 at (f, g): <f,a> + <g,b> - eps * sum_il exp((f_i+g_l-C_il)/eps),
    the last sum being the plan's total mass."""
    return float(np.dot(np.asarray(f, np.float64), np.asarray(a, np.float64))
                 + np.dot(np.asarray(g, np.float64), np.asarray(b, np.float64)) - eps * mass)
