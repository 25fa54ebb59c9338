"""ctypes binding over the C ABI of libfs_b200.so -- argument marshalling only.

Every function here has the name and the argument order of its C counterpart in
``include/fs.h``; device buffers are passed as torch CUDA tensors (or raw integer addresses),
streams as ``torch.cuda.Stream`` / integer / None.  All arithmetic runs in the library's CUDA
kernels; there is no fallback: if the shared library has not been built, ``lib()`` raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

FS_DOMAIN_SCALING, FS_DOMAIN_LOG = 0, 1
FS_MATRIX_KERNEL, FS_MATRIX_COST = 0, 1
FS_OK = 0
FS_ERR_NULL, FS_ERR_BAD_N, FS_ERR_BAD_OFFSETS, FS_ERR_BAD_EPS = -1, -2, -3, -4
FS_ERR_NONPOSITIVE_MARGINAL, FS_ERR_MASS_MISMATCH, FS_ERR_DOMAIN = -5, -6, -7
FS_ERR_CUDA, FS_ERR_NONFINITE, FS_ERR_UNSUPPORTED, FS_ERR_TOO_LARGE, FS_ERR_TIMEOUT = -8, -9, -10, -11, -12
FS_ERR_INTERNAL = -13
FS_STATIC_MAX_N = 16384
FS_OPT_USE_GRAPH, FS_OPT_BATCH_ENGINE, FS_OPT_ROW_SHAPE, FS_OPT_COL_SHAPE, FS_OPT_FUSED, FS_OPT_RESIDENT, FS_OPT_PERSISTENT = 1, 2, 3, 4, 5, 6, 7

# FS_B200_DEBUG=1 in the environment selects the checked build (canaries, launch checks, guarded stores)
LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                        "libfs_b200_debug.so" if os.environ.get("FS_B200_DEBUG") == "1" else "libfs_b200.so")

_vp = ctypes.c_void_p
_i64 = ctypes.c_int64
_i32 = ctypes.c_int32
_int = ctypes.c_int
_dbl = ctypes.c_double
_SIGNATURES = {
    "fs_create": (_int, [ctypes.POINTER(_vp), _i64, _i32, _vp, _vp, _i64, _int, _dbl, _vp, _vp, _i32, _int, _vp]),
    "fs_iterate": (_int, [_vp, _i32, _vp]),
    "fs_row_pass": (_int, [_vp, _vp]),
    "fs_col_pass": (_int, [_vp, _vp]),
    "fs_marginal_error": (_int, [_vp, _int, _vp, _vp, _vp]),
    "fs_scalings": (_int, [_vp, _vp, _vp, _vp]),
    "fs_set_scalings": (_int, [_vp, _vp, _vp, _vp]),
    "fs_reset": (_int, [_vp, _vp]),
    "fs_transport_cost": (_int, [_vp, _vp, _i64, _vp, _vp]),
    "fs_set_damping": (_int, [_vp, _dbl]),
    "fs_set_error_trace": (_int, [_vp, _i32]),
    "fs_error_trace": (_int, [_vp, _vp, _vp, _i32, ctypes.POINTER(_i32), _vp]),
    "fs_block_errors": (_int, [_vp, _vp]),
    "fs_set_option": (_int, [_vp, _int, _i64]),
    "fs_iteration_path": (ctypes.c_char_p, [_vp]),
    "fs_iterations_done": (_i64, [_vp]),
    "fs_launch_count": (_i64, [_vp]),
    "fs_fused_log_fallbacks": (_int, [_vp, ctypes.POINTER(_i64), _vp]),
    "fs_destroy": (_int, [_vp]),
    "fs_solve_host": (_int, [_i64, _i32, _vp, _vp, _i64, _int, _dbl, _vp, _vp, _i32, _int, _i32, _vp, _vp, _vp]),
    "fs_create_points": (_int, [ctypes.POINTER(_vp), _i64, _i32, _vp, _vp, _vp, _i32, _dbl, _dbl, _vp, _vp, _vp]),
    "fs_solve_host_points": (_int, [_i64, _i32, _vp, _vp, _vp, _i32, _dbl, _dbl, _vp, _vp, _i32, _vp, _vp, _vp]),
    "fs_col_pass_static": (_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp]),
    "fs_shard_create": (_int, [ctypes.POINTER(_vp), _i64, _i64, _i64, _vp, _i64, _int, _dbl, _vp, _vp, _vp]),
    "fs_shard_row_pass": (_int, [_vp, _vp]),
    "fs_shard_col_partial": (_int, [_vp, _vp, _vp]),
    "fs_shard_fused_step": (_int, [_vp, _vp, _vp]),
    "fs_shard_col_finish": (_int, [_vp, _vp, _vp]),
    "fs_shard_col_finish_gathered": (_int, [_vp, _vp, _i32, _i64, _vp]),
    "fs_shard_col_block_pass": (_int, [_vp, _vp, _vp, _vp]),
    "fs_shard_local_u": (_int, [_vp, _vp, _vp]),
    "fs_shard_scalings": (_int, [_vp, _vp, _vp, _vp]),
    "fs_shard_set_scalings": (_int, [_vp, _vp, _vp, _vp]),
    "fs_shard_row_error": (_int, [_vp, _vp, _vp, _vp]),
    "fs_shard_destroy": (_int, [_vp]),
    "fs_selftest_bounded_wait": (_int, [_i32, _i32, ctypes.POINTER(_i32), _vp]),
    "fs_selftest_ex2_rate": (_int, [_i32, ctypes.POINTER(_dbl), _vp]),
    "fs_debug_report": (_int, [ctypes.POINTER(_i32), ctypes.POINTER(_i64), ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "fs_strerror": (ctypes.c_char_p, [_int]),
    "fs_last_cuda_error": (ctypes.c_char_p, []),
}

_lib = None


class FsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if code == FS_ERR_CUDA:
            detail = " [" + lib().fs_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {lib().fs_strerror(code).decode()} ({code}){detail}")


def lib() -> ctypes.CDLL:
    """Load libfs_b200.so (built by ``python -m paper_2502_07021_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2502_07021_b200.build` "
                               "(there is no CPU fallback)")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def exported_symbols():
    return sorted(_SIGNATURES)


def _dev(t):
    """Device address of a torch CUDA tensor (contiguity in the last dimension is the caller's
    contract), an integer address, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    return t.data_ptr()


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _check(code: int, where: str, allow=()):
    if code != FS_OK and code not in allow:
        raise FsError(code, where)
    return code


def _host(arr, dtype):
    a = np.ascontiguousarray(arr, dtype=dtype)
    return a, a.ctypes.data_as(_vp)


def fs_create(n, c, row_offsets, M_dev, ld, matrix_kind, eps, a_dev, b_dev, nbatch, domain, stream=None):
    off, offp = _host(row_offsets, np.int64)
    if off.shape != (c + 1,):
        raise FsError(FS_ERR_BAD_OFFSETS, "fs_create")
    out = _vp()
    _check(lib().fs_create(ctypes.byref(out), n, c, offp, _dev(M_dev), ld, matrix_kind, float(eps), _dev(a_dev),
                           _dev(b_dev), nbatch, domain, _stream(stream)), "fs_create")
    return out


def fs_create_points(n, c, row_offsets, X_dev, Y_dev, d, cost_scale, eps, a_dev, b_dev, stream=None):
    off, offp = _host(row_offsets, np.int64)
    if off.shape != (c + 1,):
        raise FsError(FS_ERR_BAD_OFFSETS, "fs_create_points")
    out = _vp()
    _check(lib().fs_create_points(ctypes.byref(out), n, c, offp, _dev(X_dev), _dev(Y_dev), d, float(cost_scale), float(eps),
                                  _dev(a_dev), _dev(b_dev), _stream(stream)), "fs_create_points")
    return out


def fs_iterate(s, k, stream=None):
    _check(lib().fs_iterate(s, k, _stream(stream)), "fs_iterate")


def fs_row_pass(s, stream=None):
    _check(lib().fs_row_pass(s, _stream(stream)), "fs_row_pass")


def fs_col_pass(s, stream=None):
    _check(lib().fs_col_pass(s, _stream(stream)), "fs_col_pass")


def fs_marginal_error(s, norm, nbatch=1, stream=None, allow_nonfinite=False):
    """Returns (row_err[nbatch], col_err[nbatch]) as float64 numpy arrays."""
    row = np.zeros(nbatch)
    col = np.zeros(nbatch)
    _check(lib().fs_marginal_error(s, norm, row.ctypes.data_as(_vp), col.ctypes.data_as(_vp), _stream(stream)),
           "fs_marginal_error", allow=(FS_ERR_NONFINITE,) if allow_nonfinite else ())
    return row, col


def fs_scalings(s, u_dev_out, v_dev_out, stream=None):
    return _check(lib().fs_scalings(s, _dev(u_dev_out), _dev(v_dev_out), _stream(stream)), "fs_scalings")


def fs_set_scalings(s, u_dev, v_dev, stream=None):
    _check(lib().fs_set_scalings(s, _dev(u_dev), _dev(v_dev), _stream(stream)), "fs_set_scalings")


def fs_reset(s, stream=None):
    _check(lib().fs_reset(s, _stream(stream)), "fs_reset")


def fs_transport_cost(s, C_dev, ldc, nbatch=1, stream=None):
    out = np.zeros(nbatch)
    _check(lib().fs_transport_cost(s, _dev(C_dev), ldc, out.ctypes.data_as(_vp), _stream(stream)), "fs_transport_cost")
    return out


def fs_set_damping(s, eta):
    _check(lib().fs_set_damping(s, float(eta)), "fs_set_damping")


def fs_set_error_trace(s, check_every):
    _check(lib().fs_set_error_trace(s, check_every), "fs_set_error_trace")


def fs_error_trace(s, cap=65536, stream=None):
    """Returns (l1[count], l2[count])."""
    l1 = np.zeros(cap)
    l2 = np.zeros(cap)
    cnt = _i32(0)
    _check(lib().fs_error_trace(s, l1.ctypes.data_as(_vp), l2.ctypes.data_as(_vp), cap, ctypes.byref(cnt),
                                _stream(stream)), "fs_error_trace")
    m = min(cnt.value, cap)
    return l1[:m], l2[:m]


def fs_block_errors(s, c):
    out = np.zeros(c)
    _check(lib().fs_block_errors(s, out.ctypes.data_as(_vp)), "fs_block_errors")
    return out


def fs_set_option(s, option, value):
    _check(lib().fs_set_option(s, option, value), "fs_set_option")


def fs_iteration_path(s):
    return lib().fs_iteration_path(s).decode()


def fs_iterations_done(s):
    return int(lib().fs_iterations_done(s))


def fs_launch_count(s):
    return int(lib().fs_launch_count(s))


def fs_fused_log_fallbacks(s, stream=None):
    out = _i64(0)
    _check(lib().fs_fused_log_fallbacks(s, ctypes.byref(out), _stream(stream)), "fs_fused_log_fallbacks")
    return int(out.value)


def fs_destroy(s):
    _check(lib().fs_destroy(s), "fs_destroy")


def fs_col_pass_static(K_dev, ld, n, u_dev, b_dev, v_dev, stream=None):
    """v = b / (K^T u) through the entry point that allocates nothing (n <= FS_STATIC_MAX_N)."""
    _check(lib().fs_col_pass_static(_dev(K_dev), ld, n, _dev(u_dev), _dev(b_dev), _dev(v_dev), _stream(stream)),
           "fs_col_pass_static")


def fs_shard_create(n, row_lo, m, M_dev, ld, matrix_kind, eps, a_local_dev, b_dev, stream=None):
    out = _vp()
    _check(lib().fs_shard_create(ctypes.byref(out), n, row_lo, m, _dev(M_dev), ld, matrix_kind, float(eps),
                                 _dev(a_local_dev), _dev(b_dev), _stream(stream)), "fs_shard_create")
    return out


def fs_shard_row_pass(s, stream=None):
    _check(lib().fs_shard_row_pass(s, _stream(stream)), "fs_shard_row_pass")


def fs_shard_col_partial(s, r_dev_out, stream=None):
    _check(lib().fs_shard_col_partial(s, _dev(r_dev_out), _stream(stream)), "fs_shard_col_partial")


def fs_shard_fused_step(s, r_dev_out, stream=None, allow_unsupported=False):
    """Row step and column partial from one read of the block; returns False when the fused kernel does not apply."""
    rc = _check(lib().fs_shard_fused_step(s, _dev(r_dev_out), _stream(stream)), "fs_shard_fused_step",
                allow=(FS_ERR_UNSUPPORTED,) if allow_unsupported else ())
    return rc == FS_OK


def fs_shard_col_finish(s, r_total_dev, stream=None):
    _check(lib().fs_shard_col_finish(s, _dev(r_total_dev), _stream(stream)), "fs_shard_col_finish")


def fs_shard_col_finish_gathered(s, parts_dev, nparts, pitch, stream=None):
    _check(lib().fs_shard_col_finish_gathered(s, _dev(parts_dev), nparts, pitch, _stream(stream)),
           "fs_shard_col_finish_gathered")


def fs_shard_col_block_pass(s, u_full_dev, v_block_dev_out, stream=None):
    _check(lib().fs_shard_col_block_pass(s, _dev(u_full_dev), _dev(v_block_dev_out), _stream(stream)),
           "fs_shard_col_block_pass")


def fs_shard_local_u(s, u_block_dev_out, stream=None):
    _check(lib().fs_shard_local_u(s, _dev(u_block_dev_out), _stream(stream)), "fs_shard_local_u")


def fs_shard_scalings(s, u_local_dev_out, v_dev_out, stream=None):
    _check(lib().fs_shard_scalings(s, _dev(u_local_dev_out), _dev(v_dev_out), _stream(stream)), "fs_shard_scalings")


def fs_shard_set_scalings(s, u_local_dev, v_dev, stream=None):
    _check(lib().fs_shard_set_scalings(s, _dev(u_local_dev), _dev(v_dev), _stream(stream)), "fs_shard_set_scalings")


def fs_shard_row_error(s, stream=None):
    """(sum |d|, sum d^2) of the local row residual seen by the last row pass."""
    l1, sq = _dbl(0.0), _dbl(0.0)
    _check(lib().fs_shard_row_error(s, ctypes.byref(l1), ctypes.byref(sq), _stream(stream)), "fs_shard_row_error")
    return l1.value, sq.value


def fs_shard_destroy(s):
    _check(lib().fs_shard_destroy(s), "fs_shard_destroy")


def fs_selftest_bounded_wait(poll_limit, arrive, stream=None):
    """True when the probe kernel's bounded wait ran out."""
    out = _i32(-1)
    _check(lib().fs_selftest_bounded_wait(poll_limit, 1 if arrive else 0, ctypes.byref(out), _stream(stream)),
           "fs_selftest_bounded_wait")
    return out.value == 1


def _host_ptr(x):
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        if x.is_cuda:
            raise ValueError("host buffers expected")
        return x.data_ptr()
    if x.dtype != np.float32 or not x.flags["C_CONTIGUOUS"]:
        raise ValueError("host buffers must be contiguous float32")
    return x.ctypes.data


def fs_solve_host_points(n, c, row_offsets, X_host, Y_host, d, cost_scale, eps, a_host, b_host, iters, u_out, v_out,
                         want_error=True):
    """Host point clouds in, host scalings out (numpy float32 or pinned torch CPU tensors); returns the 1-norm
    row marginal error (array of one) or None."""
    off, offp = _host(row_offsets, np.int64)
    err = np.zeros(1) if want_error else None
    _check(lib().fs_solve_host_points(n, c, offp, _host_ptr(X_host), _host_ptr(Y_host), d, float(cost_scale), float(eps),
                                      _host_ptr(a_host), _host_ptr(b_host), iters, _host_ptr(u_out), _host_ptr(v_out),
                                      err.ctypes.data_as(_vp) if want_error else None), "fs_solve_host_points")
    return err


def fs_debug_report():
    """dict(checked_build, canary_failures, launch_check_failures, allocations) of the loaded library."""
    cb, cf, lf, al = _i32(0), _i64(0), _i64(0), _i64(0)
    _check(lib().fs_debug_report(ctypes.byref(cb), ctypes.byref(cf), ctypes.byref(lf), ctypes.byref(al)), "fs_debug_report")
    return dict(checked_build=bool(cb.value), canary_failures=cf.value, launch_check_failures=lf.value,
                allocations=al.value)


def fs_selftest_ex2_rate(iters=4096, stream=None):
    """ex2.approx per second sustained by the special-function units (microbenchmark)."""
    out = _dbl(0.0)
    _check(lib().fs_selftest_ex2_rate(iters, ctypes.byref(out), _stream(stream)), "fs_selftest_ex2_rate")
    return out.value


def fs_solve_host(n, c, row_offsets, M_host, ld, matrix_kind, eps, a_host, b_host, nbatch, domain, iters,
                  u_out, v_out, want_error=True):
    """All buffers are host numpy arrays or pinned torch CPU tensors (float32).  u_out, v_out are
    written in place; returns the 1-norm row marginal error per problem (or None)."""
    off, offp = _host(row_offsets, np.int64)

    def hp(x):
        if x is None:
            return None
        if hasattr(x, "data_ptr"):
            if x.is_cuda:
                raise ValueError("fs_solve_host takes host buffers")
            return x.data_ptr()
        if x.dtype != np.float32 or not x.flags["C_CONTIGUOUS"] and x.ndim == 1:
            raise ValueError("host buffers must be float32")
        return x.ctypes.data
    err = np.zeros(nbatch) if want_error else None
    _check(lib().fs_solve_host(n, c, offp, hp(M_host), ld, matrix_kind, float(eps), hp(a_host), hp(b_host), nbatch,
                               domain, iters, hp(u_out), hp(v_out), err.ctypes.data_as(_vp) if want_error else None),
           "fs_solve_host")
    return err
