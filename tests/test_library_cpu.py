"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol that
include/fs.h declares, and rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2502_07021_b200 import binding as fs
from paper_2502_07021_b200 import build as fs_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fs_build.build()
    return fs.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fs_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert "fs_create" in names and "fs_iterate" in names and "fs_marginal_error" in names and "fs_scalings" in names
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(fs.exported_symbols())


def test_strerror_covers_all_codes(lib):
    seen = set()
    for code in range(0, -14, -1):
        msg = lib.fs_strerror(code).decode()
        assert msg and msg != "unknown error code"
        seen.add(msg)
    assert len(seen) == 14
    assert lib.fs_strerror(-99).decode() == "unknown error code"


def test_host_side_validation_needs_no_device(lib):
    out = ctypes.c_void_p()
    off = np.array([0, 4, 8], dtype=np.int64)
    offp = off.ctypes.data_as(ctypes.c_void_p)
    fake = 0x1000  # never dereferenced: every case below is rejected on the host

    def create(n=8, c=2, offsets=offp, M=fake, ld=8, kind=0, eps=0.1, a=fake, b=fake, nbatch=1, domain=0):
        return lib.fs_create(ctypes.byref(out), n, c, offsets, M, ld, kind, eps, a, b, nbatch, domain, None)

    assert lib.fs_create(None, 8, 2, offp, fake, 8, 0, 0.1, fake, fake, 1, 0, None) == fs.FS_ERR_NULL
    assert create(M=None) == fs.FS_ERR_NULL
    assert create(a=None) == fs.FS_ERR_NULL
    assert create(offsets=None) == fs.FS_ERR_NULL
    assert create(n=0) == fs.FS_ERR_BAD_N
    assert create(ld=7) == fs.FS_ERR_BAD_N
    assert create(nbatch=0) == fs.FS_ERR_BAD_N
    assert create(kind=3) == fs.FS_ERR_BAD_N
    assert create(domain=2) == fs.FS_ERR_BAD_N
    assert create(c=0) == fs.FS_ERR_BAD_OFFSETS
    assert create(c=9) == fs.FS_ERR_BAD_OFFSETS
    for bad in ([1, 4, 8], [0, 4, 7], [0, 0, 8], [0, 9, 8]):
        arr = np.array(bad, dtype=np.int64)
        assert create(offsets=arr.ctypes.data_as(ctypes.c_void_p)) == fs.FS_ERR_BAD_OFFSETS
    for eps in (0.0, -1.0, float("nan"), float("inf")):
        assert create(eps=eps) == fs.FS_ERR_BAD_EPS
    assert create(domain=1, kind=0) == fs.FS_ERR_DOMAIN
    assert create(domain=1, kind=1, nbatch=2) == fs.FS_ERR_UNSUPPORTED
    assert out.value is None

    def create_points(n=8, c=2, offsets=offp, X=fake, Y=fake, d=3, scale=1.0, eps=0.1, a=fake, b=fake):
        return lib.fs_create_points(ctypes.byref(out), n, c, offsets, X, Y, d, scale, eps, a, b, None)

    assert create_points(X=None) == fs.FS_ERR_NULL
    assert create_points(b=None) == fs.FS_ERR_NULL
    assert create_points(n=0) == fs.FS_ERR_BAD_N
    assert create_points(d=0) == fs.FS_ERR_BAD_N
    assert create_points(d=123) == fs.FS_ERR_UNSUPPORTED
    assert create_points(c=9) == fs.FS_ERR_BAD_OFFSETS
    assert create_points(eps=0.0) == fs.FS_ERR_BAD_EPS
    assert create_points(scale=-1.0) == fs.FS_ERR_BAD_EPS
    assert out.value is None
    # NULL handles
    assert lib.fs_iterate(None, 1, None) == fs.FS_ERR_NULL
    assert lib.fs_destroy(None) == fs.FS_ERR_NULL
    assert lib.fs_iterations_done(None) == -1


def test_checked_build_exports_the_same_interface_and_identifies_itself(lib):
    """The checked build (-DFS_DEBUG: canaries, launch checks, guarded stores) is a second library with the same
    C ABI; fs_debug_report tells the two apart without touching a device."""
    path = fs_build.build(debug=True)
    dbg = ctypes.CDLL(path)
    for name in declared_functions():
        assert hasattr(dbg, name), name
    for handle, expect in ((dbg, 1), (lib, 0)):
        flag = ctypes.c_int32(-1)
        fails = ctypes.c_int64(-1)
        assert handle.fs_debug_report(ctypes.byref(flag), ctypes.byref(fails), None, None) == fs.FS_OK
        assert flag.value == expect and fails.value == 0


def test_binding_refuses_missing_library(monkeypatch, tmp_path):
    monkeypatch.setattr(fs, "_lib", None)
    monkeypatch.setattr(fs, "LIB_PATH", str(tmp_path / "libfs_b200.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        fs.lib()
