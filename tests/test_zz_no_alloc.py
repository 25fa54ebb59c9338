"""fs_col_pass_static: the column half-step for callers that cannot allocate device memory
(a process whose own pool owns the whole GPU, a loop that cannot take the synchronisation an
allocation may cause, a plug-in that only receives input and output buffers).  Its partial sums
live in a fixed array inside the library, so every call shares that array and finds the previous
call's data in it.  The test therefore makes TWO calls in a row, the second on a different,
smaller problem, and checks each against the regular column pass (fs_create + fs_col_pass) and
against the fp64 CPU checker's column half-step, so that an error common to both GPU paths cannot
pass.  A third case runs the largest size the fixed array admits.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

import oracle
from paper_2502_07021_b200 import binding as fs
from paper_2502_07021_b200 import workloads

pytestmark = pytest.mark.gpu


def regular_col_pass(K, b, u, eps, torch, stream):
    n = K.shape[0]
    a = torch.full((n,), 1.0 / n, device="cuda:0")
    bn = b / b.sum() * a.sum()                   # the handle insists on equal masses; v scales with b
    off = np.array([0, n], dtype=np.int64)
    torch.cuda.synchronize()
    h = fs.fs_create(n, 1, off, K, K.stride(0), fs.FS_MATRIX_KERNEL, eps, a, bn, 1, fs.FS_DOMAIN_SCALING, stream)
    try:
        fs.fs_set_scalings(h, u, None, stream)
        fs.fs_col_pass(h, stream)
        v = torch.empty_like(u)
        fs.fs_scalings(h, None, v, stream)
    finally:
        fs.fs_destroy(h)
    return v, bn


def test_static_column_pass_matches_regular_on_two_calls_in_a_row():
    import torch
    stream = torch.cuda.Stream()
    for n, seed in ((4100, 1), (777, 2)):        # several tiles + ragged tail, then a smaller problem
        w = workloads.make(2, n=n)
        K = torch.from_numpy(w.K).cuda()
        rng = np.random.default_rng(seed)
        u = torch.from_numpy((rng.random(n) + 0.5).astype(np.float32)).cuda()
        b = torch.from_numpy(w.b).cuda()
        v_ref, bn = regular_col_pass(K, b, u, w.eps, torch, stream)
        v = torch.full_like(u, float("nan"))
        torch.cuda.synchronize()
        fs.fs_col_pass_static(K, n, n, u, bn, v, stream)
        stream.synchronize()
        got, ref = v.cpu().numpy().astype(np.float64), v_ref.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        assert np.max(np.abs(got - ref) / ref) < 2e-6, n
        v_or, _ = oracle.col_pass(w.K, oracle.KIND_KERNEL, w.eps, bn.cpu().numpy(), u.cpu().numpy())
        assert np.max(np.abs(got - v_or) / v_or) < 2e-6, n


def test_static_column_pass_at_its_largest_size_against_the_checker():
    import torch
    n = fs.FS_STATIC_MAX_N
    w = workloads.make(4, n=n, want_cost=False)
    stream = torch.cuda.Stream()
    K = torch.from_numpy(w.K).cuda()
    rng = np.random.default_rng(3)
    u_host = (rng.random(n) + 0.5).astype(np.float32)
    u = torch.from_numpy(u_host).cuda()
    b = torch.from_numpy(w.b).cuda()
    v = torch.full_like(u, float("nan"))
    torch.cuda.synchronize()
    fs.fs_col_pass_static(K, n, n, u, b, v, stream)
    stream.synchronize()
    v_or, _ = oracle.col_pass(w.K, oracle.KIND_KERNEL, w.eps, w.b, u_host)
    got = v.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got)) and np.max(np.abs(got - v_or) / v_or) < 2e-6


def test_static_column_pass_rejects_oversize_and_bad_arguments():
    import torch
    x = torch.ones(8, device="cuda:0")
    n = fs.FS_STATIC_MAX_N + 1
    assert fs.lib().fs_col_pass_static(x.data_ptr(), n, n, x.data_ptr(), x.data_ptr(), x.data_ptr(), None) == fs.FS_ERR_TOO_LARGE
    assert fs.lib().fs_col_pass_static(None, 8, 8, x.data_ptr(), x.data_ptr(), x.data_ptr(), None) == fs.FS_ERR_NULL
    assert fs.lib().fs_col_pass_static(x.data_ptr(), 4, 8, x.data_ptr(), x.data_ptr(), x.data_ptr(), None) == fs.FS_ERR_BAD_N
    assert "capacity" in fs.lib().fs_strerror(fs.FS_ERR_TOO_LARGE).decode()
