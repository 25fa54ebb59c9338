"""The checked build of the library (-DFS_DEBUG) in place of a memory-checking tool: every owned device buffer
carries 256 canary bytes that are verified when it is freed, launchers verify their geometry, and the stores into
partial-result buffers are guarded.  The smallest and most ragged sizes (1, 2, 3, 31, 33, 127, 129) and one size
per kernel family go through it in a child process (the library variant is chosen when it is first loaded), are
compared with the fp64 checker, and must leave every counter at zero."""
import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    sys.path.insert(0, %r)
    import numpy as np, torch
    import oracle
    from paper_2502_07021_b200 import binding as fs, workloads
    from gpu_util import GpuSolver, rel_err
    assert fs.LIB_PATH.endswith("libfs_b200_debug.so")
    assert fs.fs_debug_report()["checked_build"]
    SC, LG, KK, KC = fs.FS_DOMAIN_SCALING, fs.FS_DOMAIN_LOG, fs.FS_MATRIX_KERNEL, fs.FS_MATRIX_COST
    cases = 0
    for n in (1, 2, 3, 31, 33, 127, 129):
        w = workloads.make(1, n=n)
        off = [0, n] if n < 3 else [0, 1, n - 1, n]
        for ld, mis in ((n, 0), (n + 3, 1)):
            with GpuSolver(w.K, KK, w.eps, w.a, w.b, off, SC, ld=ld, misalign=mis) as g:
                fs.fs_set_option(g.h, fs.FS_OPT_RESIDENT, 0)
                g.iterate(5)
                x, y = g.scalings()
                g.errors(1)
            u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 5)
            assert rel_err(x, u) < 1e-4 and rel_err(y, v) < 1e-4, n
            cases += 1
        with GpuSolver(w.C, KC, w.eps, w.a, w.b, off, LG) as g:
            g.iterate(5)
            x, y = g.scalings()
            g.errors(2)
        f, gg = oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, 5)
        assert np.max(np.abs(x - f)) / w.eps < 1e-4 and np.max(np.abs(y - gg)) / w.eps < 1e-4, n
        cases += 1
    # one size per kernel family: resident, persistent, fused, fused log, batched (both engines), implicit, shards
    for cfg, n, nb, opts in ((1, 129, 1, {}), (2, 1500, 1, {}), (4, 2052, 1, {fs.FS_OPT_FUSED: 2}), (3, 2052, 1, {fs.FS_OPT_FUSED: 2}),
                             (5, 300, 3, {}), (5, 640, 40, {})):
        w = workloads.make(cfg, n=n, nbatch=nb)
        with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, w.offsets, w.domain) as g:
            for k, val in opts.items():
                fs.fs_set_option(g.h, k, val)
            g.iterate(6)
            x, y = g.scalings()
            g.errors(1)
        if w.domain == LG:
            f, gg = oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, 6)
            assert np.max(np.abs(x - f)) / w.eps < 1e-4
        elif nb == 1:
            u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 6)
            assert rel_err(x, u) < 1e-4 and rel_err(y, v) < 1e-4
        else:
            u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a[nb - 1], w.b[nb - 1], 6)
            assert rel_err(x[nb - 1], u) < 1e-4 and rel_err(y[nb - 1], v) < 1e-4
        cases += 1
    w = workloads.make(2, n=333, fp32_points=True, want_cost=False, want_kernel=False)
    dev = torch.device("cuda:0")
    st = torch.cuda.Stream()
    X, Y = torch.from_numpy(w.X).to(dev), torch.from_numpy(w.Y).to(dev)
    a, b = torch.from_numpy(w.a).to(dev), torch.from_numpy(w.b).to(dev)
    h = fs.fs_create_points(w.n, w.c, w.offsets, X, Y, w.X.shape[1], w.cost_scale, w.eps, a, b, st)
    fs.fs_iterate(h, 6, st)
    xo, yo = torch.empty_like(a), torch.empty_like(b)
    fs.fs_scalings(h, xo, yo, st)
    fs.fs_destroy(h)
    u, v = oracle.sinkhorn_points(w.X, w.Y, w.cost_scale, w.eps, w.a, w.b, 6)
    assert rel_err(xo.cpu().numpy(), u) < 1e-4 and rel_err(yo.cpu().numpy(), v) < 1e-4
    cases += 1
    torch.cuda.synchronize()
    rep = fs.fs_debug_report()
    print("REPORT", cases, rep["canary_failures"], rep["launch_check_failures"], rep["allocations"], flush=True)
""")


def test_tiny_and_ragged_sizes_through_the_checked_build(tmp_path):
    from paper_2502_07021_b200 import build as fs_build
    fs_build.build(debug=True)                     # no-op when libfs_b200_debug.so is up to date
    script = tmp_path / "checked_child.py"
    script.write_text(CHILD % (ROOT, os.path.join(ROOT, "tests")))
    env = dict(os.environ, FS_B200_DEBUG="1")
    out = subprocess.run([sys.executable, str(script)], env=env, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-3000:]
    line = [ln for ln in out.stdout.splitlines() if ln.startswith("REPORT")][-1].split()
    cases, canary, launch, allocs = (int(t) for t in line[1:])
    assert cases == 7 * 3 + 6 + 1
    assert canary == 0 and launch == 0, out.stderr[-3000:]
    assert allocs > 300
    assert "fs debug:" not in out.stderr
