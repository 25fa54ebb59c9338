"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded fp32 inputs.

Tolerances (from the target statement): relative error <= 1e-4 on u and v after 10 iterations
(log domain: |f - f_ref|/eps <= 1e-4, which is the relative error of u = exp(f/eps)); marginal
1-norm error <= 1e-5 at convergence, evaluated by the oracle in fp64 on the scalings the GPU
returns; <P,C> within relative 1e-5.
"""
import numpy as np
import pytest

import oracle
from paper_2502_07021_b200 import binding as fs
from paper_2502_07021_b200 import workloads
from gpu_util import GpuSolver, rel_err

pytestmark = pytest.mark.gpu

TOL_UV = 1e-4
TOL_L1 = 1e-5
TOL_COST = 1e-5
SC, LG = fs.FS_DOMAIN_SCALING, fs.FS_DOMAIN_LOG
KK, KC = fs.FS_MATRIX_KERNEL, fs.FS_MATRIX_COST


def rand_problem(n, seed, eps=0.3):
    rng = np.random.default_rng(seed)
    C = rng.random((n, n)).astype(np.float32)
    K = np.exp(-C.astype(np.float64) / eps).astype(np.float32)
    a = workloads.dirichlet1(np.random.default_rng(seed + 1), n).astype(np.float32)
    b = workloads.dirichlet1(np.random.default_rng(seed + 2), n).astype(np.float32)
    return C, K, a, b


def some_offsets(n, seed):
    rng = np.random.default_rng(seed)
    c = int(min(n, rng.integers(1, 6)))
    cuts = np.sort(rng.choice(np.arange(1, n), size=c - 1, replace=False)) if c > 1 else np.array([], dtype=np.int64)
    return np.concatenate([[0], cuts, [n]]).astype(np.int64)


# ------------------------------------------------------------------ single passes, many shapes

SIZES = [1, 2, 3, 5, 31, 33, 127, 129, 255, 300, 1000, 1023, 2049, 4100]


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("layout", ["dense", "padded", "misaligned"])
def test_single_passes_scaling(n, layout):
    eps = 0.3
    C, K, a, b = rand_problem(n, 10 + n, eps)
    ld = n if layout == "dense" else n + 8 - (n % 4) if layout == "padded" else n + 3
    mis = 1 if layout == "misaligned" else 0
    off = some_offsets(n, n)
    rng = np.random.default_rng(n)
    v0 = (rng.random(n) + 0.5).astype(np.float32)
    u0 = (rng.random(n) + 0.5).astype(np.float32)
    with GpuSolver(K, KK, eps, a, b, off, SC, ld=ld, misalign=mis) as g:
        g.set_scalings(u0, v0)
        fs.fs_row_pass(g.h, g.stream)
        u1, v1 = g.scalings()
        u_ref, _ = oracle.row_pass(K, oracle.KIND_KERNEL, eps, a, v0)
        assert rel_err(u1, u_ref) < 2e-6
        assert np.array_equal(v1, v0)
        fs.fs_col_pass(g.h, g.stream)
        u2, v2 = g.scalings()
        v_ref, _ = oracle.col_pass(K, oracle.KIND_KERNEL, eps, b, u1)   # from the GPU's own (fp32) u
        assert rel_err(v2, v_ref) < 2e-6
        assert np.array_equal(u2, u1)


@pytest.mark.parametrize("n", [1, 3, 33, 129, 300, 1023, 2049])
@pytest.mark.parametrize("layout", ["dense", "misaligned"])
def test_single_passes_log(n, layout):
    eps = 0.05
    C, K, a, b = rand_problem(n, 50 + n, eps)
    ld = n if layout == "dense" else n + 1
    mis = 1 if layout == "misaligned" else 0
    off = some_offsets(n, n + 1)
    rng = np.random.default_rng(n)
    g0 = (0.1 * rng.standard_normal(n)).astype(np.float32)
    f0 = (0.1 * rng.standard_normal(n)).astype(np.float32)
    with GpuSolver(C, KC, eps, a, b, off, LG, ld=ld, misalign=mis) as g:
        g.set_scalings(f0, g0)
        fs.fs_row_pass(g.h, g.stream)
        f1, g1 = g.scalings()
        f_ref = oracle.log_row_pass(C, eps, a, g0)
        assert np.max(np.abs(f1 - f_ref)) / eps < 2e-5
        assert np.array_equal(g1, g0)
        fs.fs_col_pass(g.h, g.stream)
        _, g2 = g.scalings()
        g_ref = oracle.log_col_pass(C, eps, b, f1)
        assert np.max(np.abs(g2 - g_ref)) / eps < 2e-5


# ------------------------------------------------------------------ ten iterations on the five configurations

def check_ten_iterations(w, offsets=None):
    off = w.offsets if offsets is None else np.asarray(offsets, dtype=np.int64)
    with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, off, w.domain) as g:
        g.iterate(10)
        x, y = g.scalings()
    if w.domain == SC:
        u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 10)
        assert rel_err(x, u) <= TOL_UV
        assert rel_err(y, v) <= TOL_UV
    else:
        f, gg = oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, 10)
        assert np.max(np.abs(x - f)) / w.eps <= TOL_UV
        assert np.max(np.abs(y - gg)) / w.eps <= TOL_UV


def test_config1_ten_iterations():
    check_ten_iterations(workloads.make(1))


def test_config1_unequal_blocks():
    check_ten_iterations(workloads.make(1), offsets=[0, 100, 101, 300, 512])


def test_config2_ten_iterations():
    check_ten_iterations(workloads.make(2))


def test_config2_unequal_blocks():
    check_ten_iterations(workloads.make(2), offsets=[0, 1, 1000, 1003, 4096])


def test_config3_scaled_down_ten_iterations():
    check_ten_iterations(workloads.make(3, n=2048))


def test_config4_scaled_down_ten_iterations():
    check_ten_iterations(workloads.make(4, n=8192 + 4))     # several tiles and a ragged tail


def batched_sample(w, U, V, iters, problems):
    for p in problems:
        u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a[p], w.b[p], iters)
        assert rel_err(U[p], u) <= TOL_UV, p
        assert rel_err(V[p], v) <= TOL_UV, p


@pytest.mark.parametrize("n,nb", [(96, 3), (1000, 5), (1024, 128), (777, 130)])
def test_config5_scaled_down_ten_iterations(n, nb):
    w = workloads.make(5, n=n, nbatch=nb)
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        g.iterate(10)
        U, V = g.scalings()
    batched_sample(w, U, V, 10, sorted({0, 1, nb // 2, nb - 1}))


@pytest.mark.parametrize("n,offsets", [(2048, None), (4100, None), (8192, [0, 5, 37, 4096, 4100, 8192]),
                                       (8200, None), (16384, None)])
def test_fused_single_read_iteration(n, offsets):
    """fs_iterate with the single-read fused kernel against the two-pass path and the oracle:
    column segments that end inside a CTA (n = 4100, 8200), row tiles cut by block boundaries,
    and a run long enough for the shared-memory ring and the exchange slots to wrap many times."""
    w = workloads.make(4, n=n)
    off = w.offsets if offsets is None else np.asarray(offsets, dtype=np.int64)
    res = {}
    for mode in (0, 2):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, off, SC) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, mode)
            if n <= 5120:
                fs.fs_set_option(g.h, fs.FS_OPT_PERSISTENT, 0)     # mode 0 is to be the two-pass graph path
            before = fs.fs_launch_count(g.h)
            g.iterate(10)
            assert fs.fs_launch_count(g.h) - before == (30 if mode == 0 else 20)
            res[mode] = g.scalings()
            row, col = g.errors(1)
            res[mode] += (row[0], col[0])
    u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 10)
    for mode in (0, 2):
        assert rel_err(res[mode][0], u) <= TOL_UV and rel_err(res[mode][1], v) <= TOL_UV
    assert rel_err(res[2][0], res[0][0]) < 1e-5 and rel_err(res[2][1], res[0][1]) < 1e-5
    assert abs(res[2][2] - res[0][2]) < 1e-6


@pytest.mark.parametrize("n,offsets", [(2048, None), (4100, None), (8192, [0, 5, 37, 4096, 4100, 8192]), (8200, None)])
def test_fused_single_read_iteration_log_domain(n, offsets):
    """The log-domain fused iteration (one exponential per element with the current duals as stabilisers,
    column sums from the same on-chip rows; out-of-range rows and columns redone inside its two kernels with
    a maximum as stabiliser) against the two-pass log path and the oracle."""
    w = workloads.make(3, n=n)
    off = w.offsets if offsets is None else np.asarray(offsets, dtype=np.int64)
    res = {}
    for mode in (0, 2):
        with GpuSolver(w.C, KC, w.eps, w.a, w.b, off, LG) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, mode)
            if n <= 5120:
                fs.fs_set_option(g.h, fs.FS_OPT_PERSISTENT, 0)     # mode 0 is to be the two-pass graph path
            before = fs.fs_launch_count(g.h)
            g.iterate(10)
            assert fs.fs_launch_count(g.h) - before == (30 if mode == 0 else 20)
            res[mode] = g.scalings()
            if mode == 2:
                # a cold start is out of the fast path's range (rows and columns are then redone with a maximum);
                # the fast path must carry the run after the first few iterations
                assert fs.fs_fused_log_fallbacks(g.h, g.stream) <= 3
            row, col = g.errors(1)
            res[mode] += (row[0], col[0])
    f, gg = oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, 10)
    for mode in (0, 2):
        assert np.max(np.abs(res[mode][0] - f)) / w.eps <= TOL_UV
        assert np.max(np.abs(res[mode][1] - gg)) / w.eps <= TOL_UV
    assert np.max(np.abs(res[2][0] - res[0][0])) / w.eps < 3e-5
    assert abs(res[2][2] - res[0][2]) < 2e-5 * max(1.0, res[0][2])


def test_fused_log_is_reproducible_and_traces():
    w = workloads.make(3, n=2048)
    runs = []
    for _ in range(2):
        with GpuSolver(w.C, KC, w.eps, w.a, w.b, w.offsets, LG) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, 2)
            fs.fs_set_error_trace(g.h, 4)
            g.iterate(9)
            runs.append(g.scalings() + fs.fs_error_trace(g.h, stream=g.stream))
    assert all(np.array_equal(x, y) for x, y in zip(runs[0], runs[1]))
    l1 = runs[0][2]
    assert len(l1) == 2
    for k, t in enumerate((4, 8)):
        f, gg = oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, t)
        e = oracle.marginal_errors(w.C, oracle.KIND_COST, w.eps, LG, f, gg, w.a, w.b)
        assert l1[k] == pytest.approx(e["row_l1"], rel=2e-3, abs=1e-6)


@pytest.mark.parametrize("n", [2048, 4100, 8192, 12288])
def test_fused_log_falls_back_after_a_jump_of_the_duals(n):
    """A jump of the duals by hundreds of eps between two iterations takes the marginals out of the fast
    path's fp32 range: the rows and columns concerned must be redone with a maximum, transparently.  The sizes
    cover 4, 2 and 1 rows per stage and a ragged last column group."""
    w = workloads.make(3, n=n)
    with GpuSolver(w.C, KC, w.eps, w.a, w.b, w.offsets, LG) as g:
        fs.fs_set_option(g.h, fs.FS_OPT_FUSED, 2)
        g.iterate(6)
        before = fs.fs_fused_log_fallbacks(g.h, g.stream)
        f6, g6 = g.scalings()
        shift = np.where(np.arange(w.n) % 2 == 0, 3.0, -3.0).astype(np.float32)    # +-300 eps
        g.set_scalings(f6, g6 + shift)
        g.iterate(4)
        assert fs.fs_fused_log_fallbacks(g.h, g.stream) > before
        fj, gj = g.scalings()
    with GpuSolver(w.C, KC, w.eps, w.a, w.b, w.offsets, LG) as g:
        fs.fs_set_option(g.h, fs.FS_OPT_FUSED, 0)
        g.set_scalings(f6, g6 + shift)
        g.iterate(4)
        f0, g0 = g.scalings()
    assert np.max(np.abs(fj - f0)) / w.eps < TOL_UV and np.max(np.abs(gj - g0)) / w.eps < TOL_UV


@pytest.mark.slow
@pytest.mark.parametrize("cfg", [3, 4])
def test_large_fused_iterations_are_reproducible(cfg):
    """The fused iteration kernels start while the stage-2 kernel before them is still running (dependent
    launch) and wait for it before they read its output; a read that came too early, or through a stale
    cache line, would show as run-to-run differences at sizes where every SM is busy: two runs of the same
    problem at n = 16384 must agree bit for bit, and with the two-pass path within its tolerance."""
    w = workloads.make(cfg, n=16384, want_cost=None if cfg == 3 else False)
    runs = []
    for mode in (1, 1, 0):
        with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, w.offsets, w.domain) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, mode)
            g.iterate(25)
            runs.append(g.scalings())
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])
    if cfg == 3:
        assert np.max(np.abs(runs[0][0] - runs[2][0])) / w.eps < 3e-5 and np.max(np.abs(runs[0][1] - runs[2][1])) / w.eps < 3e-5
    else:
        assert rel_err(runs[0][0], runs[2][0]) < 1e-5 and rel_err(runs[0][1], runs[2][1]) < 1e-5


@pytest.mark.slow
def test_fused_clusters_of_four_beyond_n_32768():
    """Rows longer than 32768 columns are split over clusters of four CTAs (S = 4); this is the only
    size class that takes that path, so it gets a (slow) case of its own: n = 36864, three iterations."""
    w = workloads.make(4, n=36864, want_cost=False)
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        before = fs.fs_launch_count(g.h)
        g.iterate(3)
        assert fs.fs_launch_count(g.h) - before == 6           # fused kernel + stage 2 per iteration
        x, y = g.scalings()
    u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 3)
    assert rel_err(x, u) <= TOL_UV and rel_err(y, v) <= TOL_UV


def test_fused_is_reproducible_and_traces():
    w = workloads.make(4, n=4096)
    runs = []
    for _ in range(2):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, 2)
            fs.fs_set_error_trace(g.h, 4)
            g.iterate(9)
            runs.append(g.scalings() + fs.fs_error_trace(g.h, stream=g.stream))
    assert all(np.array_equal(x, y) for x, y in zip(runs[0], runs[1]))
    l1 = runs[0][2]
    assert len(l1) == 2
    for k, t in enumerate((4, 8)):
        u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, t)
        e = oracle.marginal_errors(w.K, oracle.KIND_KERNEL, w.eps, SC, u, v, w.a, w.b)
        assert l1[k] == pytest.approx(e["row_l1"], rel=1e-3, abs=1e-6)


@pytest.mark.parametrize("n,nb", [(512, 32), (1000, 40), (2048, 128)])
def test_batched_engines_agree(n, nb):
    """The fp32 FMA engine and the tensor-core engine (bf16 hi/lo split, fp32 accumulation) run the
    same problem; both must meet the tolerance against the oracle and agree with each other."""
    w = workloads.make(5, n=n, nbatch=nb)
    res = {}
    for engine in (1, 2):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_BATCH_ENGINE, engine)
            g.iterate(10)
            res[engine] = g.scalings()
    for engine in (1, 2):
        batched_sample(w, res[engine][0], res[engine][1], 10, sorted({0, nb // 2, nb - 1}))
    assert rel_err(res[2][0], res[1][0]) < 5e-5 and rel_err(res[2][1], res[1][1]) < 5e-5


@pytest.mark.parametrize("n,nb", [(1024, 128), (4000, 100), (640, 1300), (1100, 1030)])
def test_batched_tensor_core_cluster_sizes(n, nb):
    """The tensor-core engine splits the contraction over a cluster of 8, 4, 2 or 1 CTAs depending on the
    number of output tiles (here: 8 tiles -> 8, 32 -> 4, 5 x 11 -> 2, 9 x 9 -> 1); every size goes through
    the exchange and the in-kernel update, with ragged row and problem tiles, and must match the oracle on
    sampled problems (the problems of a batch are independent)."""
    w = workloads.make(5, n=n, nbatch=nb)
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        g.iterate(10)
        U, V = g.scalings()
        row, col = g.errors(1)
    assert np.all(np.isfinite(U)) and np.all(U > 0) and np.all(np.isfinite(V)) and np.all(V > 0)
    assert row.shape == (nb,) and np.all(col < 1e-5)      # right after a column update its marginal is exact
    batched_sample(w, U, V, 10, sorted({0, 1, 63, 64, nb // 2, nb - 2, nb - 1}))


def test_batched_tensor_core_passes_are_reproducible():
    """Consecutive tensor-core passes overlap (a pass requests its first K tiles while its predecessor is
    finishing and waits for it before reading the operand it wrote): two runs must agree bit for bit."""
    w = workloads.make(5, n=4096, nbatch=128)
    runs = []
    for _ in range(2):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
            g.iterate(30)
            runs.append(g.scalings())
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])


def test_batched_tensor_core_engine_converges():
    w = workloads.make(5, n=1024, nbatch=64)
    check_converged(w, w.iters, w.C, problems=(0, 33, 63))


@pytest.mark.slow
def test_config3_full_size_ten_iterations():
    check_ten_iterations(workloads.make(3))


@pytest.mark.slow
def test_config4_full_size_ten_iterations():
    check_ten_iterations(workloads.make(4, want_cost=False))


@pytest.mark.slow
def test_config5_full_size_ten_iterations_sampled():
    w = workloads.make(5)
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        g.iterate(10)
        U, V = g.scalings()
    batched_sample(w, U, V, 10, range(w.nbatch))            # all 128 problems
    assert np.all(np.isfinite(U)) and np.all(U > 0) and np.all(np.isfinite(V)) and np.all(V > 0)


# ------------------------------------------------------------------ convergence: marginals and cost

def check_converged(w, iters, C_for_cost, problems=(0,), cost_problems=None):
    with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, w.offsets, w.domain) as g:
        g.iterate(iters)
        x, y = g.scalings()
        row_gpu, col_gpu = g.errors(1)
        row2_gpu, _ = g.errors(2)
        blk = fs.fs_block_errors(g.h, g.c)
        cost_gpu = g.cost(C_for_cost if w.domain == SC else None) if C_for_cost is not None else None
    batched = w.nbatch > 1
    for p in problems:
        xp, yp = (x[p], y[p]) if batched else (x, y)
        ap, bp = (w.a[p], w.b[p]) if batched else (w.a, w.b)
        e = oracle.marginal_errors(w.matrix, w.kind, w.eps, w.domain, xp, yp, ap, bp)
        assert e["row_l1"] <= TOL_L1 and e["col_l1"] <= TOL_L1, (p, e)
        # the library's own numbers describe the same state.  They are computed with the same fp32
        # sums that produced the scalings, so they can miss the part of the residual that is the
        # rounding error of those sums: about sqrt(n) * 2^-24 * mass, i.e. ~1e-6 for the batched
        # path (one chain of n products per output) and far less for the tree-shaped single sums.
        agree = 3e-6 if batched else 1e-6
        assert abs(row_gpu[p] - e["row_l1"]) <= agree
        assert abs(col_gpu[p] - e["col_l1"]) <= agree
        assert abs(row2_gpu[p] - e["row_l2"]) <= agree
        if C_for_cost is not None and (cost_problems is None or p in cost_problems):
            ref = oracle.objectives(w.matrix, w.kind, w.eps, w.domain, xp, yp, C_for_cost)["cost"]
            assert abs(cost_gpu[p] - ref) <= TOL_COST * abs(ref)
    if not batched:
        assert blk.sum() == pytest.approx(row_gpu[0], rel=1e-12, abs=1e-300)
    return x, y


def test_config1_converged():
    w = workloads.make(1)
    check_converged(w, w.iters, w.C)


def test_config2_converged():
    w = workloads.make(2)
    check_converged(w, w.iters, w.C)


def test_config3_scaled_down_converged():
    w = workloads.make(3, n=2048)
    check_converged(w, w.iters, w.C)


def test_config5_scaled_down_converged():
    w = workloads.make(5, n=1024, nbatch=16)
    check_converged(w, w.iters, w.C, problems=(0, 7, 15))


@pytest.mark.slow
def test_config3_full_size_converged():
    w = workloads.make(3)
    check_converged(w, w.iters, w.C)                          # <P,C> at full size, on the fused log path


@pytest.mark.slow
def test_config4_full_size_converged():
    w = workloads.make(4, want_cost=True)
    check_converged(w, w.iters, w.C)                          # <P,C> at full size, on the fused path


@pytest.mark.slow
def test_config5_full_size_converged_sampled():
    w = workloads.make(5)
    # marginals of all 128 problems; <P,C> (a serial n*n loop in the checker) on four of them
    check_converged(w, w.iters, w.C, problems=range(w.nbatch), cost_problems=(0, 41, 86, 127))


# ------------------------------------------------------------------ set-up step: K materialised from C

@pytest.mark.parametrize("n", [33, 512, 1001])
def test_kernel_materialised_from_cost(n):
    w = workloads.make(1, n=n)
    with GpuSolver(w.C, KC, w.eps, w.a, w.b, w.offsets, SC) as g:
        g.iterate(10)
        u1, v1 = g.scalings()
    u, v = oracle.sinkhorn_scaling(w.C, oracle.KIND_COST, w.eps, w.a, w.b, 10)
    assert rel_err(u1, u) <= TOL_UV and rel_err(v1, v) <= TOL_UV


# ------------------------------------------------------------------ structure: blocks, determinism, graphs, resume

def run(w, iters, offsets=None, graph=True, ld=None):
    off = w.offsets if offsets is None else np.asarray(offsets, dtype=np.int64)
    with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, off, w.domain, ld=ld) as g:
        fs.fs_set_option(g.h, fs.FS_OPT_USE_GRAPH, 1 if graph else 0)
        g.iterate(iters)
        return g.scalings()


def test_bit_reproducible_and_graph_equals_plain_launches():
    for w in (workloads.make(1), workloads.make(3, n=1024), workloads.make(5, n=256, nbatch=4)):
        x1, y1 = run(w, 7)
        x2, y2 = run(w, 7)
        x3, y3 = run(w, 7, graph=False)
        assert np.array_equal(x1, x2) and np.array_equal(y1, y2)
        assert np.array_equal(x1, x3) and np.array_equal(y1, y3)


def test_iterates_do_not_depend_on_block_layout():
    # Proposition 1 on one GPU: bit-identical when every offset is a multiple of the row-tile
    # height (32 rows at this size), equal to rounding otherwise.
    w = workloads.make(1)
    x0, y0 = run(w, 10, offsets=[0, 512])
    for off in ([0, 128, 256, 384, 512], [0, 32, 64, 512], list(range(0, 513, 32))):
        x, y = run(w, 10, offsets=off)
        assert np.array_equal(x, x0) and np.array_equal(y, y0), off
    x, y = run(w, 10, offsets=[0, 100, 101, 300, 512])
    assert rel_err(x, x0) < 1e-5 and rel_err(y, y0) < 1e-5
    xn, yn = run(w, 10, offsets=list(range(0, 513)))          # c = n
    assert rel_err(xn, x0) < 1e-5 and rel_err(yn, y0) < 1e-5


@pytest.mark.parametrize("cfg,n", [(1, 512), (3, 512)])
def test_checkpoint_resume_is_bit_identical(cfg, n):
    w = workloads.make(cfg, n=n)
    x10, y10 = run(w, 10)
    x5, y5 = run(w, 5)
    with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, w.offsets, w.domain) as g:
        g.set_scalings(x5, y5)
        g.iterate(5)
        x, y = g.scalings()
    assert np.array_equal(x, x10) and np.array_equal(y, y10)


def test_reset_restores_initial_state():
    w = workloads.make(1)
    with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, w.offsets, w.domain) as g:
        g.iterate(4)
        a1 = g.scalings()
        fs.fs_reset(g.h, g.stream)
        assert fs.fs_iterations_done(g.h) == 0
        u, v = g.scalings()
        assert np.all(u == 1) and np.all(v == 1)
        g.iterate(4)
        a2 = g.scalings()
    assert np.array_equal(a1[0], a2[0]) and np.array_equal(a1[1], a2[1])


def test_error_trace_matches_oracle():
    w = workloads.make(3, n=512)
    every, iters = 5, 23
    for graph in (True, False):
        with GpuSolver(w.C, KC, w.eps, w.a, w.b, w.offsets, LG) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_USE_GRAPH, int(graph))
            fs.fs_set_error_trace(g.h, every)
            g.iterate(12)
            g.iterate(3)      # ends on a check point (15): recorded by the extra evaluation pass
            g.iterate(8)
            l1, l2 = fs.fs_error_trace(g.h, stream=g.stream)
        assert len(l1) == 4                                    # states 5, 10, 15, 20
        for k, t in enumerate((5, 10, 15, 20)):
            f, gg = oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, t)
            e = oracle.marginal_errors(w.C, oracle.KIND_COST, w.eps, LG, f, gg, w.a, w.b)
            assert l1[k] == pytest.approx(e["row_l1"], rel=2e-3, abs=1e-6)
            assert l2[k] == pytest.approx(e["row_l2"], rel=2e-3, abs=1e-6)
    assert iters == 23


def test_launch_count_and_iteration_counter():
    w = workloads.make(1)
    with GpuSolver(w.matrix, w.kind, w.eps, w.a, w.b, w.offsets, w.domain) as g:
        fs.fs_set_option(g.h, fs.FS_OPT_RESIDENT, 0)
        before = fs.fs_launch_count(g.h)
        g.iterate(10)
        assert fs.fs_launch_count(g.h) - before == 30          # row pass + two column stages per iteration
        assert fs.fs_iterations_done(g.h) == 10
        fs.fs_set_option(g.h, fs.FS_OPT_RESIDENT, 1)
        before = fs.fs_launch_count(g.h)
        g.iterate(10)
        assert fs.fs_launch_count(g.h) - before == 1           # K-resident kernel: all iterations in one launch
        assert fs.fs_iterations_done(g.h) == 20


@pytest.mark.parametrize("n", [8, 9, 33, 100, 512, 590, 600, 640, 700, 720])
def test_resident_kernel_small_problems(n):
    """The K-resident persistent kernel (one cluster of 8 or 16 CTAs holds K in shared memory and runs all
    iterations in one launch) against the oracle and the two-pass graph path, with unequal blocks."""
    w = workloads.make(1, n=n)
    off = some_offsets(n, 7 * n)
    res = {}
    for mode in (0, 1):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, off, SC) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_RESIDENT, mode)
            before = fs.fs_launch_count(g.h)
            g.iterate(4)
            g.iterate(6)
            launches = fs.fs_launch_count(g.h) - before
            assert launches == (30 if mode == 0 else 2)
            res[mode] = g.scalings() + tuple(e[0] for e in g.errors(1))
    u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 10)
    for mode in (0, 1):
        assert rel_err(res[mode][0], u) <= TOL_UV and rel_err(res[mode][1], v) <= TOL_UV
    assert rel_err(res[1][0], res[0][0]) < 1e-5 and rel_err(res[1][1], res[0][1]) < 1e-5
    assert abs(res[1][2] - res[0][2]) < 1e-6


@pytest.mark.parametrize("cfg,n", [(1, 772), (1, 1024), (2, 1500), (2, 2048), (2, 3000), (2, 4096), (4, 5120)])
def test_persistent_kernel_mid_size_problems(cfg, n):
    """The grid-persistent kernel (one cooperative launch runs all iterations, one read of K per iteration,
    grid barriers between the phases) against the oracle and the two-pass graph path, with unequal blocks."""
    w = workloads.make(cfg, n=n)
    off = some_offsets(n, 11 * n)
    res = {}
    for mode in (0, 2):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, off, SC) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_PERSISTENT, mode)
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, 0)
            before = fs.fs_launch_count(g.h)
            g.iterate(4)
            g.iterate(6)
            launches = fs.fs_launch_count(g.h) - before
            assert launches == (30 if mode == 0 else 2), (mode, launches)
            res[mode] = g.scalings() + tuple(e[0] for e in g.errors(1))
    u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 10)
    for mode in (0, 2):
        assert rel_err(res[mode][0], u) <= TOL_UV and rel_err(res[mode][1], v) <= TOL_UV
    assert rel_err(res[2][0], res[0][0]) < 1e-5 and rel_err(res[2][1], res[0][1]) < 1e-5
    assert abs(res[2][2] - res[0][2]) < 1e-6


def test_persistent_kernel_is_reproducible_damped_and_flags_nonfinite():
    w = workloads.make(2, n=2048)
    runs = []
    for _ in range(2):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
            g.iterate(25)
            runs.append(g.scalings())
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        fs.fs_set_damping(g.h, 0.5)
        g.iterate(10)
        ud, vd = g.scalings()
    uo, vo = oracle.sinkhorn_damped(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 0.5, 10)
    assert rel_err(ud, uo) <= TOL_UV and rel_err(vd, vo) <= TOL_UV
    K = w.K.copy()
    K[100, :] = 0.0
    with GpuSolver(K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        g.iterate(2)
        with pytest.raises(fs.FsError) as ei:
            g.scalings()
        assert ei.value.code == fs.FS_ERR_NONFINITE


def test_resident_kernel_converges_and_flags_nonfinite():
    w = workloads.make(1)
    check_converged(w, w.iters, w.C)                          # default path for n = 512 is the resident kernel
    n = 64
    C, K, a, b = rand_problem(n, 5)
    K[7, :] = 0.0
    with GpuSolver(K, KK, 0.3, a, b, [0, n], SC) as g:
        g.iterate(2)
        with pytest.raises(fs.FsError) as ei:
            g.errors(1)
        assert ei.value.code == fs.FS_ERR_NONFINITE


# ------------------------------------------------------------------ relaxed (damped) updates, Section 3.3

@pytest.mark.parametrize("cfg,n,nb,eta", [(1, 512, 1, 0.5), (2, 2048, 1, 0.25), (4, 16384, 1, 0.5), (5, 1024, 64, 0.5),
                                          (5, 300, 4, 0.7)])
def test_damped_updates(cfg, n, nb, eta):
    """Every engine (two-pass, fused, batched FMA, batched tensor cores) against the oracle's relaxed
    iteration; eta = 1 must reproduce the plain run bit for bit."""
    w = workloads.make(cfg, n=n, nbatch=nb)
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        fs.fs_set_damping(g.h, eta)
        g.iterate(10)
        x, y = g.scalings()
    with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
        fs.fs_set_damping(g.h, 1.0)
        g.iterate(3)
        x1, y1 = g.scalings()
    x0, y0 = run(w, 3)
    assert np.array_equal(x1, x0) and np.array_equal(y1, y0)
    for p in ([0] if nb == 1 else sorted({0, nb - 1})):
        ap, bp = (w.a, w.b) if nb == 1 else (w.a[p], w.b[p])
        xp, yp = (x, y) if nb == 1 else (x[p], y[p])
        u, v = oracle.sinkhorn_damped(w.K, oracle.KIND_KERNEL, w.eps, ap, bp, eta, 10)
        assert rel_err(xp, u) <= TOL_UV and rel_err(yp, v) <= TOL_UV


@pytest.mark.parametrize("n", [8192, 16384])
def test_damped_fused_iteration_reads_the_old_scalings(n):
    """Section 3.3's relaxed update needs the OLD u_i in every thread that forms the new one, while the fused
    kernel overwrites u row by row.  ONE fused iteration with eta = 0.5 from a start whose two terms
    (1 - eta) u_i and eta a_i/q_i are of the same size: u, v against the oracle's relaxed iteration from the
    same start, bit-identical over 20 repeats, and equal to the two-pass path within rounding.  A thread that
    picked up an already updated u_i would be off by tens of percent."""
    w = workloads.make(4, n=n, want_cost=False)
    u3, v3 = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 3)
    rng = np.random.default_rng(n)
    u0 = (u3 * (0.5 + rng.random(n))).astype(np.float32)
    v0 = (v3 * (0.5 + rng.random(n))).astype(np.float32)
    uo, vo = oracle.sinkhorn_damped(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 0.5, 1, u0=u0, v0=v0)
    res = {}
    for mode in (2, 0):
        with GpuSolver(w.K, KK, w.eps, w.a, w.b, w.offsets, SC) as g:
            fs.fs_set_option(g.h, fs.FS_OPT_FUSED, mode)
            fs.fs_set_damping(g.h, 0.5)
            runs = []
            for _ in range(20 if mode == 2 else 1):
                g.set_scalings(u0, v0)
                g.iterate(1)
                runs.append(g.scalings())
            for x, y in runs[1:]:
                assert np.array_equal(x, runs[0][0]) and np.array_equal(y, runs[0][1])
            res[mode] = runs[0]
            assert rel_err(runs[0][0], uo) < 2e-6 and rel_err(runs[0][1], vo) < 2e-6
    assert rel_err(res[2][0], res[0][0]) < 2e-6 and rel_err(res[2][1], res[0][1]) < 2e-6


def test_damping_is_rejected_in_the_log_domain():
    w = workloads.make(3, n=256)
    with GpuSolver(w.C, KC, w.eps, w.a, w.b, w.offsets, LG) as g:
        with pytest.raises(fs.FsError) as ei:
            fs.fs_set_damping(g.h, 0.5)
        assert ei.value.code == fs.FS_ERR_UNSUPPORTED
        fs.fs_set_damping(g.h, 1.0)
        for bad in (0.0, 1.5, float("nan")):
            with pytest.raises(fs.FsError):
                fs.fs_set_damping(g.h, bad)


# ------------------------------------------------------------------ failures are reported, not trapped

def test_nonfinite_is_flagged():
    n = 64
    C, K, a, b = rand_problem(n, 5)
    K[7, :] = 0.0                                              # violates K > 0: q_7 = 0, u_7 = inf
    with GpuSolver(K, KK, 0.3, a, b, [0, n], SC) as g:
        g.iterate(1)
        with pytest.raises(fs.FsError) as ei:
            g.errors(1)
        assert ei.value.code == fs.FS_ERR_NONFINITE


def test_bounded_wait_gives_up_and_the_context_survives():
    """Failure detection without a fault: a wait that nothing satisfies runs out after its poll limit, the
    kernel returns, the host reads the status, and the library keeps working afterwards."""
    assert fs.fs_selftest_bounded_wait(2000, arrive=False) is True
    assert fs.fs_selftest_bounded_wait(2000, arrive=True) is False
    w = workloads.make(1, n=64)
    x, y = run(w, 3)
    u, v = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 3)
    assert rel_err(x, u) <= TOL_UV and rel_err(y, v) <= TOL_UV


def test_create_rejects_bad_marginals():
    import torch
    n = 32
    C, K, a, b = rand_problem(n, 6)
    Kd = torch.from_numpy(K).cuda()
    off = np.array([0, n], dtype=np.int64)

    def create(a_, b_):
        return fs.fs_create(n, 1, off, Kd, n, KK, 0.3, torch.from_numpy(a_).cuda(), torch.from_numpy(b_).cuda(), 1, SC)

    bad = a.copy()
    bad[3] = 0.0
    with pytest.raises(fs.FsError) as ei:
        create(bad, b)
    assert ei.value.code == fs.FS_ERR_NONPOSITIVE_MARGINAL
    bad = a.copy()
    bad[3] = np.nan
    with pytest.raises(fs.FsError) as ei:
        create(bad, b)
    assert ei.value.code == fs.FS_ERR_NONPOSITIVE_MARGINAL
    with pytest.raises(fs.FsError) as ei:
        create(a, (2 * b).astype(np.float32))
    assert ei.value.code == fs.FS_ERR_MASS_MISMATCH
    h = create(a, b)
    fs.fs_destroy(h)


def test_solve_host_matches_device_path():
    w = workloads.make(1)
    u = np.empty(w.n, dtype=np.float32)
    v = np.empty(w.n, dtype=np.float32)
    err = fs.fs_solve_host(w.n, w.c, w.offsets, w.K, w.n, KK, w.eps, w.a, w.b, 1, SC, 10, u, v)
    x, y = run(w, 10)
    assert np.array_equal(u, x) and np.array_equal(v, y)
    e = oracle.marginal_errors(w.K, oracle.KIND_KERNEL, w.eps, SC, u, v, w.a, w.b)
    assert abs(err[0] - e["row_l1"]) < 1e-6
