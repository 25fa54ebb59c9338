"""Row-partitioned shards (Section 3.1) on ONE GPU: G shard handles are created on the row blocks of the
same problem and stepped one after the other, the all-reduce of the per-shard column partials being a
plain rank-order sum on the device.  This checks the three device steps and the exchange pattern that
`distributed.sharded_iterate` runs with one process per GPU; no kernel here waits on another."""
import numpy as np
import pytest

import oracle
from paper_2502_07021_b200 import binding as fs
from paper_2502_07021_b200 import distributed as fsdist
from paper_2502_07021_b200 import workloads

pytestmark = pytest.mark.gpu


def run_shards(w, G, iters, kind=fs.FS_MATRIX_KERNEL):
    import torch
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(device=dev)
    M = w.K if kind == fs.FS_MATRIX_KERNEL else w.C
    b = torch.from_numpy(w.b).to(dev)
    shards, blocks, keep = [], [], []
    for r in range(G):
        lo, hi = fsdist.row_range(w.n, r, G)
        Mb = torch.from_numpy(np.ascontiguousarray(M[lo:hi])).to(dev)
        ab = torch.from_numpy(w.a[lo:hi].copy()).to(dev)
        keep += [Mb, ab]
        torch.cuda.synchronize()
        shards.append(fs.fs_shard_create(w.n, lo, hi - lo, Mb, w.n, kind, w.eps, ab, b, stream))
        blocks.append((lo, hi))
    parts = [torch.empty(w.n, dtype=torch.float32, device=dev) for _ in range(G)]
    total = torch.empty(w.n, dtype=torch.float32, device=dev)
    try:
        with torch.cuda.stream(stream):
            for _ in range(iters):
                for s in shards:
                    fs.fs_shard_row_pass(s, stream)
                for s, p in zip(shards, parts):
                    fs.fs_shard_col_partial(s, p, stream)
                total.copy_(parts[0])
                for p in parts[1:]:
                    total.add_(p)                  # the all-reduce, in rank order
                for s in shards:
                    fs.fs_shard_col_finish(s, total, stream)
        u = np.empty(w.n, dtype=np.float32)
        v_all = []
        l1 = 0.0
        for s, (lo, hi) in zip(shards, blocks):
            ub = torch.empty(hi - lo, dtype=torch.float32, device=dev)
            vb = torch.empty(w.n, dtype=torch.float32, device=dev)
            fs.fs_shard_scalings(s, ub, vb, stream)
            u[lo:hi] = ub.cpu().numpy()
            v_all.append(vb.cpu().numpy())
            l1 += fs.fs_shard_row_error(s, stream)[0]
    finally:
        for s in shards:
            fs.fs_shard_destroy(s)
    return u, v_all, l1


@pytest.mark.parametrize("n,G", [(1000, 1), (1000, 3), (4100, 4), (8192, 2)])
def test_shards_reproduce_the_row_partition_iterates(n, G):
    w = workloads.make(2, n=n)
    u, v_all, l1 = run_shards(w, G, 10)
    for vb in v_all[1:]:
        assert np.array_equal(vb, v_all[0])          # every shard holds the same v
    off = [fsdist.row_range(n, r, G)[0] for r in range(G)] + [n]
    uo, vo = oracle.sinkhorn_rowpartition(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, off, 10)
    uc, vc = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 10)
    for ref_u, ref_v in ((uo, vo), (uc, vc)):
        assert np.max(np.abs(u - ref_u) / ref_u) <= 1e-4
        assert np.max(np.abs(v_all[0] - ref_v) / ref_v) <= 1e-4
    # the row residual recorded by the 10th row pass is that of the state after 9 iterations
    u9, v9 = oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, 9)
    e9 = oracle.marginal_errors(w.K, oracle.KIND_KERNEL, w.eps, 0, u9, v9, w.a, w.b)["row_l1"]
    assert l1 == pytest.approx(e9, rel=2e-3, abs=1e-6)


def test_shards_from_cost_blocks_and_bad_arguments():
    import torch
    w = workloads.make(1, n=300)
    u, v_all, _ = run_shards(w, 2, 10, kind=fs.FS_MATRIX_COST)
    uc, vc = oracle.sinkhorn_scaling(w.C, oracle.KIND_COST, w.eps, w.a, w.b, 10)
    assert np.max(np.abs(u - uc) / uc) <= 1e-4 and np.max(np.abs(v_all[0] - vc) / vc) <= 1e-4
    x = torch.ones(16, device="cuda:0")
    for args, code in (((8, 4, 8), fs.FS_ERR_BAD_N), ((8, 0, 0), fs.FS_ERR_BAD_N)):
        n, lo, m = args
        with pytest.raises(fs.FsError) as ei:
            fs.fs_shard_create(n, lo, m, x, n, 0, 0.1, x, x)
        assert ei.value.code == code


def make_shards(w, G, torch, dev, stream):
    b = torch.from_numpy(w.b).to(dev)
    shards, blocks, keep = [], [], []
    for r in range(G):
        lo, hi = fsdist.row_range(w.n, r, G)
        Mb = torch.from_numpy(np.ascontiguousarray(w.K[lo:hi])).to(dev)
        ab = torch.from_numpy(w.a[lo:hi].copy()).to(dev)
        keep += [Mb, ab, b]
        torch.cuda.synchronize()
        shards.append(fs.fs_shard_create(w.n, lo, hi - lo, Mb, w.n, fs.FS_MATRIX_KERNEL, w.eps, ab, b, stream))
        blocks.append((lo, hi))
    return shards, blocks, keep


@pytest.mark.parametrize("n,G", [(1000, 3), (4099, 4)])
def test_shards_run_algorithm_1_with_allgathers_on_a_symmetric_kernel(n, G):
    """Algorithm 1 as printed on G shards of one GPU: u slices are gathered (here: copied into one vector, which
    is what an Allgather leaves on every rank), each shard applies its column block as K_{I,:} u (K symmetric)
    and the v slices are gathered.  Reference: the oracle's c-client protocol, which equals centralized Sinkhorn."""
    import torch
    w = workloads.make(5, n=n, nbatch=1)                 # one cloud: symmetric kernel
    assert np.array_equal(w.K, w.K.T)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(device=dev)
    shards, blocks, keep = make_shards(w, G, torch, dev, stream)
    u_full = torch.empty(n, dtype=torch.float32, device=dev)
    v_full = torch.empty(n, dtype=torch.float32, device=dev)
    try:
        with torch.cuda.stream(stream):
            for _ in range(10):
                for s, (lo, hi) in zip(shards, blocks):
                    fs.fs_shard_row_pass(s, stream)
                    fs.fs_shard_local_u(s, u_full[lo:hi], stream)             # Allgather of u
                for s, (lo, hi) in zip(shards, blocks):
                    fs.fs_shard_col_block_pass(s, u_full, v_full[lo:hi], stream)   # Allgather of v
                for s in shards:
                    fs.fs_shard_set_scalings(s, None, v_full, stream)
        stream.synchronize()
        u, v = u_full.cpu().numpy(), v_full.cpu().numpy()
    finally:
        for s in shards:
            fs.fs_shard_destroy(s)
    off = [lo for lo, _ in blocks] + [n]
    uo, vo, agree = oracle.sinkhorn_protocol(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, off, 10)
    assert agree
    assert np.max(np.abs(u - uo) / uo) <= 1e-4 and np.max(np.abs(v - vo) / vo) <= 1e-4


def test_shards_add_gathered_partials_in_rank_order_reproducibly():
    """Fixed reduction order: the G partial vectors sit side by side (what an all-gather leaves on every rank) and
    fs_shard_col_finish_gathered adds them g = 0..G-1.  Every shard ends with the same v, two runs agree bit for
    bit, and the iterates are the oracle's row-partition iterates."""
    import torch
    n, G = 3000, 3
    w = workloads.make(2, n=n)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(device=dev)
    runs = []
    for _ in range(2):
        shards, blocks, keep = make_shards(w, G, torch, dev, stream)
        parts = torch.empty(G * n, dtype=torch.float32, device=dev)
        try:
            with torch.cuda.stream(stream):
                for _ in range(8):
                    for g, s in enumerate(shards):
                        fs.fs_shard_row_pass(s, stream)
                        fs.fs_shard_col_partial(s, parts[g * n:(g + 1) * n], stream)
                    for s in shards:
                        fs.fs_shard_col_finish_gathered(s, parts, G, n, stream)
            vs = []
            u = np.empty(n, dtype=np.float32)
            for s, (lo, hi) in zip(shards, blocks):
                ub = torch.empty(hi - lo, dtype=torch.float32, device=dev)
                vb = torch.empty(n, dtype=torch.float32, device=dev)
                fs.fs_shard_scalings(s, ub, vb, stream)
                u[lo:hi] = ub.cpu().numpy()
                vs.append(vb.cpu().numpy())
        finally:
            for s in shards:
                fs.fs_shard_destroy(s)
        assert all(np.array_equal(vb, vs[0]) for vb in vs[1:])
        runs.append((u, vs[0]))
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])
    off = [fsdist.row_range(n, r, G)[0] for r in range(G)] + [n]
    uo, vo = oracle.sinkhorn_rowpartition(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, off, 8)
    assert np.max(np.abs(runs[0][0] - uo) / uo) <= 1e-4 and np.max(np.abs(runs[0][1] - vo) / vo) <= 1e-4


@pytest.mark.parametrize("n,G", [(4100, 2), (8192, 4)])
def test_shards_single_read_local_step(n, G):
    """fs_shard_fused_step (row step and column partial from ONE read of the block) against the two separate local
    steps and the oracle's row-partition iterates; unequal blocks, ragged column segments."""
    import torch
    w = workloads.make(2, n=n)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(device=dev)
    res = {}
    for fused in (True, False):
        shards, blocks, keep = make_shards(w, G, torch, dev, stream)
        parts = torch.empty(G * n, dtype=torch.float32, device=dev)
        try:
            with torch.cuda.stream(stream):
                for _ in range(8):
                    for g, s in enumerate(shards):
                        p = parts[g * n:(g + 1) * n]
                        if fused:
                            assert fs.fs_shard_fused_step(s, p, stream)
                        else:
                            fs.fs_shard_row_pass(s, stream)
                            fs.fs_shard_col_partial(s, p, stream)
                    for s in shards:
                        fs.fs_shard_col_finish_gathered(s, parts, G, n, stream)
            u = np.empty(n, dtype=np.float32)
            for s, (lo, hi) in zip(shards, blocks):
                ub = torch.empty(hi - lo, dtype=torch.float32, device=dev)
                vb = torch.empty(n, dtype=torch.float32, device=dev)
                fs.fs_shard_scalings(s, ub, vb, stream)
                u[lo:hi] = ub.cpu().numpy()
            res[fused] = (u, vb.cpu().numpy())
        finally:
            for s in shards:
                fs.fs_shard_destroy(s)
    off = [fsdist.row_range(n, r, G)[0] for r in range(G)] + [n]
    uo, vo = oracle.sinkhorn_rowpartition(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, off, 8)
    for fused in (True, False):
        assert np.max(np.abs(res[fused][0] - uo) / uo) <= 1e-4 and np.max(np.abs(res[fused][1] - vo) / vo) <= 1e-4
    assert np.max(np.abs(res[True][0] - res[False][0]) / res[False][0]) < 1e-5
