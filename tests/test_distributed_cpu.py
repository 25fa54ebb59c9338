"""N-process plumbing on CPU: two gloo ranks exercise what bench.py does around its timed region
(barrier, max over ranks of the elapsed time, sum of the units of work) and the problem sharding."""
import os
import socket
import subprocess
import sys
import textwrap

from paper_2502_07021_b200 import distributed as fsdist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_shard_problems_partitions_exactly():
    for total in (0, 1, 7, 128, 129):
        for world in (1, 2, 3, 8):
            parts = [fsdist.shard_problems(total, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == total
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_is_identity():
    assert fsdist.aggregate(12.5, 300) == (12.5, 300.0)
    assert fsdist.env_world() == (0, 0, 1) or "WORLD_SIZE" in os.environ


def test_two_gloo_ranks_aggregate_max_time_and_sum_units(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(textwrap.dedent(f"""
        import sys
        sys.path.insert(0, {ROOT!r})
        from paper_2502_07021_b200 import distributed as fsdist
        rank, local_rank, world = fsdist.init(backend="gloo")
        fsdist.barrier()
        t, u = fsdist.aggregate(10.0 + 5.0 * rank, 300 * (rank + 1), "cpu")
        lo, hi = fsdist.shard_problems(128, rank, world)
        fsdist.barrier()
        print(f"RESULT {{rank}} {{world}} {{t}} {{u}} {{lo}} {{hi}}", flush=True)
        fsdist.finalize()
    """))
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    got = {}
    for out in outs:
        for line in out.splitlines():
            if line.startswith("RESULT"):
                _, rank, world, t, u, lo, hi = line.split()
                got[int(rank)] = (int(world), float(t), float(u), int(lo), int(hi))
    assert got[0] == (2, 15.0, 900.0, 0, 64)
    assert got[1] == (2, 15.0, 900.0, 64, 128)


def test_reference_arm_runs_only_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_two_gloo_ranks_run_the_sharded_iteration(tmp_path):
    """`sharded_iterate` with two gloo ranks: each rank owns a row block and a stand-in for the shard API
    written with numpy (row pass, column partial, finish); the all-reduce is torch.distributed's.  The
    stacked result must be the row-partition iterates of the oracle."""
    script = tmp_path / "shard_rank.py"
    script.write_text(textwrap.dedent(f"""
        import sys
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch
        import oracle
        from paper_2502_07021_b200 import distributed as fsdist, workloads

        class NumpyShardApi:
            # host stand-in with the call pattern of the C ABI's fs_shard_* steps
            def fs_shard_row_pass(self, s, stream=None):
                s["u"] = s["a"] / (s["K"] @ s["v"])
            def fs_shard_col_partial(self, s, r_buf, stream=None):
                r_buf.copy_(torch.from_numpy((s["K"].T @ s["u"]).astype(np.float32)))
            def fs_shard_col_finish(self, s, r_buf, stream=None):
                s["v"] = s["b"] / r_buf.numpy().astype(np.float64)

        rank, local_rank, world = fsdist.init(backend="gloo")
        w = workloads.make(2, n=96)
        lo, hi = fsdist.row_range(w.n, rank, world)
        shard = dict(K=w.K[lo:hi].astype(np.float64), a=w.a[lo:hi].astype(np.float64), b=w.b.astype(np.float64),
                     u=np.ones(hi - lo), v=np.ones(w.n))
        r_buf = torch.empty(w.n, dtype=torch.float32)
        fsdist.sharded_iterate(NumpyShardApi(), shard, r_buf, 6)
        uo, vo = oracle.sinkhorn_rowpartition(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, [0, 48, 96], 6)
        ok = np.max(np.abs(shard["u"] - uo[lo:hi]) / uo[lo:hi]) < 1e-5 and np.max(np.abs(shard["v"] - vo) / vo) < 1e-5
        print(f"RESULT {{rank}} {{lo}} {{hi}} {{int(ok)}}", flush=True)
        fsdist.finalize()
    """))
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    results = sorted(line.split()[1:] for out in outs for line in out.splitlines() if line.startswith("RESULT"))
    assert results == [["0", "0", "48", "1"], ["1", "48", "96", "1"]]


def _run_two_ranks(script, timeout=180):
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=timeout)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    return sorted(line.split()[1:] for out in outs for line in out.splitlines() if line.startswith("RESULT"))


SHARD_STANDIN = """
class NumpyShardApi:
    # host stand-in with the call pattern of the C ABI's fs_shard_* steps (fp64 numpy)
    def fs_shard_row_pass(self, s, stream=None):
        s["u"] = s["a"] / (s["K"] @ s["v"])
    def fs_shard_local_u(self, s, out, stream=None):
        out.copy_(torch.from_numpy(s["u"]))
    def fs_shard_col_partial(self, s, r_buf, stream=None):
        r_buf.copy_(torch.from_numpy(s["K"].T @ s["u"]))
    def fs_shard_col_finish(self, s, r_buf, stream=None):
        s["v"] = s["b"] / r_buf.numpy()
    def fs_shard_col_finish_gathered(self, s, parts, nparts, pitch, stream=None):
        r = np.zeros(pitch)
        for g in range(nparts):                       # rank order
            r = r + parts.numpy()[g * pitch:(g + 1) * pitch]
        s["v"] = s["b"] / r
    def fs_shard_col_block_pass(self, s, u_full, v_block_out, stream=None):
        lo, hi = s["lo"], s["hi"]
        v_block_out.copy_(torch.from_numpy(s["b"][lo:hi] / (s["K"] @ u_full.numpy())))   # K symmetric: (K[:,I])^T u = K[I,:] u
    def fs_shard_set_scalings(self, s, u, v, stream=None):
        if v is not None:
            s["v"] = v.numpy().copy()
"""


def test_two_gloo_ranks_run_algorithm_1_with_two_allgathers(tmp_path):
    """The Allgather form of Algorithm 1 (symmetric K, one cloud): row step, Allgather of u slices, column-block
    step on the gathered u, Allgather of v slices -- with UNEQUAL blocks.  By Proposition 1 the stacked iterates
    are those of centralized Sinkhorn; the oracle's c-client protocol is the reference."""
    script = tmp_path / "alg1_rank.py"
    script.write_text(textwrap.dedent(f"""
        import sys
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch
        import oracle
        from paper_2502_07021_b200 import distributed as fsdist, workloads
    """) + SHARD_STANDIN + textwrap.dedent("""
        rank, local_rank, world = fsdist.init(backend="gloo")
        w = workloads.make(5, n=97, nbatch=1)            # one cloud: symmetric kernel; 97 rows: blocks of 49 and 48
        assert np.array_equal(w.K, w.K.T)
        lo, hi = fsdist.row_range(w.n, rank, world)
        sizes = [fsdist.row_range(w.n, r, world)[1] - fsdist.row_range(w.n, r, world)[0] for r in range(world)]
        shard = dict(K=w.K[lo:hi].astype(np.float64), a=w.a[lo:hi].astype(np.float64), b=w.b.astype(np.float64),
                     u=np.ones(hi - lo), v=np.ones(w.n), lo=lo, hi=hi)
        v_full = torch.ones(w.n, dtype=torch.float64)
        t = fsdist.sharded_iterate(NumpyShardApi(), shard, v_full, 6, exchange="alg1", sizes=sizes, timed=True)
        uo, vo, agree = oracle.sinkhorn_protocol(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, [0, sizes[0], w.n], 6)
        ok = agree and np.max(np.abs(shard["u"] / uo[lo:hi] - 1)) < 1e-12 and np.max(np.abs(shard["v"] / vo - 1)) < 1e-12
        ok = ok and t["local_ms"] > 0 and t["exchange_ms"] > 0
        print(f"RESULT {rank} {lo} {hi} {int(ok)}", flush=True)
        fsdist.finalize()
    """))
    assert _run_two_ranks(script) == [["0", "0", "49", "1"], ["1", "49", "97", "1"]]


def test_two_gloo_ranks_add_gathered_partials_in_rank_order(tmp_path):
    """The fixed-order form: partial column sums are all-gathered and every rank adds them itself, rank 0 first.
    Both ranks must hold bit-identical v (their sums use the same operands in the same order), equal to the
    oracle's row-partition iterates."""
    script = tmp_path / "ordered_rank.py"
    script.write_text(textwrap.dedent(f"""
        import sys, hashlib
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch
        import oracle
        from paper_2502_07021_b200 import distributed as fsdist, workloads
    """) + SHARD_STANDIN + textwrap.dedent("""
        rank, local_rank, world = fsdist.init(backend="gloo")
        w = workloads.make(2, n=96)
        lo, hi = fsdist.row_range(w.n, rank, world)
        shard = dict(K=w.K[lo:hi].astype(np.float64), a=w.a[lo:hi].astype(np.float64), b=w.b.astype(np.float64),
                     u=np.ones(hi - lo), v=np.ones(w.n), lo=lo, hi=hi)
        r_buf = torch.empty(w.n, dtype=torch.float64)
        fsdist.sharded_iterate(NumpyShardApi(), shard, r_buf, 6, exchange="ordered")
        uo, vo = oracle.sinkhorn_rowpartition(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, [0, 48, 96], 6)
        ok = np.max(np.abs(shard["u"] / uo[lo:hi] - 1)) < 1e-12 and np.max(np.abs(shard["v"] / vo - 1)) < 1e-12
        digest = hashlib.sha1(shard["v"].tobytes()).hexdigest()[:12]
        print(f"RESULT {rank} {int(ok)} {digest}", flush=True)
        fsdist.finalize()
    """))
    res = _run_two_ranks(script)
    assert [r[:2] for r in res] == [["0", "1"], ["1", "1"]]
    assert res[0][2] == res[1][2]
