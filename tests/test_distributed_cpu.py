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
