"""The multi-GPU plumbing of the benchmark is replicas only: a barrier around the timed region, MAX of the
per-rank time, SUM of the per-rank units.  Checked here on two gloo ranks on the CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2504_12285_b200 import replicas
    rank, local_rank, world = replicas.init(backend="gloo")
    assert world == 2 and rank in (0, 1)
    replicas.barrier()
    # rank 0 "took" 2 s for 10 units, rank 1 3 s for 30 units: whole job = 40 units / 3 s
    value, slowest = replicas.aggregate_throughput(10.0 if rank == 0 else 30.0, 2.0 if rank == 0 else 3.0)
    assert abs(slowest - 3.0) < 1e-12 and abs(value - 40.0 / 3.0) < 1e-12, (value, slowest)
    assert replicas.max_over_ranks(float(rank)) == 1.0
    assert replicas.sum_over_ranks(1.5) == 3.0
    replicas.barrier()
    replicas.finalize()
    print("ok", rank)
""") % ROOT


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = []
    for rank in range(2):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=e, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True))
    for rank, p in enumerate(procs):
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        assert f"ok {rank}" in out


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2504_12285_b200 import replicas

    assert replicas.max_over_ranks(2.5) == 2.5
    assert replicas.aggregate_throughput(8.0, 2.0) == (4.0, 2.0)
    replicas.barrier()
