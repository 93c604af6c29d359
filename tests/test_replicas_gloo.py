"""The N > 1 path of the benchmark on CPU: two gloo ranks go through the barrier and the max-over-ranks step
that `bench.py --gpus N` uses (every rank is an independent replica; there is no data-path collective)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_PROGRAM = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import bench
    rank, world, _ = bench.dist_env()
    reps = bench.Replicas(world, "gloo")
    reps.barrier()
    slowest = reps.max_ms(10.0 + 5.0 * rank)          # rank 1 is the slower replica
    value = reps.job_value(1000.0, slowest)            # 1000 units per rank per step
    reps.barrier()
    print(f"rank={{rank}} slowest={{slowest}} value={{value}}")
    reps.close()
""")


def test_two_gloo_ranks_agree_on_the_slowest_replica(tmp_path):
    prog = tmp_path / "rank_program.py"
    prog.write_text(RANK_PROGRAM.format(root=ROOT))
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(prog)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    for rank, (out, _) in enumerate(outs):
        line = [l for l in out.splitlines() if l.startswith("rank=")][-1]
        # both ranks see the slowest replica's 15 ms, and the job value counts both ranks' units
        assert line == f"rank={rank} slowest=15.0 value={2 * 1000.0 / 15e-3}"


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    reps = bench.Replicas(1)
    reps.barrier()
    assert reps.max_ms(3.5) == 3.5
    assert reps.job_value(10.0, 2.0) == 10.0 / 2e-3
    reps.close()
