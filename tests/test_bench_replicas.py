"""The N > 1 path of the benchmark is "independent replicas": no data-path collective, only the max-over-ranks of
the device time and the whole-job throughput built from it.  Exercised here with two gloo ranks on the CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_RANK_PROGRAM = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    local_ms = 100.0 + 50.0 * rank                 # rank 1 is the slow replica
    ms, value = bench.whole_job_throughput(local_ms, steps=10, units_per_step=4, world=world)
    assert ms == 150.0, ms
    assert abs(value - world * 10 * 4 / 0.150) < 1e-6, value
    assert bench.max_over_ranks(7.0 - rank, world) == 7.0
    dist.barrier()
    dist.destroy_process_group()
    sys.stdout.write("rank %d ok\\n" % rank)   # one write per rank: the two ranks share the pipe
    sys.stdout.flush()
""")


def test_two_gloo_ranks_report_the_slowest_time_and_the_sum_of_work(tmp_path):
    prog = tmp_path / "rank_program.py"
    prog.write_text(_RANK_PROGRAM.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29641", str(prog)]
    env = dict(os.environ, OMP_NUM_THREADS="1")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "rank 0 ok" in r.stdout and "rank 1 ok" in r.stdout


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms, value = bench.whole_job_throughput(2.0, steps=128, units_per_step=1, world=1)
    assert ms == 2.0 and abs(value - 64000.0) < 1e-9
