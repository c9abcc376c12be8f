"""Host logic of bench.py's N > 1 path on two gloo ranks (CPU): the slowest rank's time is what
every rank reports, the value is the whole job's samples over that time, and the reference arm
prints on rank 0 only."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, '@ROOT@')
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    value = bench.whole_job_value(dist.get_world_size(), 1000, 4, ms)
    open(os.path.join(os.environ["RESULT_DIR"], "rank%d.txt" % rank), "w").write("%d %r %r" % (rank, ms, value))
    dist.destroy_process_group()
""").replace("@ROOT@", ROOT)


def test_two_gloo_ranks_report_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", RESULT_DIR=str(tmp_path))
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29611", str(script)],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [(tmp_path / ("rank%d.txt" % r)).read_text().split() for r in (0, 1)]
    for r in rows:
        assert float(r[1]) == 15.0
        assert abs(float(r[2]) - 2 * 1000 * 4 / 0.015) < 1e-6


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5) == 7.5
    assert bench.whole_job_value(1, 65536, 5, 500.0) == 65536 * 5 / 0.5


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
