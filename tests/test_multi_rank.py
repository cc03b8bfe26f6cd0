"""The N > 1 path of the benchmark is independent replicas: no data-path collective, only a barrier and a
max-over-ranks of the time.  Covered here with two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["DAB_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
dist.barrier()
slowest = bench.max_over_ranks(10.0 * (rank + 1), world)       # rank r took 10*(r+1) seconds
value = bench.aggregate_throughput(100.0, 4, slowest, world)    # 100 units per rank and step, 4 steps
if rank == 0:
    print("RESULT", slowest, value)
dist.destroy_process_group()
"""


def test_replicas_report_the_slowest_rank_and_the_sum_of_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, DAB_ROOT=ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("RESULT")]
    assert len(line) == 1
    _, slowest, value = line[0].split()
    assert float(slowest) == 20.0                      # max over ranks
    assert float(value) == 2 * 100.0 * 4 / 20.0        # whole-job units / slowest rank's time


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    code = ("import sys; sys.argv=['bench.py','--impl','reference','--steps','0','--warmup','0']; "
            "import runpy; runpy.run_path(%r, run_name='__main__')" % os.path.join(ROOT, "bench.py"))
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""        # ranks other than 0 exit without work
