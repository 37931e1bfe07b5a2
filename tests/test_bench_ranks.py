"""Host logic of bench.py for more than one rank (replicas only: no data-path collective),
exercised with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
local_ms = 100.0 + 25.0 * rank                      # rank 1 is the slow replica
ms = bench.max_over_ranks(local_ms, world, device="cpu")
assert ms == 125.0, ms
value = bench.whole_job_value(1000, world, ms)
assert abs(value - 2 * 1000 / 0.125) < 1e-9, value
dist.barrier()
dist.destroy_process_group()
print("rank %%d ok" %% rank)
""" % ROOT


def test_two_gloo_ranks_take_the_slowest_replicas_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29517", str(script)],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "rank 0 ok" in out.stdout and "rank 1 ok" in out.stdout


def test_reference_arm_prints_from_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_launch_count_formula_matches_the_round_structure():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2302_13053_b200 import workloads as wl
    w = wl.make_config(1, scale=0.2)
    a, b = bench.launches_per_step(w, 10), bench.launches_per_step(w, 20)
    per_iter = (b - a) / 10
    assert per_iter == (5 + 5 + 3)          # two rounds with a hidden layer, one without; validation rides along
                                            # and is booked by the update kernel's last block
