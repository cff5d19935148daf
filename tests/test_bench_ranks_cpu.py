"""The multi-rank arithmetic of bench.py on CPU: two gloo ranks (the path itself has no exchange step - ranks are
independent replicas - so all that crosses ranks is the max of the timed region)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    dist.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    assert ms == 15.0, ms
    assert bench.whole_job_us_per_token(ms, 100, world) == 75.0    # 200 tokens in 15 ms
    assert bench.max_over_ranks(3.0, 1) == 3.0
    dist.barrier()
    dist.destroy_process_group()
    sys.stdout.write("rank" + str(rank) + "-ok" + chr(10)); sys.stdout.flush()
""") % ROOT


def test_two_gloo_ranks_take_the_max_and_count_all_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                        "--master-addr", "127.0.0.1", "--master-port", "29517", str(script)],
                       capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "rank0-ok" in r.stdout and "rank1-ok" in r.stdout


def test_region_repeats_and_operating_point_overrides():
    """Host logic of bench.py: how many timed regions are taken, and the switches that select the paper's
    operating points (K, stride / QC, threshold, schedule)."""
    import argparse
    sys.path.insert(0, ROOT)
    import bench
    assert bench.region_repeats(800.0) == 1                 # a long region is taken once
    assert bench.region_repeats(100.0) == 5                 # short ones at least five times
    assert bench.region_repeats(4.9) == 50                  # and at most fifty
    base = dict(workload="cfg2", ctx=0, layers=0, k_small=0, stride=0, qc=0, threshold=-1.0, schedule="")
    w = bench.make_workload(argparse.Namespace(**base))
    assert (w.lens, w.k_small, w.stride, w.schedule) == ([32768], [2048], 10, "fixed")
    w = bench.make_workload(argparse.Namespace(**dict(base, k_small=4096, stride=15)))
    assert (w.k_small, w.stride, w.schedule) == ([4096], 15, "fixed") and "K4096" in w.name
    w = bench.make_workload(argparse.Namespace(**dict(base, schedule="dynamic", qc=5, threshold=0.85)))
    assert (w.schedule, w.stride, w.threshold) == ("dynamic", 5, 0.85)
    w = bench.make_workload(argparse.Namespace(**dict(base, workload="lm16k_S15")))
    assert (w.lens, w.k_small, w.stride, w.steps) == ([16384], [2048], 15, 256)       # K = L / 8, 256 generated tokens
    w = bench.make_workload(argparse.Namespace(**dict(base, workload="novel128k_S10")))
    assert (w.lens, w.k_small) == ([131072], [4096])
    w = bench.make_workload(argparse.Namespace(**dict(base, workload="qwen16k_dyn095_qc5")))
    assert (w.n_q_heads, w.n_kv_heads, w.schedule, w.threshold, w.stride) == (28, 4, "dynamic", 0.95, 5)
