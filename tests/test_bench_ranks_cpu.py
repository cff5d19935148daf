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
