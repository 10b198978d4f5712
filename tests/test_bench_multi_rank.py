"""bench.py at N > 1 runs independent replicas (the path shards by replication only): every rank
times its own copy, the slowest rank's time is taken, the whole-job value is all ranks' bytes over
that time.  Checked here with two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, os.environ["VQ_ROOT"])
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist)      # rank 1 is the slow replica
    assert ms == 15.0, ms
    v = bench.whole_job_gbs(3_000_000, world, ms)
    assert abs(v - world * 3_000_000 / 15e-3 / 1e9) < 1e-12, v
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


def test_two_rank_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, VQ_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                        "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)],
                       env=env, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.count("ok") == 2


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5) == 7.5
    assert bench.whole_job_gbs(1_000_000_000, 1, 1000.0) == 1.0
