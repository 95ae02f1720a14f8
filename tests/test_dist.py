"""The multi-GPU leg runs independent replicas; ranks only meet for a barrier and to combine timings.
This covers that host logic with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_1901_08924_b200 import dist_util
    size, rank = dist_util.init("gloo")
    assert size == 2
    dist_util.barrier()
    # rank 0 processes 1000 units in 10 ms, rank 1 processes 3000 units in 20 ms
    units, ms = (1000, 10.0) if rank == 0 else (3000, 20.0)
    value, slowest = dist_util.whole_job_throughput(units, ms)
    assert slowest == 20.0, slowest
    assert abs(value - 4000 / 0.020) < 1e-6, value
    assert dist_util.max_over_ranks(rank) == 1.0 and dist_util.sum_over_ranks(rank + 1) == 3.0
    dist_util.barrier()
    dist_util.shutdown()
    print("rank", rank, "ok")
""") % ROOT


def _free_port():
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_rank_timing_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    env = dict(os.environ, OMP_NUM_THREADS="1")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, env=env)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert r.stdout.count("ok") == 2


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_1901_08924_b200 import dist_util
    value, ms = dist_util.whole_job_throughput(500, 5.0)
    assert ms == 5.0 and abs(value - 100000.0) < 1e-9
