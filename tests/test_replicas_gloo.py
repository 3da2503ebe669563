"""The multi-GPU mode of the benchmark is "replicas only": every rank runs the same workload on its own GPU
and only the timing is reduced (max over ranks).  This covers that reduction with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, os.environ["PRQ_ROOT"])
    import torch.distributed as dist
    from paper_2609_22106_b200.replicas import job_time_and_throughput
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    # rank 0 needs 2 s for 10 units, rank 1 needs 4 s for 10 units: the job takes 4 s for 20 units
    t, thr = job_time_and_throughput(2.0 if rank == 0 else 4.0, 10.0, dist)
    assert t == 4.0 and thr == 5.0, (t, thr)
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


def test_two_ranks_take_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, PRQ_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), str(script)]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    assert out.stdout.count("ok") == 2


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    from paper_2609_22106_b200.replicas import job_time_and_throughput

    assert job_time_and_throughput(2.0, 10.0) == (2.0, 5.0)
