"""The N>1 launch path of the benchmark (independent replicas): gloo, world size 2, CPU only."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent("""
    import sys, torch
    sys.path.insert(0, %r)
    from paper_2607_16184_b200 import replicas
    rank, local_rank, world = replicas.init("gloo")
    dev = torch.device("cpu")
    replicas.barrier(dev)
    t, u = replicas.aggregate(10.0 + 5.0 * rank, 64.0, dev)
    assert world == 2 and t == 15.0 and u == 128.0, (world, t, u)
    replicas.barrier(dev)
    replicas.shutdown()
    sys.stdout.write("rank" + str(rank) + "_ok" + chr(10))
    sys.stdout.flush()
""") % ROOT


def test_two_replicas_aggregate_max_time_and_summed_units(tmp_path):
    script = tmp_path / "w.py"
    script.write_text(SCRIPT)
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("_ok") == 2 and "rank0" in out.stdout and "rank1" in out.stdout


def test_single_process_is_identity():
    import torch
    from paper_2607_16184_b200 import replicas
    assert replicas.env_world()[2] >= 1
    assert replicas.aggregate(3.0, 7.0, torch.device("cpu")) == (3.0, 7.0)
