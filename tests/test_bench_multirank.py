"""Host-side logic of the N > 1 benchmark path: ranks are independent replicas; the reported time
is the max over ranks.  Runs two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    mine = 10.0 + 5.0 * rank                       # rank 1 is slower
    agg = bench.aggregate_over_ranks(mine, world)
    assert agg == 15.0, agg
    assert bench.aggregate_over_ranks(3.0, 1) == 3.0
    dist.barrier()
    dist.destroy_process_group()
    print("rank" + str(rank) + "-ok")              # one token per rank: the two ranks share a pipe
""") % ROOT


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    with socket.socket() as sock:                       # a port nobody is using right now
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    res = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
         "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
        capture_output=True, text=True, timeout=240, env=env)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "rank0-ok" in res.stdout and "rank1-ok" in res.stdout


def test_reference_arm_exits_quietly_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_pass_dims_and_flops():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.pass_dims(0, 8192, 4096, 6144) == (8192, 6144, 4096)
    assert bench.pass_dims(1, 8192, 4096, 6144) == (8192, 4096, 6144)
    assert bench.pass_dims(2, 8192, 4096, 6144) == (6144, 4096, 8192)
