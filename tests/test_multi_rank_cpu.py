"""The N > 1 path of the benchmark is replicas only (the method does not shard); what the ranks share is the
timing reduction.  Two gloo ranks on CPU check it: whole-job rate = all ranks' units over the slowest rank."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
rate, ms, world = bench.whole_job_rate(640, 1000.0 if rank == 0 else 2500.0, dist)
dist.barrier()
print(json.dumps(dict(rank=rank, rate=rate, ms=ms, world=world)))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_report_the_slowest_ranks_time():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    code = CHILD.format(root=ROOT, port=port)
    procs = [subprocess.Popen([sys.executable, "-c", code, str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e[-2000:]
        outs.append(__import__("json").loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["world"] == 2 and o["ms"] == 2500.0
        assert abs(o["rate"] - 2 * 640 / 2.5) < 1e-9


def test_single_process_rate_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job_rate(640, 2000.0) == (320.0, 2000.0, 1)
