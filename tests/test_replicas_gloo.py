"""The multi-replica bookkeeping of the benchmark (bench.py --gpus N runs N independent replicas, the path
has no collective): barrier, maximum over the ranks and the whole-job throughput, on two CPU processes over gloo."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
bench.rank_barrier(2)
slowest = bench.rank_max(1.5 + rank, 2)          # rank 0 measured 1.5 ms, rank 1 2.5 ms
assert slowest == 2.5, slowest
total = bench.replica_throughput(1000, 2, slowest)
assert abs(total - 2 * 1000 / 2.5e-3) < 1e-6, total
assert bench.rank_max(7.0, 1) == 7.0             # one replica: no communication
bench.rank_barrier(2)
dist.destroy_process_group()
print("ok", rank)
"""


def test_two_replicas_report_the_slowest_time_and_the_summed_throughput(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
             for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"ok {r}" in out
