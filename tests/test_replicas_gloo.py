"""The multi-GPU shape of the benchmark on CPU: independent replicas, one process per rank, no data-path
collective; the only exchange is the max over ranks of the step time (gloo, world size 2)."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank, local, world = bench.dist_env()
dist.init_process_group("gloo")
mine = 2.0 + 3.0 * rank                     # rank 1 is the slow replica
worst = bench.max_over_ranks(mine, world)
assert world == 2 and worst == 5.0, (rank, worst)
# whole-job throughput of weak-scaled replicas: every rank's units over the slowest rank's time
units_per_rank = 32
value = world * units_per_rank / (worst * 1e-3)
assert abs(value - 12800.0) < 1e-6
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_replica_timing_is_max_over_ranks(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out
