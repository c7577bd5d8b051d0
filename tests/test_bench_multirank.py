"""The N > 1 path of bench.py (replicas, no data-path collective): the per-rank times are
reduced with a maximum over ranks and the value counts every replica.  Run here as two gloo
ranks on the CPU."""
import os
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
got = bench.max_over_ranks([10.0 + rank, 5.0 - rank])
assert got == [11.0, 5.0], got
assert bench.whole_job_value(1000, dist.get_world_size(), got[0]) == 2 * 1000 / 11e-3
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), REPO_ROOT=str(ROOT))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_is_the_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.whole_job_value(10, 1, 2.0) == 10 / 2e-3
