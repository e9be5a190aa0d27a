"""bench.py --gpus N runs N independent replicas (one stream per GPU, no collective on the data path).  What
the ranks share is the timing protocol: the slowest rank's time (all-reduce MAX) and the aggregate frames/s
computed from it.  Here: two gloo ranks on CPU with different local times."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["NFD_ROOT"])
import torch
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
ms_local = [40.0, 55.0][rank]                  # rank 1 is the slow one
dist.barrier()
ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
value = bench.aggregate_frames_per_s(dist.get_world_size(), 8, ms)
dist.barrier()
print(json.dumps({"rank": rank, "ms": ms, "value": value}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_agree_on_the_slowest_rank_and_the_aggregate():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), NFD_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    assert {o["rank"] for o in outs} == {0, 1}
    for o in outs:
        assert o["ms"] == 55.0                                   # the slowest rank, on every rank
        assert abs(o["value"] - 2 * 8 / 0.055) < 1e-9            # 2 replicas x 8 frames in 55 ms


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(12.5, None, None) == 12.5
    assert abs(bench.aggregate_frames_per_s(1, 64, 8000.0) - 8.0) < 1e-12
