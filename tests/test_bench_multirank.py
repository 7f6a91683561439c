"""The benchmark's N > 1 path on CPU: two gloo ranks, max-over-ranks timing, whole-job aggregation (replicas only,
no data-path collective), and the reference arm's rule that rank 0 alone prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
mine = [100.0 + 10 * rank, 5.0 - rank, 7.0, 400.0 + rank]
got = bench.max_over_ranks(mine)
dist.barrier()
if rank == 0:
    jm = bench.job_metrics(dist.get_world_size(), got[0], got[1], got[3])
    print(json.dumps({"max": got, "jm": jm}))
dist.destroy_process_group()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_ranks_aggregate():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % ROOT], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert outs[1][0].strip() == ""                                   # only rank 0 prints
    assert line["max"] == [110.0, 5.0, 7.0, 401.0]                    # element-wise max over the two ranks
    jm = line["jm"]
    assert abs(jm["value"] - 0.401 / 2) < 1e-12                       # two replicas finish two projections in 401 ms
    assert abs(jm["ntt_limbs_per_s"] - 2 * 2 * 768 / 0.110) < 1e-6
    assert abs(jm["key_switches_per_s"] - 2 * 129 / 0.005) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    jm = bench.job_metrics(1, 1.0, 25.0, 450.0)
    assert jm["value"] == 0.45 and jm["key_switches_per_s"] == 129 / 0.025
