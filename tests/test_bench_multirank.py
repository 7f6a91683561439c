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
    assert abs(jm["key_switches_per_s"] - 2 * 64 / 0.005) < 1e-6        # 64 plain rotations per replica in 5 ms


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    jm = bench.job_metrics(1, 1.0, 25.0, 450.0)
    assert jm["value"] == 0.45 and jm["key_switches_per_s"] == 64 / 0.025


def test_algorithmic_work_counts():
    """The operation counts behind the roofline fractions: one key switch at level 24 with 8 special primes and 3 digits
    is 160 limb transforms and 81.3 M multiply-add pairs, a hoisted rotation 64 and 42 M (counted by hand from the steps:
    24 inverse + 72 forward transforms and 600 pairs per coefficient for ModUp, 192 for the key product, 16 + 48
    transforms and 448 pairs for ModDown)."""
    sys.path.insert(0, ROOT)
    import bench
    ks, h = bench.ks_work(), bench.ks_work(hoisted=True)
    assert ks["limb_ntts"] == 24 + 72 + 16 + 48 == 160 and h["limb_ntts"] == 64
    assert ks["pairs_per_coeff"] == 600 + 192 + 448 and h["pairs_per_coeff"] == 192 + 448
    assert round(ks["pairs_per_coeff"] * 65536 / 1e6, 1) == 81.3 and round(h["pairs_per_coeff"] * 65536 / 1e6, 1) == 41.9
    assert ks["fp64_instr"] == 160 * 524288 * 8 + 1240 * 65536 * 7
    lazy, eager = bench.projection_work(True), bench.projection_work(False)
    assert lazy["encode"]["count"] == 4096 and lazy["mac"]["count"] == 65536
    assert lazy["baby_hoisted_rotations"]["count"] == 1008 and lazy["giant_terms"]["count"] == 1008 and eager["giant_rotations"]["count"] == 1008
    assert lazy["mac"]["hbm_bytes"] == (4096 * 24 + 16 * 64 * 48 + 16 * 64 * 48) * 524288      # plaintexts, baby ciphertexts, accumulators
    assert bench.bound_ms(eager, 18.6, 6527.0) > bench.bound_ms(lazy, 18.6, 6527.0) > 100.0
