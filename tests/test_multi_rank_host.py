"""Host-side logic of the multi-GPU benchmark path, on CPU with the gloo backend.

Decode attention and encode shard over sequences with no exchange on the data path, so a
multi-GPU run is N independent replicas of the batch; what the ranks share is only the timing
protocol of bench.py (rendezvous, barrier, maximum over ranks, rank 0 prints).  Two CPU
processes exercise exactly that code."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["CQ_ROOT"])
import torch
import bench
rank, world, local = bench.dist_setup(2)
assert world == 2 and rank in (0, 1)
bench.barrier(world)
m = bench.max_over_ranks(10.0 + rank, world, torch.device("cpu"))
assert m == 11.0, m
# whole-job value = units of all ranks / slowest rank's time
tokens = 1000 * world
value = tokens / (m * 1e-3)
bench.barrier(world)
if rank == 0:
    print("RESULT", value)
import torch.distributed as dist
dist.destroy_process_group()
"""


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_rank_timing_protocol_over_gloo():
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CQ_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    assert "RESULT" in outs[0][0] and "RESULT" not in outs[1][0]
    assert abs(float(outs[0][0].split("RESULT")[1]) - 2000 / 11e-3) < 1e-6


def test_reference_arm_prints_on_rank0_only():
    # the oracle-timed arm: rank 0 prints one JSON line, every other rank exits 0 without work
    base = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()),
                CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "1", "--workload", "cfg0"]
    r1 = subprocess.run(cmd, env=dict(base, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(base, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr[-2000:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
