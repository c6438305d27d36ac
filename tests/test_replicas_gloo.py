"""The multi-GPU story is "independent replicas": check the process-group plumbing the benchmark uses
(barrier, max and sum over ranks) with two gloo ranks on the CPU."""

import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["SAGEKV_ROOT"])
from paper_2503_08879_b200 import replicas
rank, world = replicas.init("gloo")
assert world == 2 and rank == int(os.environ["RANK"])
replicas.barrier()
t = 10.0 + 5.0 * rank                      # rank 1 is the slow one
assert replicas.max_over_ranks(t) == 15.0
assert replicas.sum_over_ranks(t) == 25.0
replicas.barrier()
replicas.shutdown()
print("rank", rank, "ok")
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_max_and_sum():
    port = str(free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=port, SAGEKV_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_needs_no_group():
    from paper_2503_08879_b200 import replicas
    env = {k: os.environ.pop(k, None) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    try:
        assert replicas.env_world() == (0, 0, 1)
        assert replicas.init("gloo") == (0, 1)
        replicas.barrier()
        assert replicas.max_over_ranks(3.5) == 3.5 and replicas.sum_over_ranks(3.5) == 3.5
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v
