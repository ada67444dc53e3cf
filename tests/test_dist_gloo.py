"""World-size-2 check of the multi-process plumbing on CPU (gloo): rendezvous
from the environment, barrier, and the max-over-ranks reduction the benchmark
uses for whole-job rates of independent replicas."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, os.environ["GCNSA_ROOT"])
from paper_2012_04930_b200 import dist as gdist
rank, world, local = gdist.init_from_env("gloo")
assert world == 2 and rank in (0, 1)
gdist.barrier()
slowest = gdist.max_over_ranks(10.0 + 5.0 * rank)       # rank 1 is the slow replica
assert slowest == 15.0, slowest
steps = 3
value = world * steps / slowest                          # whole-job rate of the replicas
print(f"rank {rank} value {value:.6f}", flush=True)
gdist.finish()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_on_gloo():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), GCNSA_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} value 0.400000" in out, out
