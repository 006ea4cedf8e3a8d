"""World-size-2 check of the rank plumbing the benchmark uses (gloo, CPU): max-over-ranks timing, summed
token counts, request sharding."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import sys
sys.path.insert(0, {root!r})
from paper_2609_34388_b200.dist import DistEnv, shard_requests
env = DistEnv.from_env(backend="gloo")
env.barrier()
ms = env.max_float(10.0 + 5.0 * env.rank)          # slowest rank decides
tok = env.sum_float(100.0 * (env.rank + 1))        # whole-job token count
mine = shard_requests(5, env.rank, env.world)
print("RESULT", env.rank, env.world, ms, tok, mine, flush=True)
env.close()
"""


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_ranks_reduce_and_shard():
    port = free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=ROOT)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    lines = sorted(l for o, _ in outs for l in o.splitlines() if l.startswith("RESULT"))
    assert lines[0] == "RESULT 0 2 15.0 300.0 [0, 1, 2]"
    assert lines[1] == "RESULT 1 2 15.0 300.0 [3, 4]"


def test_single_process_needs_no_group():
    from paper_2609_34388_b200.dist import DistEnv, shard_requests

    env = DistEnv()
    env.barrier()
    assert env.max_float(3.5) == 3.5 and env.sum_float(2.0) == 2.0
    assert shard_requests(7, 0, 1) == list(range(7))
    assert sum(len(shard_requests(7, r, 3)) for r in range(3)) == 7
