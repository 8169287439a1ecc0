"""The N > 1 path on CPU: two gloo ranks shard a batch and reduce (max time, sum bytes)."""
import os
import socket
import subprocess
import sys

from paper_2411_18462_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
from paper_2411_18462_b200 import sharding, workloads
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=2)
rank = dist.get_rank()
w = workloads.make_workload("chat", seed=sharding.rank_seed(7, rank), B=2, V=64, threads=1)
ms, units = sharding.aggregate(10.0 + 5.0 * rank, float(w.q_logits.nbytes))
lo, hi = sharding.shard_sequences(5, rank, 2)
print("RESULT", rank, ms, units, lo, hi, int(w.q_logits[0, 0]))
dist.barrier()
dist.destroy_process_group()
""" % ROOT


def test_shard_sequences_cover_the_batch():
    for n in (1, 5, 128, 129):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_sequences(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


def test_aggregate_without_process_group_is_identity():
    assert sharding.aggregate(3.5, 100.0) == (3.5, 100.0)


def test_two_gloo_ranks():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = {}
    for o in outs:
        line = [l for l in o.splitlines() if l.startswith("RESULT")][0].split()
        res[int(line[1])] = line[2:]
    # both ranks see max time 15 ms and the sum of the two ranks' bytes
    assert float(res[0][0]) == 15.0 and float(res[1][0]) == 15.0
    assert float(res[0][1]) == float(res[1][1]) == 2 * (2 * 16 * 64 * 2)
    assert (res[0][2], res[0][3], res[1][2], res[1][3]) == ("0", "3", "3", "5")
    assert res[0][4] != res[1][4]     # different seeds -> different batches
