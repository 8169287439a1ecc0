"""The two collectives of the vocabulary-parallel draft step, on CPU with two gloo ranks."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch, torch.distributed as dist
from paper_2411_18462_b200 import vocab_parallel as VP
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=2)
r = dist.get_rank()
partial = torch.full((3, 4), float(r + 1))
g = VP.gather_partials(partial)
tok = torch.tensor([7, -1, -1] if r == 0 else [-1, 9, -1], dtype=torch.int32)
VP.share_tokens(tok)
lo, hi = VP.shard_bounds(1000, 2, r)
print("RESULT", r, tuple(g.shape), g[0, 0, 0].item(), g[1, 2, 3].item(), tok.tolist(), lo, hi)
dist.barrier(); dist.destroy_process_group()
""" % ROOT


def test_two_gloo_ranks_exchange():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = [subprocess.Popen([sys.executable, "-c", WORKER], env=dict(os.environ, RANK=str(r), PORT=str(port)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    lines = sorted(l for o in outs for l in o.splitlines() if l.startswith("RESULT"))
    assert lines[0] == "RESULT 0 (2, 3, 4) 1.0 2.0 [7, 9, -1] 0 504"
    assert lines[1] == "RESULT 1 (2, 3, 4) 1.0 2.0 [7, 9, -1] 504 1000"
