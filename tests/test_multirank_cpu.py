"""World-size-2 CPU check (gloo) of the multi-rank logic the bench uses: the path has no data-path collective,
ranks draw different batches (weak scaling) and the reported time is the max over ranks."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import numpy as np
import torch
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = bench.make_workload("cfg2", seed_offset=rank, batch=4)
ctx_sum = int(w.tables.ctx_len.sum())
t = torch.tensor([10.0 + rank], dtype=torch.float64)       # stand-in for a per-rank device time
dist.barrier()
dist.all_reduce(t, op=dist.ReduceOp.MAX)
sums = [None] * world
dist.all_gather_object(sums, ctx_sum)
if rank == 0:
    print(json.dumps({{"tmax": float(t.item()), "ctx_sums": sums, "tokens_per_step": w.tables.batch * world}}))
dist.destroy_process_group()
"""


def test_two_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), str(script)]
    env = dict(os.environ, OMP_NUM_THREADS="1")
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["tmax"] == 11.0                       # max over ranks, not rank 0's own time
    assert res["ctx_sums"][0] != res["ctx_sums"][1]  # ranks draw different batches
    assert res["tokens_per_step"] == 8
