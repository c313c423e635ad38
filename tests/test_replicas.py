"""The multi-GPU path has no data exchange; what there is to test is the
timing aggregation and the partition arithmetic, run here as two gloo ranks."""
import os
import socket
import subprocess
import sys

from paper_2608_10103_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %(root)r)
import torch, torch.distributed as dist
from paper_2608_10103_b200 import replicas
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
mine = [10.0 + rank, 5.0 - rank, 1.0]
out = replicas.max_over_ranks(mine, dist)
lo, hi = replicas.row_block(1000, rank, world)
spans = [None] * world
dist.all_gather_object(spans, (lo, hi))
dist.barrier()
if rank == 0:
    print(json.dumps({"max": out, "spans": spans, "seed": replicas.replica_seed(3, 1),
                      "rate": replicas.whole_job_rate(2.0e12, world, out[0])}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_max_and_cover_rows(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % {"root": ROOT})
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["max"] == [11.0, 5.0, 1.0]
    assert res["spans"] == [[0, 512], [512, 1000]]
    assert res["seed"] == 1003
    assert abs(res["rate"] - 2 * 2.0 / 11.0e-3) < 1e-9


def test_row_blocks_partition_exactly():
    for M in (1, 255, 256, 257, 1000, 8192, 8200):
        for world in (1, 2, 3, 4, 8):
            spans = [replicas.row_block(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            assert all(lo <= hi for lo, hi in spans)
            assert all(lo % 256 == 0 for lo, _ in spans if lo < M)


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert replicas.whole_job_rate(1.0e12, 1, 1000.0) == 1.0
