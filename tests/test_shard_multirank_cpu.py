"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, max-over-ranks timing, token split."""
import os
import socket
import subprocess
import sys

import pytest

from paper_2304_01089_b200 import shard

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
from paper_2304_01089_b200 import shard
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
dist.barrier()
ms = shard.max_over_ranks([10.0 + 5.0 * rank, 3.0 - rank], dist)
lo, hi = shard.token_range(4097, rank, world)
if rank == 0:
    print("RESULT", ms[0], ms[1], shard.aggregate_throughput(1000.0, world, ms[0]), lo, hi)
else:
    print("RANK1", lo, hi)
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_token_ranges_tile_the_batch():
    for total, world in ((4096, 8), (4097, 2), (5, 8), (0, 3)):
        spans = [shard.token_range(total, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == total
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.token_range(10, 2, 2)


def test_two_gloo_ranks_report_the_slowest_rank():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD, ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = [l for l in outs[0][0].splitlines() if l.startswith("RESULT")][0].split()
    assert float(line[1]) == 15.0 and float(line[2]) == 3.0
    assert abs(float(line[3]) - 2 * 1000.0 / 15e-3) < 1e-6
    assert (int(line[4]), int(line[5])) == (0, 2049)
    assert outs[1][0].split()[1:] == ["2049", "4097"]
