"""world_size-2 gloo test of the multi-rank plumbing (timing reduction, row sharding)."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
from paper_2510_02822_b200 import dist
rank, local, world = dist.init("gloo")
dist.barrier()
mx = dist.max_over_ranks(10.0 + rank)
sm = dist.sum_over_ranks(100.0 * (rank + 1))
lo, hi = dist.shard_rows(12608, rank, world)
cover = dist.sum_over_ranks(hi - lo)
assert mx == 11.0 and sm == 300.0 and cover == 12608, (mx, sm, cover)
print("rank", rank, "ok", lo, hi)
"""


def test_two_rank_timing_reduction_and_sharding(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29533")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
        assert "ok" in o


def test_shard_rows_partition():
    from paper_2510_02822_b200 import dist
    for M in (0, 1, 7, 197, 12608):
        for world in (1, 2, 3, 8):
            spans = [dist.shard_rows(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
