"""The N>1 host logic on CPU: two gloo ranks, row sharding, max-over-ranks timing reduction."""
import os
import socket
import subprocess
import sys
import textwrap
from pathlib import Path

from paper_2507_11959_b200 import dist as pdist

ROOT = Path(__file__).resolve().parent.parent


def test_shard_rows_partitions_in_blocks_of_16():
    for N in (16, 4096, 11008, 12288, 48):
        for world in (1, 2, 3, 4, 8):
            spans = [pdist.shard_rows(N, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == N
            for (a, b), (c, d) in zip(spans, spans[1:]):
                assert b == c
            sizes = [b - a for a, b in spans]
            assert all(s % 16 == 0 for s in sizes) and max(sizes) - min(sizes) <= 16


def test_two_gloo_ranks_reduce_timing_and_shard():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        from paper_2507_11959_b200 import dist as pdist
        rank, local, world = pdist.init("gloo")
        assert world == 2
        pdist.barrier()
        t = pdist.max_over_ranks(1.0 + rank)
        s = pdist.sum_over_ranks(10.0 * (rank + 1))
        lo, hi = pdist.shard_rows(4096, rank, world)
        print(f"RESULT {rank} {t} {s} {lo} {hi}")
    """ % str(ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = sorted(line.split()[1:] for o in outs for line in o.splitlines() if line.startswith("RESULT"))
    assert res == [["0", "2.0", "30.0", "0", "2048"], ["1", "2.0", "30.0", "2048", "4096"]]
