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
        print(f"RESULT {rank} {t} {s} {lo} {hi}", flush=True)
        pdist.shutdown()
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


def test_two_gloo_ranks_row_sharded_gemv_chain_equals_single_rank(oracle):
    """Two dependent row-sharded GEMVs (the second consumes the gathered output of the first) on two gloo ranks give,
    on every rank, exactly the single-rank result.  The ranks' local GEMV is the oracle here (no GPU in this test):
    what is tested is the sharding, the padding of unequal shards and the gather."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        import numpy as np, torch
        from oracle import pot_oracle as oracle
        from paper_2507_11959_b200 import dist as pdist, synth
        rank, local, world = pdist.init("gloo")
        bits, G = 3, 128
        shapes = [(176, 256), (256, 176 + 80)]          # 11 row blocks over 2 ranks: unequal shards; then equal ones
        mats = []
        for i, (N, K) in enumerate(shapes):
            W = synth.weights(synth.rng_for(0, 900 + i), N, K, "t5")
            codes, S = oracle.quantize(W, bits, G, oracle.RULE_TOP)
            mats.append((oracle.pack(codes, bits), S, N, K))
        def to_f16_bits(y):  # FP64 -> FP16 bits, the rounding the GPU kernels apply to their FP32 sums
            return np.ascontiguousarray(y.astype(np.float16)).view(np.uint16)
        def ref_gemv(packed, S, K, x_bits):
            Y, _ = oracle.matmul(packed, S, K, bits, G, x_bits.reshape(1, K))
            return to_f16_bits(Y[0])
        x0 = synth.activations(synth.rng_for(0, 950), 1, 256)[0]
        # single-rank reference chain (the second GEMV reads the first 256 outputs... of a 176-vector padded with x0)
        y1 = ref_gemv(mats[0][0], mats[0][1], 256, x0)
        x1 = np.concatenate([y1, x0[:80]])
        y2 = ref_gemv(mats[1][0], mats[1][1], 256, x1)
        # sharded chain; 16-bit patterns travel as int32 tensors (gloo has no uint16)
        ident = lambda t: t
        as_t = lambda a: torch.from_numpy(np.ascontiguousarray(a).astype(np.int32))
        as_u16 = lambda t: t.numpy().astype(np.uint16)
        sh = [pdist.RowShard(torch.from_numpy(p), as_t(S), K, bits, G, rank, world, repack=ident, repack_scales=ident)
              for (p, S, N, K) in mats]
        def lg(c, s, K, bits_, group, xx):
            return as_t(ref_gemv(c.numpy(), as_u16(s), K, as_u16(xx)))
        g1 = pdist.sharded_gemv(sh[0], as_t(x0), torch.zeros(176, dtype=torch.int32), gemv=lg)
        xs = torch.cat([g1, as_t(x0[:80])])
        g2 = pdist.sharded_gemv(sh[1], xs, torch.zeros(256, dtype=torch.int32), gemv=lg)
        ok = bool(np.array_equal(as_u16(g1), y1) and np.array_equal(as_u16(g2), y2))
        print(f"RESULT {rank} {ok} {sh[0].begin} {sh[0].end} {sh[0].even} {sh[1].even}", flush=True)
        pdist.shutdown()
    """ % str(ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = sorted(line.split()[1:] for o, _ in outs for line in o.splitlines() if line.startswith("RESULT"))
    assert res == [["0", "True", "0", "96", "False", "True"], ["1", "True", "96", "176", "False", "True"]], res
