"""GPU parity at the sizes and launch plans that bench.py times: every configuration's shapes go through the same entry
points with the same plans, and sampled outputs are compared with the oracle element by element (sampled rows of the
FP64 product; sampled rows of the dequantized matrix bit for bit)."""
import numpy as np
import pytest
import torch

from paper_2507_11959_b200 import synth
from tests.gpu_util import GuardedBinding, PotCase, UintCase, bits_of, f16_dev, gate

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    return GuardedBinding()


def sample_rows(N, seed, n=48):
    """first / last rows, rows around the 16-row block and CTA boundaries, and seeded random rows"""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 15, 16, 17, N // 2 - 1, N // 2, N - 17, N - 16, N - 1]
    rows = np.unique(np.concatenate([np.array(fixed), rng.integers(0, N, n)]))
    return rows[(rows >= 0) & (rows < N)].astype(np.int64)


def check_gemv(B, oracle, N, K, bits, dist, seed, expect_plan=None):
    c = PotCase(N, K, bits, 128, dist=dist, seed=seed)
    X = synth.activations(synth.rng_for(seed[0], seed[1] + 1), 1, K)
    rows = sample_rows(N, seed[1])
    Y, A = oracle.matmul(c.packed, c.S, K, bits, 128, X, rows=rows)
    plan = B.pot_debug_gemv_plan(N, K, bits, 128)
    if expect_plan is not None:
        for k, v in expect_plan.items():
            assert plan[k] == v, (N, K, bits, plan)
    y = bits_of(B.pot_gemv(c.tiled(), c.tiled_S(), K, bits, 128, f16_dev(X[0]), B.TILED))
    assert B.pot_debug_errors() == (0, 0, 0)
    ok, worst, tight = gate(y[rows], Y[0], A[0])
    assert ok and tight < 4.0, (N, K, bits, worst, tight)
    return plan


def test_config1_gemv_4096x4096_3bit(B, oracle):
    check_gemv(B, oracle, 4096, 4096, 3, "normal", (1, 0), {"row_block_split": 1})


@pytest.mark.parametrize("bits", [2, 3])
def test_config2_llama7b_projections(B, oracle, bits):
    """The five 7B projections as bench.py runs them: every one takes the two-CTAs-per-SM variant (a chain must not mix
    the variants); the one-CTA variant is reached by the 28672 x 8192 and 13B tests below."""
    seen = set()
    for i, pr in enumerate(synth.LLAMA2_7B):
        if pr.name == "up":
            continue  # same shape as gate
        plan = check_gemv(B, oracle, pr.N, pr.K, bits, "t5", (2, 2 * i))
        seen.add(plan["ctas_per_sm"])
        assert plan["units_per_slot"] == (2 if pr.K == 11008 and bits == 3 else 4), (pr.name, plan)
    assert seen == {2}, seen


@pytest.mark.parametrize("bits", [3])
def test_config2_uniform_twin_gate_and_down(B, oracle, bits):
    for i, (N, K) in enumerate([(11008, 4096), (4096, 11008)]):
        c = UintCase(N, K, bits, 128, dist="t5", seed=(2, 40 + i))
        X = synth.activations(synth.rng_for(2, 50 + i), 1, K)
        rows = sample_rows(N, 60 + i)
        Y, A = oracle.uint_matmul(c.packed, c.S, c.Z, K, bits, 128, X, rows=rows)
        y = bits_of(B.uint_gemv(c.tiled(), c.tiled_S(), c.tiled_Z(), K, bits, 128, f16_dev(X[0]), B.TILED))
        assert B.pot_debug_errors() == (0, 0, 0)
        ok, worst, tight = gate(y[rows], Y[0], A[0])
        assert ok and tight < 4.0, (N, K, worst, tight)


def test_unit_split_with_sums_crossing_ctas_at_full_width(B, oracle):
    """13B down (5120 x 13824) keeps the even unit split: 320 row blocks of 108 units on 148 CTAs, so most row blocks are
    shared between CTAs and go through the workspace."""
    check_gemv(B, oracle, 5120, 13824, 3, "t5", (4, 30), {"row_block_split": 0})


@pytest.mark.parametrize("M", list(synth.SMALL_BATCH_M))
def test_config4_llama13b_small_batch(B, oracle, M):
    for i, pr in enumerate(synth.LLAMA2_13B):
        c = PotCase(pr.N, pr.K, 3, 128, dist="t5", seed=(4, 2 * i))
        X = synth.activations(synth.rng_for(4, 2 * i + 1), M, pr.K)
        rows = sample_rows(pr.N, 70 + i, n=24)
        Y, A = oracle.matmul(c.packed, c.S, pr.K, 3, 128, X, rows=rows)
        Yg = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), pr.K, 3, 128, f16_dev(X), B.TILED))
        assert B.pot_debug_errors() == (0, 0, 0)
        ok, worst, tight = gate(Yg[:, rows], Y, A)
        assert ok and tight < 4.0, (pr.name, M, worst, tight)


@pytest.mark.parametrize("bits,shape", [(2, 0), (2, 1), (3, 1), (3, 2), (2, 2)])
def test_config5_llama70b_prefill(B, oracle, bits, shape):
    """M = 2048 through the tcgen05 kernel at the benchmarked sizes (8192 -> 10240 at 3 bits is in test_gpu_prefill):
    tile-boundary feature rows plus seeded ones, every token."""
    pr = synth.LLAMA2_70B[shape]
    M = synth.PREFILL_M
    c = PotCase(pr.N, pr.K, bits, 128, dist="normal", sigma=0.015, seed=(5, 200 + 10 * bits + shape))
    X = synth.activations(synth.rng_for(5, 300 + shape), M, pr.K, outliers=False)
    Yg = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), pr.K, bits, 128, f16_dev(X), B.TILED))
    assert B.pot_debug_errors() == (0, 0, 0)
    N = pr.N
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, N - 129, N - 128, N - 1],
                                     synth.rng_for(5, 400 + shape).integers(0, N, 24)])).astype(np.int64)
    Y, A = oracle.matmul(c.packed, c.S, pr.K, bits, 128, X, rows)
    ok, worst, tight = gate(Yg[:, rows], Y, A)
    assert ok and tight < 4.0, (pr.name, bits, worst, tight)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_config3_dequant_largest_matrix_sampled_rows(B, oracle, bits):
    """28672 x 8192 (235 M weights, 64-bit bit offsets inside the kernel): 64 seeded rows plus the first and last, bit
    for bit, FP16 and -- at 3 bits -- BF16; and the uniform twin at the same size."""
    N, K, G = 28672, 8192, 128
    c = PotCase(N, K, bits, G, dist="normal", seed=(3, 500 + bits))
    rows = sample_rows(N, 600 + bits, n=64)
    sub_packed, sub_S = np.ascontiguousarray(c.packed[rows]), np.ascontiguousarray(c.S[rows])
    for dtype in ((0, 1) if bits == 3 else (0,)):
        ref, rounded = oracle.dequant(sub_packed, sub_S, K, bits, G, dtype)
        assert rounded == 0
        out = B.pot_dequant(c.d_packed, c.d_S, K, bits, G, dtype)
        got = bits_of(out[torch.from_numpy(rows).cuda()])
        assert np.array_equal(got, ref), (bits, dtype)
        del out
    # the same matrix through the fused GEMV (a share per CTA large enough for the one-CTA-per-SM variant)
    plan = B.pot_debug_gemv_plan(N, K, bits, G)
    assert plan["ctas_per_sm"] == 1 and plan["units_per_slot"] == (4 if bits == 4 else 8), plan
    X = synth.activations(synth.rng_for(3, 650 + bits), 1, K)
    Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X, rows=rows)
    y = bits_of(B.pot_gemv(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X[0]), B.TILED))
    ok, worst, tight = gate(y[rows], Y[0], A[0])
    assert ok and tight < 4.0 and B.pot_debug_errors() == (0, 0, 0), (bits, worst, tight)
    if bits == 3:
        u = UintCase(N, K, bits, G, dist="normal", W_bits=c.W_bits)
        ref = oracle.uint_dequant(np.ascontiguousarray(u.packed[rows]), np.ascontiguousarray(u.S[rows]),
                                  np.ascontiguousarray(u.Z[rows]), K, bits, G)
        out = B.uint_dequant(u.d_packed, u.d_S, u.d_Z, K, bits, G, B.UINT_FAST)
        got = bits_of(out[torch.from_numpy(rows).cuda()])
        zero = (ref & 0x7FFF) == 0
        assert np.array_equal(got[~zero], ref[~zero]) and np.all((got[zero] & 0x7FFF) == 0)


@pytest.mark.parametrize("N,K", [(4096, 4096), (8192, 8192)])
def test_config3_dequant_other_sizes_group_64_and_128(B, oracle, N, K):
    for bits, G in ((3, 64), (2, 128), (4, 64)):
        c = PotCase(N, K, bits, G, dist="normal", seed=(3, 700 + bits + G))
        rows = sample_rows(N, 800 + bits, n=32)
        ref, rounded = oracle.dequant(np.ascontiguousarray(c.packed[rows]), np.ascontiguousarray(c.S[rows]), K, bits, G)
        assert rounded == 0
        out = B.pot_dequant(c.d_packed, c.d_S, K, bits, G, 0)
        assert np.array_equal(bits_of(out[torch.from_numpy(rows).cuda()]), ref), (N, K, bits, G)


def test_workspace_shared_between_shapes_after_clearing(B, oracle):
    """A workspace may be reused by calls of the same shape as it is; handed to another shape it must be cleared first
    (the counters sit at shape-dependent offsets).  Alternate two shapes on one buffer, clearing in between."""
    bits, G = 3, 128
    shapes = [(256, 4096), (64, 11008)]
    cases = [PotCase(N, K, bits, G, dist="t5", seed=(4, 950 + i)) for i, (N, K) in enumerate(shapes)]
    need = max(B.pot_gemv_workspace_bytes(N, K, bits, G) for N, K in shapes)
    ws = B.new_workspace(need)
    for rep in range(3):
        for c in cases:
            X = synth.activations(synth.rng_for(4, 960 + rep), 1, c.K)
            Y, A = oracle.matmul(c.packed, c.S, c.K, bits, G, X)
            for again in range(2):  # same shape twice without clearing
                y = bits_of(B.pot_gemv(c.tiled(), c.tiled_S(), c.K, bits, G, f16_dev(X[0]), B.TILED, workspace=ws))
                ok, worst, tight = gate(y, Y[0], A[0])
                assert ok and tight < 4.0, (c.N, c.K, rep, again, worst, tight)
            ws.zero_()
    assert ws._guard.intact()
