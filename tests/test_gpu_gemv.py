"""GPU parity: fused dequant + GEMV / small-batch and fallback GEMM against the FP64 oracle."""
import numpy as np
import pytest
import torch

from paper_2507_11959_b200 import synth
from tests.gpu_util import PotCase, UintCase, bits_of, f16_dev, gate, to_dev

pytestmark = pytest.mark.gpu

# (N, K): one unit, several units + partial 512-chunk, split-K shapes, a ragged N for the canonical path
TILED_SHAPES = [(16, 128), (48, 640), (256, 4096), (64, 11008), (512, 1664)]
CANON_SHAPES = [(1, 128), (37, 1152), (130, 2176)]


@pytest.fixture(scope="module")
def B():
    from tests.gpu_util import GuardedBinding
    return GuardedBinding()  # outputs and workspaces between canary pads, checked after every call


def acts(M, K, seed):
    return synth.activations(synth.rng_for(4, seed), M, K)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
def test_pot_gemv_matches_oracle(B, oracle, bits, G):
    for i, (N, K) in enumerate(TILED_SHAPES + CANON_SHAPES):
        c = PotCase(N, K, bits, G, dist="t5", seed=(4, 10 * bits + i))
        X = acts(1, K, 100 + i)
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
        y = B.pot_gemv(c.d_packed, c.d_S, K, bits, G, f16_dev(X[0]), B.CANONICAL)
        ok, worst, tight = gate(bits_of(y), Y[0], A[0])
        assert ok and tight < 4.0, ("canonical", N, K, worst, tight)
        if N % 16 == 0:
            y = B.pot_gemv(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X[0]), B.TILED)
            ok, worst, tight = gate(bits_of(y), Y[0], A[0])
            assert ok and tight < 4.0, ("tiled", N, K, worst, tight)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_pot_gemv_one_hot_returns_dequantized_column(B, oracle, bits):
    """x = e_j: every other product is +-0, so y must equal column j of the dequantized matrix bit
    for bit -- pins the layout, the repack and the group -> scale mapping through the fused kernels."""
    G, N, K = 64, 64, 1152
    c = PotCase(N, K, bits, G, dist="normal", seed=(4, 50 + bits))
    deq, _ = oracle.dequant(c.packed, c.S, K, bits, G)
    tiled, tiled_S = c.tiled(), c.tiled_S()
    for j in (0, 1, 2, 3, 63, 64, 127, 128, 129, 500, 511, 512, 1023, 1151):
        x = np.zeros(K, dtype=np.uint16)
        x[j] = 0x3C00
        for layout, P, S in ((B.CANONICAL, c.d_packed, c.d_S), (B.TILED, tiled, tiled_S)):
            y = bits_of(B.pot_gemv(P, S, K, bits, G, f16_dev(x), layout))
            assert np.array_equal(y, deq[:, j]), (layout, j)
            Yg = bits_of(B.pot_gemm(P, S, K, bits, G, f16_dev(x).reshape(1, K), layout))
            assert np.array_equal(Yg[0], deq[:, j]), ("gemm", layout, j)


def test_pot_gemv_closed_form_and_determinism(B, oracle):
    bits, G, N, K = 3, 128, 4096, 11008          # split-K configuration of the tiled kernel
    assert B.pot_gemv_workspace_bytes(N, K, bits, G) > 0
    c = PotCase(N, K, bits, G, dist="t5", seed=(4, 60))
    x = f16_dev(acts(1, K, 160)[0])
    tiled, tiled_S = c.tiled(), c.tiled_S()
    ws = B.new_workspace(B.pot_gemv_workspace_bytes(N, K, bits, G))
    y0 = bits_of(B.pot_gemv(tiled, tiled_S, K, bits, G, x, B.TILED, workspace=ws))
    for _ in range(5):  # same workspace reused: counters must come back to zero; sums in fixed order
        assert np.array_equal(bits_of(B.pot_gemv(tiled, tiled_S, K, bits, G, x, B.TILED, workspace=ws)), y0)
    # all codes 0 (sign +, E = 0), x = 1: y_i = G * sum_g S_ig
    S = np.full((16, 4), 0x2000, dtype=np.uint16)
    S[:, 1] = 0x2400
    packed = np.zeros((16, 512 * bits // 8), dtype=np.uint8)
    ones = f16_dev(np.full(512, 0x3C00, dtype=np.uint16))
    y = B.pot_gemv(B.pot_repack(to_dev(packed), 512, bits, 0), B.pot_repack_scales(f16_dev(S), 512, 128, 0), 512, bits, 128, ones, B.TILED)
    assert torch.all(y.float() == 128 * (3 * 2.0 ** -7 + 2.0 ** -6))


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
def test_uint_gemv_matches_oracle(B, oracle, bits, G):
    for i, (N, K) in enumerate(TILED_SHAPES[:4] + CANON_SHAPES[:2]):
        c = UintCase(N, K, bits, G, dist="t5", seed=(4, 300 + 10 * bits + i))
        X = acts(1, K, 400 + i)
        Y, A = oracle.uint_matmul(c.packed, c.S, c.Z, K, bits, G, X)
        y = B.uint_gemv(c.d_packed, c.d_S, c.d_Z, K, bits, G, f16_dev(X[0]), B.CANONICAL)
        ok, worst, tight = gate(bits_of(y), Y[0], A[0])
        assert ok and tight < 4.0, ("canonical", N, K, worst, tight)
        if N % 16 == 0:
            y = B.uint_gemv(c.tiled(), c.tiled_S(), c.tiled_Z(), K, bits, G, f16_dev(X[0]), B.TILED)
            ok, worst, tight = gate(bits_of(y), Y[0], A[0])
            assert ok and tight < 4.0, ("tiled", N, K, worst, tight)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 7, 8, 13, 16, 32])
def test_pot_gemm_small_batch_matches_oracle(B, oracle, bits, M):
    """M = 1: the GEMV kernel; 2 / 3-4 / 5-8 tokens: the streaming kernel with 2 / 4 / 8 token slots (K = 11008 at 5-8
    tokens: the tcgen05 kernel, its activation block does not fit in shared memory); above: the tcgen05 kernel."""
    G = 128
    for i, (N, K) in enumerate([(48, 640), (256, 4096), (64, 11008)]):
        c = PotCase(N, K, bits, G, dist="t5", seed=(4, 500 + 10 * bits + i))
        X = acts(M, K, 600 + i)
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
        Yg = B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X), B.TILED)
        ok, worst, tight = gate(bits_of(Yg), Y, A)
        assert ok and tight < 4.0, ("small", N, K, M, worst, tight)
        # every row of the batch equals the separate GEMV within the gate
        y0 = B.pot_gemv(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X[M - 1]), B.TILED)
        assert gate(bits_of(y0), Y[M - 1], A[M - 1])[0]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("M", [1, 33, 64, 100])
def test_pot_gemm_fallback_matches_oracle(B, oracle, bits, M):
    G = 64
    for i, (N, K) in enumerate([(37, 384), (130, 1152)]):
        c = PotCase(N, K, bits, G, dist="normal", seed=(4, 700 + 10 * bits + i))
        X = acts(M, K, 800 + i)
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
        Yg = B.pot_gemm(c.d_packed, c.d_S, K, bits, G, f16_dev(X), B.CANONICAL)
        ok, worst, tight = gate(bits_of(Yg), Y, A)
        assert ok and tight < 4.0, ("fallback", N, K, M, worst, tight)


@pytest.mark.parametrize("M", [2, 4])
def test_small_batch_with_activations_too_long_for_shared_memory(B, oracle, M):
    """K = 28672: two tokens still fit in the streaming kernel's staging area (two token slots), four do not and are
    read from global memory for every unit."""
    bits, G, N, K = 3, 128, 32, 28672
    c = PotCase(N, K, bits, G, dist="t5", seed=(4, 950))
    X = acts(M, K, 951)
    Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
    Yg = B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X), B.TILED)
    ok, worst, tight = gate(bits_of(Yg), Y, A)
    assert ok and tight < 4.0, (M, worst, tight)
    assert B.pot_debug_errors() == (0, 0, 0)


def test_gemv_with_activations_too_long_for_shared_memory(B, oracle):
    """K = 65536: the activation vector (128 KB) no longer fits the kernel's shared-memory staging area and is read
    from global memory instead -- PoT and uniform twin."""
    bits, G, N, K = 3, 128, 32, 65536
    X = acts(1, K, 900)
    c = PotCase(N, K, bits, G, dist="t5", seed=(4, 900))
    Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
    y = B.pot_gemv(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X[0]), B.TILED)
    ok, worst, tight = gate(bits_of(y), Y[0], A[0])
    assert ok and tight < 4.0, ("pot", worst, tight)
    u = UintCase(N, K, bits, G, dist="t5", seed=(4, 901))
    Y, A = oracle.uint_matmul(u.packed, u.S, u.Z, K, bits, G, X)
    y = B.uint_gemv(u.tiled(), u.tiled_S(), u.tiled_Z(), K, bits, G, f16_dev(X[0]), B.TILED)
    ok, worst, tight = gate(bits_of(y), Y[0], A[0])
    assert ok and tight < 4.0, ("uint", worst, tight)
    assert B.pot_debug_errors() == (0, 0, 0)
