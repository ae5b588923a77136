"""GPU parity of the BF16 route (BF16 activations, BF16 reconstruction w~ = +-2^E bf16(S), BF16 output) through the
fused GEMV and GEMM kernels, against the oracle's BF16 contraction; one-hot activations pin the decode bit for bit."""
import numpy as np
import pytest

from paper_2507_11959_b200 import synth
from tests.gpu_util import GuardedBinding, PotCase, bf16_dev, bits_of, f16_bits_to_bf16_bits, gate

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    return GuardedBinding()


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
def test_bf16_gemv_matches_oracle(B, oracle, bits, G):
    for i, (N, K) in enumerate([(16, 128), (48, 640), (256, 4096), (64, 11008), (37, 1152), (1024, 2048)]):
        c = PotCase(N, K, bits, G, dist="t5", seed=(7, 10 * bits + i))
        Xb = f16_bits_to_bf16_bits(synth.activations(synth.rng_for(7, 100 + i), 1, K))
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, Xb, dtype=oracle.BF16)
        y = B.pot_gemv(c.d_packed, c.d_S, K, bits, G, bf16_dev(Xb[0]), B.CANONICAL)
        ok, worst, tight = gate(bits_of(y), Y[0], A[0], bf16=True)
        assert ok and tight < 4.0, ("canonical", N, K, worst, tight)
        if N % 16 == 0:
            y = B.pot_gemv(c.tiled(), c.tiled_S(), K, bits, G, bf16_dev(Xb[0]), B.TILED)
            ok, worst, tight = gate(bits_of(y), Y[0], A[0], bf16=True)
            assert ok and tight < 4.0, ("tiled", N, K, worst, tight)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_bf16_one_hot_returns_the_bf16_dequantized_column(B, oracle, bits):
    """x = e_j in BF16: y must equal column j of the BF16 dequantization bit for bit, through every kernel route."""
    G, N, K = 64, 64, 1152
    c = PotCase(N, K, bits, G, dist="normal", seed=(7, 50 + bits))
    deq, _ = oracle.dequant(c.packed, c.S, K, bits, G, oracle.BF16)
    tiled, tiled_S = c.tiled(), c.tiled_S()
    for j in (0, 1, 2, 3, 31, 32, 63, 64, 127, 128, 129, 500, 1023, 1151):
        x = np.zeros(K, dtype=np.uint16)
        x[j] = 0x3F80
        for layout, P, S in ((B.CANONICAL, c.d_packed, c.d_S), (B.TILED, tiled, tiled_S)):
            assert np.array_equal(bits_of(B.pot_gemv(P, S, K, bits, G, bf16_dev(x), layout)), deq[:, j]), (layout, j)
            assert np.array_equal(bits_of(B.pot_gemm(P, S, K, bits, G, bf16_dev(x).reshape(1, K), layout))[0], deq[:, j]), ("gemm", layout, j)
    # the tcgen05 route: 40 one-hot tokens
    ks = (np.arange(40) * 29 + 3) % K
    X = np.zeros((40, K), dtype=np.uint16)
    X[np.arange(40), ks] = 0x3F80
    Yg = bits_of(B.pot_gemm(tiled, tiled_S, K, bits, G, bf16_dev(X), B.TILED))
    assert np.array_equal(Yg, deq[:, ks].T)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("M", [4, 8, 20, 200])
def test_bf16_gemm_matches_oracle(B, oracle, bits, M):
    G = 128
    for i, (N, K) in enumerate([(48, 640), (272, 1152), (256, 4096)]):
        c = PotCase(N, K, bits, G, dist="t5", seed=(7, 500 + 10 * bits + i))
        Xb = f16_bits_to_bf16_bits(synth.activations(synth.rng_for(7, 600 + i), M, K))
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, Xb, dtype=oracle.BF16)
        for layout, P, S in ((B.TILED, c.tiled(), c.tiled_S()), (B.CANONICAL, c.d_packed, c.d_S)):
            Yg = B.pot_gemm(P, S, K, bits, G, bf16_dev(Xb), layout)
            ok, worst, tight = gate(bits_of(Yg), Y, A, bf16=True)
            assert ok and tight < 4.0, (layout, N, K, M, worst, tight)
