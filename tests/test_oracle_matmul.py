"""Pins for the oracle's FP64 contraction: numpy's matmul, one-hot probes, closed forms."""
import numpy as np
import pytest

from paper_2507_11959_b200 import synth

QMAX = {2: 1, 3: 3, 4: 7}


def _case(oracle, bits, G, N, K, M, dist="t5", seed=0):
    W = synth.weights(synth.rng_for(0, 100 + seed), N, K, dist)
    X = synth.activations(synth.rng_for(0, 200 + seed), M, K)
    codes, S = oracle.quantize(W, bits, G, oracle.RULE_TOP)
    return oracle.pack(codes, bits), S, X


@pytest.mark.parametrize("bits,G", [(2, 128), (3, 128), (4, 64), (3, 64)])
def test_matmul_matches_numpy(oracle, bits, G):
    N, K, M = 96, 1024, 5
    packed, S, X = _case(oracle, bits, G, N, K, M, seed=bits)
    deq, _ = oracle.dequant(packed, S, K, bits, G)
    w = synth.f16_bits_to_f64(deq)      # numpy's half -> double
    x = synth.f16_bits_to_f64(X)
    Y, A = oracle.matmul(packed, S, K, bits, G, X)
    assert Y.shape == (M, N)
    ref = x @ w.T
    refA = np.abs(x) @ np.abs(w).T
    assert np.allclose(Y, ref, rtol=0, atol=1e-12 * refA.max())
    assert np.allclose(A, refA, rtol=1e-13, atol=0)
    # row subset, in the order given
    rows = np.array([7, 0, 95, 33], dtype=np.int64)
    Ys, As = oracle.matmul(packed, S, K, bits, G, X, rows)
    assert np.array_equal(Ys, Y[:, rows]) and np.array_equal(As, A[:, rows])


def test_matmul_one_hot_returns_a_column(oracle):
    bits, G, N, K = 3, 128, 32, 512
    packed, S, _ = _case(oracle, bits, G, N, K, 1)
    deq, _ = oracle.dequant(packed, S, K, bits, G)
    w = synth.f16_bits_to_f64(deq)
    for j in (0, 1, 127, 128, 300, 511):
        x = np.zeros((1, K), dtype=np.uint16)
        x[0, j] = 0x3C00  # 1.0
        Y, A = oracle.matmul(packed, S, K, bits, G, x)
        assert np.array_equal(Y[0], w[:, j]) and np.array_equal(A[0], np.abs(w[:, j]))


def test_matmul_closed_form_all_codes_zero(oracle):
    # every code 0 (sign +, E = 0) and x = 1: y_i = G * sum_g S_ig
    bits, G, N, K = 3, 64, 4, 256
    S = np.array([[0x2000, 0x2400, 0x2800, 0x2C00]] * N, dtype=np.uint16)  # 2^-7, 2^-6, 2^-5, 2^-4
    packed = np.zeros((N, K * bits // 8), dtype=np.uint8)
    x = np.full((1, K), 0x3C00, dtype=np.uint16)
    Y, A = oracle.matmul(packed, S, K, bits, G, x)
    expect = G * (2.0 ** -7 + 2.0 ** -6 + 2.0 ** -5 + 2.0 ** -4)
    assert np.all(Y == expect) and np.all(A == expect)
    # flipping every sign bit negates y and leaves A
    codes = np.full((N, K), 1 << (bits - 1), dtype=np.uint8)
    Y2, A2 = oracle.matmul(oracle.pack(codes, bits), S, K, bits, G, x)
    assert np.all(Y2 == -expect) and np.all(A2 == expect)


def test_matmul_rows_equal_separate_gemvs(oracle):
    bits, G, N, K, M = 3, 128, 16, 512, 4
    packed, S, X = _case(oracle, bits, G, N, K, M, seed=9)
    Y, A = oracle.matmul(packed, S, K, bits, G, X)
    for m in range(M):
        y1, a1 = oracle.matmul(packed, S, K, bits, G, X[m:m + 1])
        assert np.array_equal(y1[0], Y[m]) and np.array_equal(a1[0], A[m])


def _bf16_bits_to_f64(bits):
    """BF16 bit patterns -> FP64 through numpy's float32 view (independent of the oracle's own conversion)"""
    return (np.ascontiguousarray(bits).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _f16_bits_to_bf16_bits(bits):
    """round-to-nearest-even FP16 -> BF16 by integer arithmetic on the float32 pattern"""
    u = np.ascontiguousarray(bits).view(np.float16).astype(np.float32).view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


@pytest.mark.parametrize("bits,G", [(2, 128), (3, 128), (4, 64), (3, 64)])
def test_bf16_matmul_matches_numpy(oracle, bits, G):
    """The BF16 contraction against numpy on the oracle's BF16 dequantization (itself pinned in test_oracle_formats),
    with activations rounded to BF16 by independent integer arithmetic; and a closed form: codes 0, x = 1."""
    N, K, M = 64, 768, 3
    packed, S, X16 = _case(oracle, bits, G, N, K, M, seed=10 + bits)
    Xb = _f16_bits_to_bf16_bits(X16)
    deq, rounded = oracle.dequant(packed, S, K, bits, G, oracle.BF16)
    assert rounded == 0
    w, x = _bf16_bits_to_f64(deq), _bf16_bits_to_f64(Xb)
    Y, A = oracle.matmul(packed, S, K, bits, G, Xb, dtype=oracle.BF16)
    ref, refA = x @ w.T, np.abs(x) @ np.abs(w).T
    assert np.allclose(Y, ref, rtol=0, atol=1e-12 * refA.max()) and np.allclose(A, refA, rtol=1e-13, atol=0)
    # it is not the FP16 contraction: the scale is rounded to 8 significant bits first
    Y16, _ = oracle.matmul(packed, S, K, bits, G, X16)
    assert not np.allclose(Y, Y16, rtol=1e-6, atol=0)
    # all codes 0 (sign +, E = 0), x = 1: y_i = G * sum_g bf16(S_ig), exactly
    z = np.zeros((4, 256 * bits // 8), dtype=np.uint8)
    S2 = np.array([[0x2E66, 0x3555]] * 4, dtype=np.uint16)       # bf16: 0x3DCD, 0x3EAB
    ones = np.full((1, 256), 0x3F80, dtype=np.uint16)
    Y1, _ = oracle.matmul(z, S2, 256, bits, 128, ones, dtype=oracle.BF16)
    expect = 128 * (_bf16_bits_to_f64(np.array([0x3DCD], dtype=np.uint16))[0] + _bf16_bits_to_f64(np.array([0x3EAB], dtype=np.uint16))[0])
    assert np.all(Y1 == expect)
