"""Pins for the uniform (zero-point) twin: w~ = (W_Q + Z) o S with Z = -z  (Sec. 4.1)."""
from fractions import Fraction

import numpy as np
import pytest

from paper_2507_11959_b200 import synth
from tests.test_oracle_formats import f16_fraction


def rne_to_f16_exact(v: Fraction) -> int:
    """Round an exact rational to FP16 (ties to even) by searching the neighbouring patterns."""
    sign = 0x8000 if v < 0 else 0
    a = abs(v)
    lo, hi = 0, 0x7BFF
    while lo < hi:  # largest pattern whose value is <= a
        mid = (lo + hi + 1) // 2
        if f16_fraction(mid) <= a:
            lo = mid
        else:
            hi = mid - 1
    below, above = f16_fraction(lo), f16_fraction(min(lo + 1, 0x7BFF))
    if a - below < above - a or lo == 0x7BFF:
        return sign | lo
    if a - below > above - a:
        return sign | (lo + 1)
    return sign | (lo if lo % 2 == 0 else lo + 1)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_uniform_dequant_enumeration(oracle, bits):
    """every (q, z) pair x a sample of scales: one rounding of the exact product (q - z) * s."""
    L = 1 << bits
    rng = np.random.default_rng(bits)
    scales = np.concatenate([[0x0400, 0x2E66, 0x3555, 0x1D1F], rng.integers(0x0400, 0x4000, 24)]).astype(np.uint16)
    G = 16
    for z in range(L):
        codes = np.tile(np.arange(G, dtype=np.uint8) % L, (scales.size, 1))
        Z = np.full((scales.size, 1), np.float16(z).view(np.uint16), dtype=np.uint16)
        out = oracle.uint_dequant(oracle.pack(codes, bits), scales.reshape(-1, 1), Z, G, bits, G)
        for r in range(scales.size):
            s = f16_fraction(int(scales[r]))
            for q in range(L):
                assert int(out[r, q]) == rne_to_f16_exact((q - z) * s) or ((q - z) == 0 and out[r, q] in (0, 0x8000))


def rint_exact(v: Fraction) -> int:
    f = v.numerator // v.denominator
    r = v - f
    if r > Fraction(1, 2) or (r == Fraction(1, 2) and f % 2 == 1):
        return f + 1
    return f


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_uniform_quantizer_exact_on_small_groups(oracle, bits):
    L = (1 << bits) - 1
    G = 16
    W = synth.weights(synth.rng_for(0, 300 + bits), 32, G, "normal")
    codes, S, Z = oracle.uint_quantize(W, bits, G)
    for i in range(W.shape[0]):
        w = [f16_fraction(int(b)) for b in W[i]]
        mn, mx = min(w), max(w)
        sb = max(rne_to_f16_exact((mx - mn) / L), 0x0400)
        assert int(S[i, 0]) == sb
        s = f16_fraction(sb)
        z = min(max(rint_exact(-mn / s), 0), L)
        assert f16_fraction(int(Z[i, 0])) == z
        q = [min(max(rint_exact(v / s) + z, 0), L) for v in w]
        assert codes[i].tolist() == q


def test_uniform_reconstruction_error_bound(oracle):
    # inside the clipping range a uniform quantizer is off by at most s/2 (plus one FP16 rounding)
    bits, G = 4, 128
    W = synth.weights(synth.rng_for(0, 310), 64, 1024, "normal")
    codes, S, Z = oracle.uint_quantize(W, bits, G)
    deq = oracle.uint_dequant(oracle.pack(codes, bits), S, Z, 1024, bits, G)
    w, d = synth.f16_bits_to_f64(W), synth.f16_bits_to_f64(deq)
    s = np.repeat(synth.f16_bits_to_f64(S), G, axis=1)
    assert np.all(np.abs(w - d) <= 0.5 * s * (1 + 2 ** -9) + s * 1.001)  # z rounding can shift the grid by < s
    assert np.mean(np.abs(w - d) <= 0.5 * s * (1 + 2 ** -9)) > 0.95


def test_uniform_matmul_matches_numpy(oracle):
    bits, G, N, K, M = 3, 128, 48, 512, 3
    W = synth.weights(synth.rng_for(0, 320), N, K, "t5")
    X = synth.activations(synth.rng_for(0, 321), M, K)
    codes, S, Z = oracle.uint_quantize(W, bits, G)
    packed = oracle.pack(codes, bits)
    w = synth.f16_bits_to_f64(oracle.uint_dequant(packed, S, Z, K, bits, G))
    x = synth.f16_bits_to_f64(X)
    Y, A = oracle.uint_matmul(packed, S, Z, K, bits, G, X)
    assert np.allclose(Y, x @ w.T, rtol=0, atol=1e-12 * A.max())
    assert np.allclose(A, np.abs(x) @ np.abs(w).T, rtol=1e-13)
