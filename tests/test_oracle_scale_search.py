"""Pins for the oracle's Algorithm 1 (data-agnostic scale initialisation)."""
import numpy as np
import pytest

from paper_2507_11959_b200 import synth

QMAX = {2: 1, 3: 3, 4: 7}


def q1_curve(w, qmax):
    """Q1(b) for all 200 candidates, numpy FP64 (an independent evaluation of the objective)."""
    amax = np.abs(w).max()
    s0 = amax / (2.0 ** qmax - 1)
    out = np.empty(200)
    for i in range(1, 201):
        sb = s0 * (0.01 * i)
        with np.errstate(divide="ignore"):
            E = np.clip(np.rint(np.log2(np.abs(w) / sb)), 0, qmax)
        rec = np.where(w < 0, -1.0, 1.0) * sb * 2.0 ** E
        out[i - 1] = np.sum((w - rec) ** 2)
    return s0, out


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("dist", ["normal", "t5"])
def test_search_attains_the_grid_minimum(oracle, bits, dist):
    G = 128
    W = synth.weights(synth.rng_for(0, 400 + bits), 8, 4 * G, dist)
    S, bstar = oracle.scale_search(W, bits, G)
    w = synth.f16_bits_to_f64(W).reshape(-1, G)
    for g in range(w.shape[0]):
        s0, q1 = q1_curve(w[g], QMAX[bits])
        i = int(bstar.ravel()[g])
        assert 1 <= i <= 200
        assert q1[i - 1] <= q1.min() * (1 + 1e-12)
        assert np.all(q1[: i - 1] > q1[i - 1] * (1 - 1e-12))  # ties keep the smallest b
        ref = np.float16(s0 * (0.01 * i))
        assert S.ravel()[g] == max(int(ref.view(np.uint16)), 0x0400)
    # the paper notes that chosen multipliers often deviate from b = 1
    assert np.mean(bstar != 100) > 0.5


def test_search_closed_form_equal_magnitudes(oracle):
    """All |w| equal to a: Q1 = 0 iff s0*b*2^E = a.  2-bit: s0 = a, so b = 0.5 (E = 1) and b = 1
    (E = 0) both reconstruct exactly and the smaller wins.  3-bit: s0 = a/7, b*2^E = 7 has the
    grid solutions b = 1.75 (E = 2) only (0.875 and 3.5/… are not multiples of 0.01 in range)."""
    G = 64
    a = np.float16(0.03125)
    W = np.full((1, G), a.view(np.uint16), dtype=np.uint16)
    W[0, ::2] |= 0x8000
    _, b2 = oracle.scale_search(W, 2, G)
    assert b2[0, 0] == 50
    S3, b3 = oracle.scale_search(W, 3, G)
    assert b3[0, 0] == 175
    assert S3.view(np.float16)[0, 0] == np.float16(float(a) / 7 * 1.75)


def test_search_zero_group(oracle):
    W = np.zeros((1, 128), dtype=np.uint16)
    S, b = oracle.scale_search(W, 3, 128)
    assert S[0, 0] == 0x0400 and b[0, 0] == 1
