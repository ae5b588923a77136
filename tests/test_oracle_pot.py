"""Pins for the oracle's PoT quantizer (Eq. 2), packing and reconstruction (Eq. 1).

The oracle evaluates the paper's formulas in FP64.  The pins below use routes that share
nothing with that code: exact integer / rational arithmetic, the integer-add formulation of
Sec. 4.2, hand-derived fixtures, and structural invariants."""
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

from paper_2507_11959_b200 import synth
from tests.test_oracle_formats import _golden_rows, f16_fraction

GOLD = Path(__file__).parent / "golden"
QMAX = {2: 1, 3: 3, 4: 7}


def f16_int_parts(bits: int):
    """finite FP16 pattern -> (m, e) with |value| = m * 2^e, integers."""
    e, m = (bits >> 10) & 31, bits & 1023
    return (m, -24) if e == 0 else (1024 + m, e - 25)


def exact_exponent(wbits: int, sbits: int, qmax: int) -> int:
    """clamp(round(log2(|w|/S)), 0, q_max) in exact integer arithmetic:
    round(t) >= k+1  <=>  t > k + 1/2  <=>  (|w|/S)^2 > 2^(2k+1)   (a tie is impossible)."""
    mw, ew = f16_int_parts(wbits & 0x7FFF)
    ms, es = f16_int_parts(sbits)
    E = 0
    for k in range(qmax):
        # mw^2 * 2^(2ew)  >  2^(2k+1) * ms^2 * 2^(2es)
        lhs, rhs = mw * mw, ms * ms
        sh = 2 * ew - (2 * es + 2 * k + 1)
        if sh >= 0:
            lhs <<= sh
        else:
            rhs <<= -sh
        assert lhs != rhs or mw == 0  # no ties
        E += lhs > rhs
    return E


# ----------------------------------------------------------------- Eq. 2
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_quantizer_matches_exact_integer_evaluation(oracle, bits):
    qmax = QMAX[bits]
    G = 64
    # all finite FP16 magnitudes (both signs), a handful of legal scales supplied by the caller
    wb = np.concatenate([np.arange(0, 0x7C00, dtype=np.uint32), np.arange(0x8000, 0xFC00, 37, dtype=np.uint32)]).astype(np.uint16)
    wb = wb[: (wb.size // G) * G].reshape(-1, G)
    for sbits in (0x0400, 0x1D1F, 0x2E66, 0x2000, 0x3555, ((30 - qmax) << 10) | 0x3FF):
        S = np.full((wb.shape[0], 1), sbits, dtype=np.uint16)
        codes, S2 = oracle.quantize(wb, bits, G, oracle.RULE_GIVEN, S)
        assert np.array_equal(S2, S)
        step = 5 if bits != 3 else 1
        flat_w, flat_c = wb.ravel()[::step], codes.ravel()[::step]
        for w, c in zip(flat_w.tolist(), flat_c.tolist()):
            assert c & qmax == exact_exponent(w, sbits, qmax), (hex(w), hex(sbits))
            neg = (w >> 15) == 1 and (w & 0x7FFF) != 0
            assert (c >> (bits - 1)) == int(neg)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_threshold_neighbours_land_on_opposite_sides(oracle, bits):
    """The decision boundary between levels k and k+1 is |w| = S * sqrt(2) * 2^k (rounding is
    in the log domain, not nearest-value, whose boundary would be 1.5 * 2^k)."""
    qmax = QMAX[bits]
    for sbits in (0x2000, 0x2E66, 0x1D1F):
        s = float(f16_fraction(sbits))
        for k in range(qmax):
            t = s * np.sqrt(2.0) * 2.0 ** k
            below = np.float16(t)
            if float(below) > t:
                below = np.nextafter(below, np.float16(0))
            above = np.nextafter(below, np.float16(np.inf))
            assert float(below) < t < float(above)
            wb = np.zeros((1, 64), dtype=np.uint16)
            wb[0, 0] = below.view(np.uint16)
            wb[0, 1] = above.view(np.uint16)
            codes, _ = oracle.quantize(wb, bits, 64, oracle.RULE_GIVEN, np.array([[sbits]], dtype=np.uint16))
            assert codes[0, 0] == k and codes[0, 1] == k + 1


def test_toy_group_fixture(oracle):
    rows = {}
    for row in _golden_rows("toy_group.txt"):
        key, *vals = row.split()
        rows[key] = vals
    w = np.array([int(v, 16) for v in rows["w_bits"]], dtype=np.uint16).reshape(1, 8)
    codes, S = oracle.quantize(w, 3, 8, oracle.RULE_TOP)
    assert S[0, 0] == int(rows["scale"][0], 16)
    assert codes[0].tolist() == [int(v) for v in rows["codes"]]
    packed = oracle.pack(codes, 3)
    assert packed[0].tolist() == [int(v, 16) for v in rows["packed"]]
    out, rounded = oracle.dequant(packed, S, 8, 3, 8)
    assert rounded == 0
    assert out[0].tolist() == [int(v, 16) for v in rows["dequant"]]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("rule", [0, 1])
@pytest.mark.parametrize("dist", ["normal", "t5"])
def test_quantizer_invariants(oracle, bits, rule, dist):
    qmax = QMAX[bits]
    G, N, K = 128, 64, 1024
    rng = synth.rng_for(0, bits * 10 + rule)
    W = synth.weights(rng, N, K, dist)
    codes, S = oracle.quantize(W, bits, G, rule)
    E = (codes & qmax).astype(np.int64)
    sign = codes >> (bits - 1)
    w = synth.f16_bits_to_f64(W)
    # scales: legal range; rule TOP: S * 2^q_max == max|w| exactly whenever that is representable
    assert all(oracle.clamp_scale_bits(int(s), bits) == int(s) for s in S.ravel()[::17])
    amax = np.abs(w).reshape(N, K // G, G).max(-1)
    s = synth.f16_bits_to_f64(S)
    if rule == 0:
        assert np.array_equal(s * 2.0 ** qmax, amax)
        # the largest element sits on the top level and is reconstructed exactly
        top = np.abs(w).reshape(N, K // G, G).argmax(-1)
        Eg = E.reshape(N, K // G, G)
        assert np.all(np.take_along_axis(Eg, top[..., None], -1) == qmax)
    else:
        # Algorithm 1's s0 = max|w| / (2^q_max - 1), rounded once to FP16 (numpy's rounding as the reference)
        ref = (amax / (2.0 ** qmax - 1)).astype(np.float16).astype(np.float64)
        assert np.array_equal(s, ref)
    # sign = [w < 0]; exponent is monotone in |w| inside each group
    assert np.array_equal(sign.astype(bool), w < 0)
    aw = np.abs(w).reshape(-1, G)
    Eg = E.reshape(-1, G)
    order = np.argsort(aw, axis=1, kind="stable")
    assert np.all(np.diff(np.take_along_axis(Eg, order, 1), axis=1) >= 0)
    # requantizing the reconstruction with the same scales returns the same codes
    packed = oracle.pack(codes, bits)
    deq, rounded = oracle.dequant(packed, S, K, bits, G)
    assert rounded == 0
    codes2, _ = oracle.quantize(deq, bits, G, oracle.RULE_GIVEN, S)
    assert np.array_equal(codes2, codes)
    # |w~| / S is exactly a power of two 2^E (the format has no zero level)
    ratio = np.abs(synth.f16_bits_to_f64(deq)) / np.repeat(s, G, axis=1)
    assert np.array_equal(ratio, 2.0 ** E)


def test_quantizer_zero_group_and_signed_zero(oracle):
    W = np.zeros((1, 128), dtype=np.uint16)
    W[0, 3] = 0x8000  # -0
    for bits in (2, 3, 4):
        codes, S = oracle.quantize(W, bits, 128, oracle.RULE_TOP)
        assert S[0, 0] == 0x0400 and not codes.any()
    W[0, 5] = 0x7C00  # inf is rejected
    with pytest.raises(ValueError):
        oracle.quantize(W, 3, 128, oracle.RULE_TOP)


def test_quantizer_rejects_illegal_given_scale(oracle):
    W = np.full((1, 64), 0x2000, dtype=np.uint16)
    for bad in (0x0000, 0x03FF, 0x7000):  # zero, subnormal, too large for q_max = 3
        with pytest.raises(ValueError):
            oracle.quantize(W, 3, 64, oracle.RULE_GIVEN, np.array([[bad]], dtype=np.uint16))


# ----------------------------------------------------------------- packing
def test_packing_fixture_and_roundtrip(oracle):
    for row in _golden_rows("packing_example.txt"):
        n, codes, bytes_ = [p.strip() for p in row.split("|")]
        n = int(n)
        c = np.array([int(v) for v in codes.split()], dtype=np.uint8).reshape(1, -1)
        expect = [int(v, 16) for v in bytes_.split()]
        assert oracle.pack(c, n)[0].tolist() == expect
        assert np.array_equal(oracle.unpack(np.array([expect], dtype=np.uint8), c.shape[1], n), c)
    rng = np.random.default_rng(3)
    for bits in (2, 3, 4):
        c = rng.integers(0, 1 << bits, (5, 256)).astype(np.uint8)
        p = oracle.pack(c, bits)
        assert p.shape == (5, 256 * bits // 8)
        assert np.array_equal(oracle.unpack(p, 256, bits), c)
        # independent unpack: the row as one big little-endian integer
        for i in range(5):
            big = int.from_bytes(p[i].tobytes(), "little")
            assert [(big >> (bits * k)) & ((1 << bits) - 1) for k in range(256)] == c[i].tolist()


# ----------------------------------------------------------------- Eq. 1
def test_dequant_golden_vectors(oracle):
    for row in _golden_rows("pot_dequant_vectors.txt"):
        n, sb, code, expect = row.split()
        n = int(n)
        c = np.zeros((1, 8), dtype=np.uint8)
        c[0, 0] = int(code, 2)
        out, rounded = oracle.dequant(oracle.pack(c, n), np.array([[int(sb, 16)]], dtype=np.uint16), 8, n, 8)
        assert rounded == 0 and out[0, 0] == int(expect, 16), row
    for row in _golden_rows("pot_bf16_vectors.txt"):
        n, sb, code, expect = row.split()
        n = int(n)
        c = np.zeros((1, 8), dtype=np.uint8)
        c[0, 0] = int(code, 2)
        out, rounded = oracle.dequant(oracle.pack(c, n), np.array([[int(sb, 16)]], dtype=np.uint16), 8, n, 8, oracle.BF16)
        assert rounded == 0 and out[0, 0] == int(expect, 16), row


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_dequant_every_code_every_legal_scale(oracle, bits):
    """Brute force: every code x every legal FP16 scale.  Two independent routes must agree with
    the oracle's FP64 evaluation of Eq. 1: (a) exact rational arithmetic, (b) the integer route
    of Sec. 4.2 -- move the sign to bit 15, shift the exponent to bit 10, integer-add to the
    scale's bit pattern."""
    qmax = QMAX[bits]
    ncodes = 1 << bits
    scales = np.arange(0x0400, (((30 - qmax) << 10) | 0x3FF) + 1, dtype=np.uint32).astype(np.uint16)
    assert scales.size == (30 - qmax) * 1024
    G = 16  # one group per row, the codes 0..2^n-1 (repeated) in each
    codes = np.tile(np.arange(G, dtype=np.uint8) % ncodes, (scales.size, 1))
    out, rounded = oracle.dequant(oracle.pack(codes, bits), scales.reshape(-1, 1), G, bits, G)
    assert rounded == 0
    sign = (codes >> (bits - 1)).astype(np.uint32)
    E = (codes & qmax).astype(np.uint32)
    integer_route = ((scales.reshape(-1, 1).astype(np.uint32) + (E << 10)) | (sign << 15)).astype(np.uint16)
    assert np.array_equal(out, integer_route)
    for r in range(0, scales.size, 53):  # exact rational check on a stride of the scales, all codes
        S = f16_fraction(int(scales[r]))
        for c in range(ncodes):
            val = S * (1 << (c & qmax)) * (-1 if c >> (bits - 1) else 1)
            assert f16_fraction(int(out[r, c])) == val


def test_dequant_bf16_equals_rounding_the_product(oracle):
    """2^E * bf16(S) == bf16(2^E * S): scaling by a power of two commutes with rounding (no
    overflow or underflow in BF16's range), checked against torch's cast."""
    import torch
    rng = np.random.default_rng(5)
    bits, G = 4, 16
    scales = rng.integers(0x0400, ((30 - 7) << 10) | 0x3FF, 4096).astype(np.uint16)
    codes = np.tile(np.arange(16, dtype=np.uint8), (scales.size, 1))
    out, rounded = oracle.dequant(oracle.pack(codes, bits), scales.reshape(-1, 1), G, bits, G, oracle.BF16)
    assert rounded == 0
    s = scales.view(np.float16).astype(np.float32).reshape(-1, 1)
    val = s * (2.0 ** (codes & 7)).astype(np.float32) * np.where(codes >> 3, -1.0, 1.0).astype(np.float32)
    ref = torch.from_numpy(val).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(out, ref)


def test_dequant_reports_out_of_contract_scales(oracle):
    # a subnormal scale times 2^E is still exact in FP16, but too large a scale overflows: flagged
    c = np.full((1, 8), 3, dtype=np.uint8)
    _, rounded = oracle.dequant(oracle.pack(c, 3), np.array([[0x7400]], dtype=np.uint16), 8, 3, 8)
    assert rounded == 8
