"""Pins for the oracle's own FP16 / BF16 conversions (Sec. 4.1 field layout).

Independent references: numpy's float16 (a separate implementation), exact rational
arithmetic (fractions.Fraction), torch's bfloat16 cast, and hand-derived bit patterns."""
from fractions import Fraction
from pathlib import Path

import numpy as np
import torch

GOLD = Path(__file__).parent / "golden"


def _golden_rows(name):
    for line in (GOLD / name).read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            yield line


def f16_fraction(bits: int) -> Fraction:
    """Exact value of a finite FP16 pattern from its fields (Sec. 4.1)."""
    s, e, m = bits >> 15, (bits >> 10) & 31, bits & 1023
    v = Fraction(m, 1 << 24) if e == 0 else Fraction(1024 + m, 1024) * Fraction(2) ** (e - 15)
    return -v if s else v


def test_f16_golden_patterns(oracle):
    for row in _golden_rows("fp16_fields.txt"):
        expr, bits = row.split()
        v = float(eval(expr))
        assert oracle.f16_to_f64(int(bits, 16)) == v
        assert oracle.f64_to_f16(v) == (int(bits, 16), False)


def test_f16_to_f64_all_patterns_match_numpy(oracle):
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = allbits.view(np.float16).astype(np.float64)
    got = np.array([oracle.f16_to_f64(int(b)) for b in allbits])
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin], ref[fin])
    assert np.array_equal(np.signbit(got[fin]), np.signbit(ref[fin]))
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isinf(got), np.isinf(ref))


def test_f16_to_f64_exact_rational(oracle):
    for bits in list(range(0, 0x7C00, 97)) + [0x0001, 0x03FF, 0x0400, 0x7BFF, 0x8001, 0xFBFF]:
        assert Fraction(oracle.f16_to_f64(bits)) == f16_fraction(bits)


def test_f64_to_f16_roundtrip_and_ties(oracle):
    # every finite pattern converts back to itself, exactly
    for bits in range(0, 0x7C00, 7):
        v = oracle.f16_to_f64(bits)
        assert oracle.f64_to_f16(v) == (bits, False)
        assert oracle.f64_to_f16(-v)[0] == (bits | 0x8000)
    # exact midpoints between neighbours go to the even mantissa; just off the midpoint goes to the nearer
    for bits in list(range(0, 0x7BFF, 131)) + [0x03FF, 0x0400, 0x3BFF]:
        lo, hi = oracle.f16_to_f64(bits), oracle.f16_to_f64(bits + 1)
        mid = (lo + hi) / 2  # exact in FP64
        even = bits if bits % 2 == 0 else bits + 1
        assert oracle.f64_to_f16(mid) == (even, True)
        assert oracle.f64_to_f16(np.nextafter(mid, 0.0)) == (bits, True)
        assert oracle.f64_to_f16(np.nextafter(mid, 1e9)) == (bits + 1, True)
    # overflow: the midpoint between 65504 and 65536 rounds to infinity, just below stays finite
    assert oracle.f64_to_f16(65520.0)[0] == 0x7C00
    assert oracle.f64_to_f16(np.nextafter(65520.0, 0.0))[0] == 0x7BFF


def test_f64_to_f16_random_matches_numpy(oracle):
    rng = np.random.default_rng(7)
    vals = np.concatenate([rng.standard_normal(20000) * 0.02, rng.standard_normal(5000) * 100.0,
                           rng.standard_normal(5000) * 1e-6, rng.uniform(-7e4, 7e4, 2000)])
    ref = vals.astype(np.float16).view(np.uint16)
    got = np.array([oracle.f64_to_f16(float(v))[0] for v in vals], dtype=np.uint16)
    assert np.array_equal(got, ref)


def test_bf16_conversions_match_torch(oracle):
    rng = np.random.default_rng(11)
    # FP16-representable inputs (what the path converts) plus general doubles
    h = rng.integers(0x0400, 0x7C00, 20000).astype(np.uint16).view(np.float16).astype(np.float64)
    vals = np.concatenate([h, -h[:1000], rng.standard_normal(5000) * 3.0, [0.0, 1.0, 2.0 ** -126, 2.0 ** -133, 3.0e38]])
    t = torch.from_numpy(vals.astype(np.float32)).to(torch.bfloat16)
    ref = t.view(torch.int16).numpy().view(np.uint16)
    # torch rounds float32 -> bf16; the inputs above are exactly representable in float32 or are
    # re-rounded identically only when float32 conversion is exact, so restrict to those
    exact32 = vals.astype(np.float32).astype(np.float64) == vals
    got = np.array([oracle.f64_to_bf16(float(v))[0] for v in vals], dtype=np.uint16)
    assert exact32.sum() > 20000
    assert np.array_equal(got[exact32], ref[exact32])
    back = t.to(torch.float64).numpy()
    got_back = np.array([oracle.bf16_to_f64(int(b)) for b in ref])
    assert np.array_equal(got_back[exact32], back[exact32])


def test_scale_clamp_range(oracle):
    # legal scales: normal, exponent field e with 1 <= e and e + q_max <= 30
    for n, qmax in ((2, 1), (3, 3), (4, 7)):
        hi = ((30 - qmax) << 10) | 0x3FF
        assert oracle.clamp_scale_bits(0x0000, n) == 0x0400
        assert oracle.clamp_scale_bits(0x03FF, n) == 0x0400
        assert oracle.clamp_scale_bits(0x0400, n) == 0x0400
        assert oracle.clamp_scale_bits(hi, n) == hi
        assert oracle.clamp_scale_bits(hi + 1, n) == hi
        assert oracle.clamp_scale_bits(0x7BFF, n) == hi
        # the largest legal scale times the top level is still finite
        assert f16_fraction(hi) * 2 ** qmax <= f16_fraction(0x7BFF)
        assert f16_fraction(hi + 1) * 2 ** qmax > f16_fraction(0x7BFF)
