"""GPU parity: quantizer, repack and the standalone dequantization kernels against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

from tests.gpu_util import PotCase, UintCase, bits_of, f16_dev, to_dev

pytestmark = pytest.mark.gpu

SHAPES = [(1, 128), (3, 384), (37, 1152), (256, 4096), (130, 2176)]  # several tiles + ragged tails


@pytest.fixture(scope="module")
def B():
    from tests.gpu_util import GuardedBinding
    return GuardedBinding()  # outputs and workspaces between canary pads, checked after every call


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
@pytest.mark.parametrize("rule", [0, 1])
def test_quantize_ref_bit_exact(B, oracle, bits, G, rule):
    for i, (N, K) in enumerate(SHAPES):
        c = PotCase(N, K, bits, G, dist="t5" if i % 2 else "normal", rule=rule, seed=(3, 10 * bits + i))
        packed, S = B.pot_quantize_ref(f16_dev(c.W_bits), bits, G, rule)
        assert np.array_equal(bits_of(S), c.S)
        assert np.array_equal(packed.cpu().numpy(), c.packed)
        assert int(B.pot_validate_scales(S, bits).item()) == 0


def test_quantize_ref_given_scales_and_edge_values(B, oracle):
    bits, G, N, K = 3, 128, 8, 256
    W = np.zeros((N, K), dtype=np.uint16)
    W[0, :] = 0x8000                  # all -0: scale clamps to 2^-14, every code 0
    W[1, ::2] = 0x7BFF                # largest finite FP16
    W[1, 1::2] = 0xFBFF
    W[2, :] = 0x0001                  # smallest subnormal
    W[3, :64] = 0x3C00
    W[4:] = np.random.default_rng(0).integers(0, 0x7C00, (4, K)).astype(np.uint16)
    for rule in (0, 1):
        codes, S = oracle.quantize(W, bits, G, rule)
        packed, Sg = B.pot_quantize_ref(f16_dev(W), bits, G, rule)
        assert np.array_equal(bits_of(Sg), S) and np.array_equal(packed.cpu().numpy(), oracle.pack(codes, bits))
    S = np.full((N, K // G), 0x2E66, dtype=np.uint16)
    codes, _ = oracle.quantize(W, bits, G, oracle.RULE_GIVEN, S)
    packed, Sg = B.pot_quantize_ref(f16_dev(W), bits, G, B.SCALE_GIVEN, f16_dev(S))
    assert np.array_equal(packed.cpu().numpy(), oracle.pack(codes, bits)) and np.array_equal(bits_of(Sg), S)


def test_validate_scales_counts_illegal_entries(B):
    S = np.array([0x0000, 0x03FF, 0x0400, 0x2E66, 0x6FFF, 0x7000, 0x7BFF, 0x7C00] * 5, dtype=np.uint16)
    assert int(B.pot_validate_scales(f16_dev(S), 3).item()) == 5 * 5   # zero, subnormal, 3 too large for q_max = 3
    assert int(B.pot_validate_scales(f16_dev(S), 2).item()) == 5 * 4   # q_max = 1: 0x7000 (field 28) is legal


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_scale_search_rule_matches_algorithm_1(B, oracle, bits):
    from paper_2507_11959_b200 import synth
    G, N, K = 128, 96, 2048
    W = synth.weights(synth.rng_for(3, 70 + bits), N, K, "normal" if bits != 3 else "t5")
    S_ref, bstar = oracle.scale_search(W, bits, G)
    packed, S = B.pot_quantize_ref(f16_dev(W), bits, G, B.SCALE_SEARCH)
    Sg = bits_of(S)
    # both sides add the 128 squared errors of a candidate in the same order with the same FP64 roundings, so the
    # argmin -- index work -- must agree for every group, not just for most
    assert np.array_equal(Sg, S_ref), np.argwhere(Sg != S_ref)[:5]
    codes, _ = oracle.quantize(W, bits, G, oracle.RULE_GIVEN, Sg)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack(codes, bits))


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
@pytest.mark.parametrize("dtype", [0, 1])
def test_pot_dequant_bit_exact(B, oracle, bits, G, dtype):
    for i, (N, K) in enumerate(SHAPES):
        c = PotCase(N, K, bits, G, dist="t5" if i % 2 else "normal", seed=(3, 100 + 10 * bits + i))
        ref, rounded = oracle.dequant(c.packed, c.S, K, bits, G, dtype)
        assert rounded == 0
        out = B.pot_dequant(c.d_packed, c.d_S, K, bits, G, dtype)
        assert out.dtype == (torch.float16 if dtype == 0 else torch.bfloat16)
        assert np.array_equal(bits_of(out), ref), (N, K)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_pot_dequant_every_code_and_extreme_scales(B, oracle, bits):
    qmax = (1 << (bits - 1)) - 1
    hi = ((30 - qmax) << 10) | 0x3FF
    scales = np.array([0x0400, 0x0401, 0x2000, 0x2E66, 0x3555, 0x3BFF, 0x3C00, hi - 1, hi], dtype=np.uint16)
    G, K = 64, 128
    codes = np.tile(np.arange(K, dtype=np.uint8) % (1 << bits), (scales.size, 1))
    S = np.stack([scales, scales[::-1]], axis=1).copy()
    packed = oracle.pack(codes, bits)
    for dtype in (0, 1):
        ref, rounded = oracle.dequant(packed, S, K, bits, G, dtype)
        assert rounded == 0
        out = B.pot_dequant(to_dev(packed), f16_dev(S), K, bits, G, dtype)
        assert np.array_equal(bits_of(out), ref)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
def test_uint_quantize_and_dequant_bit_exact(B, oracle, bits, G):
    for i, (N, K) in enumerate(SHAPES):
        c = UintCase(N, K, bits, G, dist="t5" if i % 2 else "normal", seed=(3, 200 + 10 * bits + i))
        packed, S, Z = B.uint_quantize_ref(f16_dev(c.W_bits), bits, G)
        assert np.array_equal(bits_of(S), c.S) and np.array_equal(bits_of(Z), c.Z)
        assert np.array_equal(packed.cpu().numpy(), c.packed)
        ref = oracle.uint_dequant(c.packed, c.S, c.Z, K, bits, G)
        for kernel in (B.UINT_FAST, B.UINT_NAIVE):
            out = B.uint_dequant(c.d_packed, c.d_S, c.d_Z, K, bits, G, kernel)
            got = bits_of(out)
            # (q - z) = 0 may come out as +0 or -0 depending on the route; compare values there
            zero = (ref & 0x7FFF) == 0
            assert np.array_equal(got[~zero], ref[~zero]) and np.all((got[zero] & 0x7FFF) == 0), (N, K, kernel)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_repack_is_a_bijection(B, oracle, bits):
    N, K = 48, 640
    rng = np.random.default_rng(bits)
    packed = rng.integers(0, 256, (N, K * bits // 8)).astype(np.uint8)
    d = to_dev(packed)
    for repack in (B.pot_repack, B.uint_repack):
        tiled = repack(d, K, bits, 0)
        back = repack(tiled, K, bits, 1)
        assert np.array_equal(back.cpu().numpy(), packed)
        # same multiset of bits per 16x128 unit (size preserving, no padding)
        assert int(np.unpackbits(tiled.cpu().numpy()).sum()) == int(np.unpackbits(packed).sum())
        assert not np.array_equal(tiled.cpu().numpy(), packed)
    # the host-side layout map describes exactly what the device wrote
    tiled = B.pot_repack(d, K, bits, 0).cpu().numpy().view(np.uint32).ravel()
    codes = oracle.unpack(packed, K, bits)
    ncb, nw = K // 128, 4 * bits
    for (i, k) in [(0, 0), (5, 1), (17, 130), (47, 639), (33, 511), (16, 256)]:
        rb, r, cb, q = i // 16, i % 16, k // 128, k % 128
        for b in range(bits):
            w, bit = B.pot_layout_bit(bits, 0, q, b)
            idx = (rb * ncb + cb) * 16 * nw + (w >> 2) * 64 + r * 4 + (w & 3)
            assert (int(tiled[idx]) >> bit) & 1 == (int(codes[i, k]) >> b) & 1
