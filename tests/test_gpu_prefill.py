"""GPU parity: the tcgen05 GEMM (tiled layout, M > 8) against the FP64 oracle."""
import numpy as np
import pytest

from paper_2507_11959_b200 import synth
from tests.gpu_util import PotCase, bits_of, f16_dev, gate

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from tests.gpu_util import GuardedBinding
    return GuardedBinding()  # outputs and workspaces between canary pads, checked after every call


# (M, N, K).  M <= 64 runs the one-token-tile variant (eight stages, a TMA box of exactly M rows, two TMA threads), larger
# M the 256-token tiles: one exact tile; ragged M and N with several K blocks; several tiles in both directions;
# (300, ...) and (20, ...) run split-K; 129 tokens = a second token tile that holds one token; 64 / 65 tokens = either
# side of the variant boundary; K = 1152 / 2048 = more K blocks than pipeline stages; K = 128 = a single stage (one-tile
# kernel) or two (256-token kernel); 896 = seven column blocks, one more than the one-tile kernel's six stages
SHAPES = [(128, 128, 128), (200, 144, 384), (33, 16, 256), (300, 272, 1152), (20, 256, 4096), (129, 144, 640),
          (64, 272, 1152), (9, 48, 2048), (65, 160, 1152), (17, 32, 128), (70, 16, 128), (48, 400, 896)]


@pytest.fixture(params=["smem", "tmem", "tmem-narrow"])
def weight_tile(request, monkeypatch):
    """The tcgen05 kernels keep the decoded weight tile in tensor memory (the default: a single wave of CTAs then runs
    128-column stages; "tmem-narrow" keeps the 64-column stages that larger launches use) or in shared memory: the parity
    tests run all three through the library's diagnostic switch."""
    monkeypatch.setenv("POT_PREFILL_WEIGHT_TILE", request.param)
    return request.param


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [64, 128])
def test_prefill_gemm_matches_oracle(B, oracle, bits, G, weight_tile):
    for i, (M, N, K) in enumerate(SHAPES):
        c = PotCase(N, K, bits, G, dist="normal", sigma=0.015, seed=(5, 10 * bits + i))
        X = synth.activations(synth.rng_for(5, 100 + i), M, K, outliers=(i % 2 == 1))
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
        Yg = B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X), B.TILED)
        assert B.pot_debug_errors() == (0, 0, 0)
        ok, worst, tight = gate(bits_of(Yg), Y, A)
        assert ok and tight < 4.0, (M, N, K, worst, tight)


def test_split_k_workspace_is_reusable(B, oracle, weight_tile):
    """Few tiles and a deep K: the kernel splits K (8 ways here), adds the splits in a fixed order and leaves its
    arrival counters at zero -- two calls on one workspace give the same bits, equal to the oracle within the gate."""
    bits, G, M, N, K = 3, 128, 40, 384, 4096
    c = PotCase(N, K, bits, G, dist="t5", seed=(5, 77))
    X = synth.activations(synth.rng_for(5, 177), M, K, outliers=True)
    Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
    need = B.pot_gemm_workspace_bytes(M, N, K, bits, G)
    assert need > 0
    ws = B.new_workspace(need)
    dX = f16_dev(X)
    y1 = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, dX, B.TILED, workspace=ws))
    y2 = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, dX, B.TILED, workspace=ws))
    assert B.pot_debug_errors() == (0, 0, 0)
    assert np.array_equal(y1, y2)
    ok, worst, tight = gate(y1, Y, A)
    assert ok and tight < 4.0, (worst, tight)


def test_two_issuers_give_the_same_bits_every_time(B, oracle, weight_tile):
    """The two MMA issuers accumulate into separate accumulators (alternate K blocks, added by the epilogue in a fixed
    order; or, with the weight tile in tensor memory, one token tile each): nothing in the result may depend on which of
    them ran first."""
    bits, G, M, N, K = 3, 128, 300, 272, 2304
    c = PotCase(N, K, bits, G, dist="t5", seed=(5, 88))
    dX = f16_dev(synth.activations(synth.rng_for(5, 188), M, K, outliers=True))
    ws = B.new_workspace(B.pot_gemm_workspace_bytes(M, N, K, bits, G))
    y0 = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, dX, B.TILED, workspace=ws))
    for _ in range(4):
        assert np.array_equal(bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, dX, B.TILED, workspace=ws)), y0)
    assert B.pot_debug_errors() == (0, 0, 0)


@pytest.mark.parametrize("bits", [3])
def test_prefill_one_hot_tokens_return_dequantized_columns(B, oracle, bits, weight_tile):
    """token t = e_{k_t}: row t of Y must equal column k_t of the dequantized matrix bit for bit."""
    G, N, K, M = 128, 256, 640, 160
    c = PotCase(N, K, bits, G, dist="normal", seed=(5, 60))
    deq, _ = oracle.dequant(c.packed, c.S, K, bits, G)
    ks = (np.arange(M) * 37 + 5) % K
    X = np.zeros((M, K), dtype=np.uint16)
    X[np.arange(M), ks] = 0x3C00
    Yg = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X), B.TILED))
    assert np.array_equal(Yg, deq[:, ks].T)


def test_prefill_config5_shape_sampled(B, oracle):
    """Llama-2-70B-shaped projection at the benchmarked size, checked on sampled output columns."""
    bits, G, M, N, K = 3, 128, 2048, 10240, 8192
    c = PotCase(N, K, bits, G, dist="normal", sigma=0.015, seed=(5, 70))
    X = synth.activations(synth.rng_for(5, 71), M, K, outliers=False)
    Yg = bits_of(B.pot_gemm(c.tiled(), c.tiled_S(), K, bits, G, f16_dev(X), B.TILED))
    assert B.pot_debug_errors() == (0, 0, 0)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, N - 129, N - 128, N - 1],
                                     synth.rng_for(5, 72).integers(0, N, 24)])).astype(np.int64)
    Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X, rows)
    ok, worst, tight = gate(Yg[:, rows], Y, A)
    assert ok and tight < 4.0, (worst, tight)
