"""pot_gemv_chain_*: a list of dependent GEMVs in one persistent kernel must reproduce pot_gemv bit for bit."""
import numpy as np
import pytest
import torch

from paper_2507_11959_b200 import synth
from tests.gpu_util import PotCase, bits_of, f16_dev, gate

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_11959_b200 import binding
    binding.lib()
    return binding


def _ws(B, N, K, bits, G):
    return B.new_workspace(B.pot_gemv_workspace_bytes(N, K, bits, G))


@pytest.mark.parametrize("bits,G", [(3, 128), (2, 64), (4, 128)])
def test_dependent_chain_equals_sequential_gemvs(B, oracle, bits, G):
    """y of each operation is the x of the next: 640 -> 256 -> 1152 -> 4096 -> 384 (several steps per row block,
    row blocks shared between CTAs, ragged last step)."""
    dims = [640, 256, 1152, 4096, 384]
    cases = [PotCase(dims[i + 1], dims[i], bits, G, dist="normal", sigma=0.05, seed=(6, 10 * bits + i)) for i in range(4)]
    x0 = f16_dev(synth.activations(synth.rng_for(6, 50 + bits), 1, dims[0])[0])
    # sequential reference through pot_gemv
    xs, ref = x0, []
    for c, n, k in zip(cases, dims[1:], dims[:-1]):
        xs = B.pot_gemv(c.tiled(), c.d_S, k, bits, G, xs, B.TILED, workspace=_ws(B, n, k, bits, G))
        ref.append(bits_of(xs))
    # the same list in one kernel
    ys = [torch.zeros(n, dtype=torch.float16, device="cuda") for n in dims[1:]]
    ops, x = [], x0
    for c, n, k, y in zip(cases, dims[1:], dims[:-1], ys):
        ops.append((c.tiled(), c.d_S, k, G, x, y, _ws(B, n, k, bits, G)))
        x = y
    scratch = B.pot_gemv_chain_prepare(ops, bits)
    for _ in range(3):  # the counters in scratch and in the workspaces are left ready for the next run
        for y in ys:
            y.zero_()
        B.pot_gemv_chain_run(scratch, len(ops), bits)
        torch.cuda.synchronize()
        assert B.pot_debug_errors() == (0, 0, 0)
        for y, r in zip(ys, ref):
            assert np.array_equal(bits_of(y), r)
    # and the first link against the oracle
    Y, A = oracle.matmul(cases[0].packed, cases[0].S, dims[0], bits, G, bits_of(x0).reshape(1, -1))
    ok, worst, tight = gate(ref[0], Y[0], A[0])
    assert ok and tight < 4.0, (worst, tight)


def test_chain_of_llama_layer_shapes_equals_gemv(B):
    """The five projections of a Llama-2-7B layer, twice (ten operations sharing five workspaces)."""
    bits, G = 3, 128
    ops, refs, keep = [], [], []
    for rep in range(2):
        for i, pr in enumerate(synth.LLAMA2_7B):
            W = f16_dev(synth.weights(synth.rng_for(6, 100 + i), pr.N, pr.K, "t5"))
            packed, S = B.pot_quantize_ref(W, bits, G, B.SCALE_TOP)
            tiled = B.pot_repack(packed, pr.K, bits, 0)
            x = f16_dev(synth.activations(synth.rng_for(6, 200 + i), 1, pr.K)[0])
            y = torch.zeros(pr.N, dtype=torch.float16, device="cuda")
            ws = keep[i][2] if rep else _ws(B, pr.N, pr.K, bits, G)
            if not rep:
                keep.append((tiled, S, ws))
            refs.append(bits_of(B.pot_gemv(tiled, S, pr.K, bits, G, x, B.TILED, workspace=_ws(B, pr.N, pr.K, bits, G))))
            ops.append((tiled, S, pr.K, G, x, y, ws))
            del W, packed
    scratch = B.pot_gemv_chain_prepare(ops, bits)
    B.pot_gemv_chain_run(scratch, len(ops), bits)
    torch.cuda.synchronize()
    assert B.pot_debug_errors() == (0, 0, 0)
    for op, r in zip(ops, refs):
        assert np.array_equal(bits_of(op[5]), r)


def test_chain_argument_errors(B):
    c = PotCase(64, 256, 3, 128, seed=(6, 300))
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    y = torch.zeros(64, dtype=torch.float16, device="cuda")
    with pytest.raises(B.PotError):  # K % 128 != 0
        B.pot_gemv_chain_prepare([(c.tiled(), c.d_S, 200, 128, x, y, None)], 3)
    with pytest.raises(B.PotError):  # missing workspace for a shape that splits K
        big = torch.zeros(4096 * 11008 * 3 // 8, dtype=torch.uint8, device="cuda")
        S = torch.zeros((4096, 86), dtype=torch.float16, device="cuda")
        B.pot_gemv_chain_prepare([(big.view(4096, -1), S, 11008, 128, torch.zeros(11008, dtype=torch.float16, device="cuda"),
                                   torch.zeros(4096, dtype=torch.float16, device="cuda"), None)], 3)
