"""pot_gemv_noalloc: the split-K GEMV whose scratch is an array inside the library, for callers that
are not allowed to allocate device memory (see include/pot.h).  Collected last on purpose: if it
fails, a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from tests.gpu_util import PotCase, bits_of, f16_dev, gate

pytestmark = pytest.mark.gpu


def test_noalloc_gemv_matches_workspace_gemv_twice_in_a_row(oracle):
    from paper_2507_11959_b200 import binding as B
    from paper_2507_11959_b200 import synth
    bits, G, N, K = 3, 128, 1024, 11008          # short and wide: the kernel splits K and needs scratch
    need = B.pot_gemv_workspace_bytes(N, K, bits, G)
    assert 0 < need <= B.pot_gemv_noalloc_max_scratch_bytes()
    c = PotCase(N, K, bits, G, dist="t5", seed=(6, 1))
    tiled, tiled_S = c.tiled(), c.tiled_S()
    Y, A = None, None
    for call in range(2):  # second call finds the first call's leftovers in the shared array
        X = synth.activations(synth.rng_for(6, 10 + call), 1, K)
        x = f16_dev(X[0])
        ref = B.pot_gemv(tiled, tiled_S, K, bits, G, x, B.TILED)            # existing entry, caller workspace
        y = torch.empty(N, dtype=torch.float16, device="cuda")
        B.pot_gemv_noalloc(tiled, tiled_S, K, bits, G, x, y)                 # new entry, built-in scratch
        torch.cuda.synchronize()
        assert np.array_equal(bits_of(y), bits_of(ref)), f"call {call}"   # same kernel, same summation order
        Y, A = oracle.matmul(c.packed, c.S, K, bits, G, X)
        ok, worst, tight = gate(bits_of(y), Y[0], A[0])
        assert ok and tight < 4.0, (call, worst, tight)


def test_noalloc_gemv_rejects_shapes_beyond_its_scratch():
    from paper_2507_11959_b200 import binding as B
    bits, G, N, K = 3, 128, 262144, 11008
    assert B.pot_gemv_workspace_bytes(N, K, bits, G) > B.pot_gemv_noalloc_max_scratch_bytes()
    a = torch.zeros(16, dtype=torch.uint8, device="cuda")   # never read: the size check comes first
    fake_packed = torch.empty((N, 16), dtype=torch.uint8, device="cuda")  # only its row count is used
    before = B.pot_launch_count()
    with pytest.raises(B.PotError, match="workspace"):
        B.pot_gemv_noalloc(fake_packed, a, K, bits, G, a, a)
    assert B.pot_launch_count() == before
