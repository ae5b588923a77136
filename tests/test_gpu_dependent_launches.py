"""GPU: kernels launched behind one another in a stream (programmatic dependent launch: the next kernel starts while its
predecessor drains) must read the activations their predecessor WROTE, not what the buffer held before.  A dependent pair
(and a small-batch pair) is recorded in a CUDA graph and replayed with a different input every time; every replay is
compared with the same pair run one kernel at a time, and the first replays with the FP64 oracle."""
import numpy as np
import pytest
import torch

from paper_2507_11959_b200 import binding as B
from paper_2507_11959_b200 import synth
from tests.gpu_util import DEV, PotCase, bits_of, f16_dev, gate

pytestmark = pytest.mark.gpu


def _pair(bits, N, K):
    a = PotCase(K, K, bits, 128, dist="t5", seed=(8, bits))       # K -> K, its output feeds b
    b = PotCase(N, K, bits, 128, dist="t5", seed=(8, 10 + bits))  # K -> N
    return a, b


@pytest.mark.parametrize("bits", [2, 3])
def test_graph_replays_of_a_dependent_pair_follow_their_input(oracle, bits):
    N, K, G, R = 4096, 4096, 128, 12
    a, b = _pair(bits, N, K)
    Pa, Sa, Pb, Sb = a.tiled(), a.tiled_S(), b.tiled(), b.tiled_S()
    xs = [f16_dev(synth.activations(synth.rng_for(8, 100 + r), 1, K, outliers=(r % 2 == 1))[0]) for r in range(R)]
    wa = B.new_workspace(B.pot_gemv_workspace_bytes(K, K, bits, G), DEV)
    wb = B.new_workspace(B.pot_gemv_workspace_bytes(N, K, bits, G), DEV)
    x = torch.empty(K, dtype=torch.float16, device=DEV)
    mid = torch.empty(K, dtype=torch.float16, device=DEV)
    y = torch.empty(N, dtype=torch.float16, device=DEV)
    # one kernel at a time
    ref = []
    for r in range(R):
        B.pot_gemv(Pa, Sa, K, bits, G, xs[r], B.TILED, y=mid, workspace=wa)
        torch.cuda.synchronize()
        m = mid.clone()
        B.pot_gemv(Pb, Sb, K, bits, G, mid, B.TILED, y=y, workspace=wb)
        torch.cuda.synchronize()
        ref.append((m, y.clone()))
    # the first two against the oracle: A on x, then B on the FP16 result of A
    for r in range(2):
        Xa = bits_of(xs[r]).reshape(1, K)
        Y1, A1 = oracle.matmul(a.packed, a.S, K, bits, G, Xa)
        ok, worst, tight = gate(bits_of(ref[r][0]), Y1[0], A1[0])
        assert ok and tight < 4.0, (worst, tight)
        Y2, A2 = oracle.matmul(b.packed, b.S, K, bits, G, bits_of(ref[r][0]).reshape(1, K))
        ok, worst, tight = gate(bits_of(ref[r][1]), Y2[0], A2[0])
        assert ok and tight < 4.0, (worst, tight)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        B.pot_gemv(Pa, Sa, K, bits, G, x, B.TILED, y=mid, workspace=wa, stream=st)   # (loads the kernels before the capture)
        B.pot_gemv(Pb, Sb, K, bits, G, mid, B.TILED, y=y, workspace=wb, stream=st)
        st.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=st):
            B.pot_gemv(Pa, Sa, K, bits, G, x, B.TILED, y=mid, workspace=wa, stream=st)
            B.pot_gemv(Pb, Sb, K, bits, G, mid, B.TILED, y=y, workspace=wb, stream=st)
        for it in range(5 * R):
            r = (7 * it) % R
            x.copy_(xs[r])
            gr.replay()
            st.synchronize()
            assert torch.equal(mid, ref[r][0]) and torch.equal(y, ref[r][1]), (it, r)
    assert B.pot_debug_errors() == (0, 0, 0)


def test_eager_chain_without_synchronisation_follows_its_input(oracle):
    """the same through plain stream order, four dependent kernels deep, small batch included"""
    bits, G, K, R, M = 3, 128, 2048, 8, 4
    c = [PotCase(K, K, bits, G, dist="normal", seed=(8, 40 + i)) for i in range(4)]
    P = [(ci.tiled(), ci.tiled_S()) for ci in c]
    xs = [f16_dev(synth.activations(synth.rng_for(8, 200 + r), M, K)) for r in range(R)]
    ws = [B.new_workspace(B.pot_gemm_workspace_bytes(M, K, K, bits, G), DEV) for _ in range(4)]
    bufs = [torch.empty((M, K), dtype=torch.float16, device=DEV) for _ in range(4)]

    def chain(x, sync):
        cur = x
        for i in range(4):
            B.pot_gemm(P[i][0], P[i][1], K, bits, G, cur, B.TILED, Y=bufs[i], workspace=ws[i])
            if sync:
                torch.cuda.synchronize()
            cur = bufs[i]
        return bufs[3]

    ref = []
    for r in range(R):
        ref.append(chain(xs[r], True).clone())
    Y, A = oracle.matmul(c[0].packed, c[0].S, K, bits, G, bits_of(xs[0]))
    B.pot_gemm(P[0][0], P[0][1], K, bits, G, xs[0], B.TILED, Y=bufs[0], workspace=ws[0])
    ok, worst, tight = gate(bits_of(bufs[0]), Y, A)
    assert ok and tight < 4.0, (worst, tight)
    for it in range(6 * R):
        r = (5 * it) % R
        out = chain(xs[r], False)
        torch.cuda.synchronize()
        assert torch.equal(out, ref[r]), (it, r)
    assert B.pot_debug_errors() == (0, 0, 0)


def test_weights_written_just_before_the_gemv_are_complete(oracle):
    """The fused kernels fetch codes and scales before they wait for their predecessor, so the kernels that WRITE codes
    and scales must not let their successors start early: quantize -> repack -> repack_scales -> GEMV on one stream,
    nothing synchronised in between, new weights every time, against the same sequence run step by step."""
    bits, G, N, K, R = 3, 128, 4096, 4096, 6
    x = f16_dev(synth.activations(synth.rng_for(8, 300), 1, K)[0])
    ws = B.new_workspace(B.pot_gemv_workspace_bytes(N, K, bits, G), DEV)
    Ws = [f16_dev(synth.weights(synth.rng_for(8, 310 + r), N, K, "t5")) for r in range(R)]

    def run(W, sync):
        packed, S = B.pot_quantize_ref(W, bits, G, B.SCALE_TOP)
        if sync:
            torch.cuda.synchronize()
        tiled = B.pot_repack(packed, K, bits, 0)
        tS = B.pot_repack_scales(S, K, G, 0)
        if sync:
            torch.cuda.synchronize()
        y = B.pot_gemv(tiled, tS, K, bits, G, x, B.TILED, workspace=ws)
        torch.cuda.synchronize()
        return y, packed, S

    ref = [run(W, True) for W in Ws]
    Y, A = oracle.matmul(ref[0][1].cpu().numpy(), bits_of(ref[0][2]), K, bits, G, bits_of(x).reshape(1, K))
    ok, worst, tight = gate(bits_of(ref[0][0]), Y[0], A[0])
    assert ok and tight < 4.0, (worst, tight)
    for it in range(4 * R):
        r = (5 * it) % R
        y, _, _ = run(Ws[r], False)
        assert torch.equal(y, ref[r][0]), (it, r)
    assert B.pot_debug_errors() == (0, 0, 0)


@pytest.mark.parametrize("M", [16, 200])
def test_weights_written_just_before_the_tcgen05_gemm_are_complete(oracle, M):
    """The same for the tcgen05 kernels (one-tile and 256-token variants), whose producers fetch their first codes and
    scales even before the kernel's set-up."""
    bits, G, N, K, R = 3, 128, 1024, 2048, 4
    X = f16_dev(synth.activations(synth.rng_for(8, 400), M, K))
    ws = B.new_workspace(B.pot_gemm_workspace_bytes(M, N, K, bits, G), DEV)
    Ws = [f16_dev(synth.weights(synth.rng_for(8, 410 + r), N, K, "normal")) for r in range(R)]

    def run(W, sync):
        packed, S = B.pot_quantize_ref(W, bits, G, B.SCALE_TOP)
        if sync:
            torch.cuda.synchronize()
        tiled = B.pot_repack(packed, K, bits, 0)
        tS = B.pot_repack_scales(S, K, G, 0)
        if sync:
            torch.cuda.synchronize()
        Y = B.pot_gemm(tiled, tS, K, bits, G, X, B.TILED, workspace=ws)
        torch.cuda.synchronize()
        return Y, packed, S

    ref = [run(W, True) for W in Ws]
    Yo, A = oracle.matmul(ref[0][1].cpu().numpy(), bits_of(ref[0][2]), K, bits, G, bits_of(X))
    ok, worst, tight = gate(bits_of(ref[0][0]), Yo, A)
    assert ok and tight < 4.0, (worst, tight)
    for it in range(4 * R):
        r = (3 * it) % R
        Y, _, _ = run(Ws[r], False)
        assert torch.equal(Y, ref[r][0]), (it, r)
    assert B.pot_debug_errors() == (0, 0, 0)
