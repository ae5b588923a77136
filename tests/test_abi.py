"""The C-ABI library: builds, loads, exports what include/pot.h declares, validates arguments on
the host before touching the GPU, and its layout map is a bijection.  No kernel is launched."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def L():
    from paper_2507_11959_b200 import build
    build.build()
    from paper_2507_11959_b200 import binding
    return binding.lib()


def declared_functions():
    text = (ROOT / "include" / "pot.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:pot|uint)_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"pot_quantize_ref", "pot_dequant", "pot_gemv", "pot_gemm", "uint_dequant", "uint_gemv"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    from paper_2507_11959_b200 import binding
    assert set(binding.EXPORTS) == set(names)


def test_size_helpers(L):
    assert L.pot_packed_bytes(4096, 4096, 3) == 4096 * 1536
    assert L.pot_packed_bytes(4096, 4096, 2) == 4096 * 1024
    assert L.pot_packed_bytes(4096, 4100, 3) == 0       # K % 128
    assert L.pot_packed_bytes(4096, 4096, 5) == 0
    assert L.pot_scales_bytes(4096, 4096, 128) == 4096 * 32 * 2
    assert L.pot_scales_bytes(4096, 4096, 64) == 4096 * 64 * 2
    assert L.pot_scales_bytes(4096, 4096, 32) == 0
    # one unit (128 columns) per row block: every warp writes whole row blocks, nothing to combine; longer rows
    # need an arrival counter per row block and FP32 partial slots
    assert L.pot_gemv_workspace_bytes(12288, 128, 3, 128) == 0
    ws = L.pot_gemv_workspace_bytes(4096, 11008, 3, 128)
    assert ws >= 1024 + 256 * 2 * 16 * 4 and ws % 16 == 0
    wg = L.pot_gemm_workspace_bytes(4, 4096, 11008, 3, 128)   # small batch: eight token columns per slot
    assert wg >= 1024 + 256 * 2 * 16 * 8 * 4 and wg % 16 == 0
    # 2 to 8 tokens run the streaming kernel (one workspace size for all of them) while their activations fit in
    # shared memory; 5 to 8 tokens of a longer K run the tcgen05 kernel; one token runs the GEMV kernel
    assert L.pot_gemm_workspace_bytes(8, 12288, 4096, 3, 128) == L.pot_gemm_workspace_bytes(2, 12288, 4096, 3, 128)
    assert L.pot_gemm_workspace_bytes(2, 4096, 11008, 3, 128) == wg
    assert L.pot_gemm_workspace_bytes(8, 4096, 11008, 3, 128) == 256 + 32 * 4 * 8 * 128 * 4   # (see the tcgen05 sizes below)
    assert L.pot_gemm_workspace_bytes(1, 4096, 11008, 3, 128) >= ws
    # Larger M runs the tcgen05 kernel.  It needs scratch only for the tiles it splits along K: all of them when they
    # cover at most half of the SMs (32 tiles -> 4 splits of 32 token rows x 128 features), or those of a last
    # wave that fills at most half of the 148 CTA slots (640 tiles -> 48 tail tiles x 3 splits x 256 rows).
    assert L.pot_gemm_workspace_bytes(32, 4096, 11008, 3, 128) == 256 + 32 * 4 * 32 * 128 * 4
    assert L.pot_gemm_workspace_bytes(2048, 10240, 8192, 3, 128) == 256 + 48 * 3 * 256 * 128 * 4
    assert L.pot_gemm_workspace_bytes(2048, 8192, 28672, 3, 128) == 512 + 68 * 2 * 256 * 128 * 4  # 512 tiles: 68 in the last wave
    assert L.pot_gemm_workspace_bytes(2048, 3584, 8192, 3, 128) == 0     # 224 tiles: the last wave is 51 % full


def test_status_strings(L):
    seen = set()
    for code in range(8):
        s = L.pot_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert L.pot_status_string(99).decode() == "unknown status"


def test_argument_errors_are_reported_before_any_launch(L):
    before = L.pot_launch_count()
    a = ctypes.c_void_p(0x1000)      # never dereferenced: all of these fail validation on the host
    odd = ctypes.c_void_p(0x1008)
    null = ctypes.c_void_p(0)
    assert L.pot_dequant(null, a, 16, 128, 3, 128, 0, a, null) == 1
    assert L.pot_dequant(a, a, 16, 128, 5, 128, 0, a, null) == 2
    assert L.pot_dequant(a, a, 16, 128, 3, 32, 0, a, null) == 2
    assert L.pot_dequant(a, a, 16, 128, 3, 128, 7, a, null) == 2
    assert L.pot_dequant(a, a, 16, 100, 3, 128, 0, a, null) == 3
    assert L.pot_dequant(a, a, 0, 128, 3, 128, 0, a, null) == 3
    assert L.pot_dequant(a, a, 16, 128, 3, 128, 0, odd, null) == 4
    assert L.pot_gemv(a, a, 24, 128, 3, 128, 1, a, a, null, 0, null) == 3     # tiled needs N % 16 == 0
    assert L.pot_gemv(a, a, 4096, 11008, 3, 128, 1, a, a, null, 0, null) == 5  # split-K without workspace
    assert L.pot_gemv(a, a, 4096, 11008, 3, 128, 1, a, a, a, 64, null) == 5    # workspace too small
    assert L.pot_gemv(a, a, 16, 128, 3, 128, 9, a, a, null, 0, null) == 2
    assert L.pot_gemm(a, a, 16, 128, 3, 128, 0, a, 0, a, null, 0, null) == 3
    assert L.pot_gemm(a, null, 16, 128, 3, 128, 0, a, 4, a, null, 0, null) == 1
    assert L.pot_quantize_ref(a, 16, 128, 3, 128, 9, a, a, null) == 2
    assert L.pot_repack(a, a, 24, 128, 3, 0, null) == 3
    assert L.uint_dequant(a, a, null, 16, 128, 3, 128, 0, a, null) == 1
    assert L.uint_dequant(a, a, a, 16, 128, 3, 128, 5, a, null) == 2
    assert L.pot_validate_scales(a, 0, 3, a, null) == 3
    assert L.pot_launch_count() == before


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("kind", [0, 1])
def test_tiled_layout_map_is_a_bijection_with_pairs_16_apart(L, bits, kind):
    from paper_2507_11959_b200 import binding
    seen = {}
    for q in range(128):
        for b in range(bits):
            w, bit = binding.pot_layout_bit(bits, kind, q, b)
            assert 0 <= w < 4 * bits and 0 <= bit < 32
            assert (w, bit) not in seen
            seen[(w, bit)] = (q, b)
    assert len(seen) == 128 * bits == 4 * bits * 32        # exactly n bits per weight, nothing unused
    for q in range(0, 128, 2):                             # the two codes of a pair: same word, 16 bits apart
        for b in range(bits):
            w0, b0 = binding.pot_layout_bit(bits, kind, q, b)
            w1, b1 = binding.pot_layout_bit(bits, kind, q + 1, b)
            assert w0 == w1 and (b1 - b0) % 32 == 16
    with pytest.raises(binding.PotError):
        binding.pot_layout_bit(bits, kind, 128, 0)
