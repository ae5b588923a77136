"""Thin ctypes binding of the C-ABI library (``include/pot.h``), same names as the C entry
points.  It only marshals arguments: every step of the path runs in the library's CUDA
kernels.  Tensors are torch CUDA tensors (PyTorch is used for device memory and streams
only); there is no CPU fallback -- if the library is missing or fails to load, importing a
symbol from it raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

import os

_HERE = Path(__file__).resolve().parent
# POT_B200_LIB selects another build of the same library (e.g. libpot_b200_checked.so, the -DPOT_CHECKED build)
LIB_PATH = Path(os.environ["POT_B200_LIB"]) if os.environ.get("POT_B200_LIB") else _HERE / "libpot_b200.so"

POT_OK = 0
F16, BF16 = 0, 1
SCALE_TOP, SCALE_PAPER_S0, SCALE_GIVEN, SCALE_SEARCH = 0, 1, 2, 3
CANONICAL, TILED = 0, 1
UINT_FAST, UINT_NAIVE = 0, 1

EXPORTS = [
    "pot_status_string", "pot_packed_bytes", "pot_scales_bytes", "pot_gemv_workspace_bytes",
    "pot_gemm_workspace_bytes", "pot_launch_count", "pot_quantize_ref", "pot_validate_scales", "pot_repack", "pot_repack_scales", "pot_layout_scale_index",
    "uint_repack", "pot_dequant", "pot_gemv", "pot_gemv_bf16", "pot_gemv_host", "pot_gemm", "pot_gemm_bf16", "uint_quantize_ref", "uint_dequant",
    "uint_gemv", "pot_layout_bit", "pot_gemv_noalloc", "pot_gemv_noalloc_max_scratch_bytes", "pot_debug_gemv_error", "pot_debug_gemv_plan", "pot_debug_gemm_error", "pot_debug_prefill_error",
]

_lib = None


class PotError(RuntimeError):
    pass


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built by ``python -m paper_2507_11959_b200.build``)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise PotError(f"{LIB_PATH} not built: run `python -m paper_2507_11959_b200.build`")
        L = ctypes.CDLL(str(LIB_PATH))
        i64, i32, vp, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t
        L.pot_status_string.restype = ctypes.c_char_p
        L.pot_status_string.argtypes = [i32]
        L.pot_packed_bytes.restype = sz
        L.pot_packed_bytes.argtypes = [i64, i64, i32]
        L.pot_scales_bytes.restype = sz
        L.pot_scales_bytes.argtypes = [i64, i64, i32]
        L.pot_gemv_workspace_bytes.restype = sz
        L.pot_gemv_workspace_bytes.argtypes = [i64, i64, i32, i32]
        L.pot_gemm_workspace_bytes.restype = sz
        L.pot_gemm_workspace_bytes.argtypes = [i64, i64, i64, i32, i32]
        L.pot_launch_count.restype = ctypes.c_uint64
        L.pot_launch_count.argtypes = []
        L.pot_quantize_ref.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp, vp]
        L.pot_validate_scales.argtypes = [vp, i64, i32, vp, vp]
        L.pot_repack.argtypes = [vp, vp, i64, i64, i32, i32, vp]
        L.uint_repack.argtypes = [vp, vp, i64, i64, i32, i32, vp]
        L.pot_repack_scales.argtypes = [vp, vp, i64, i64, i32, i32, vp]
        L.pot_debug_gemv_plan.argtypes = [i64, i64, i32, i32, i32, vp, vp, vp, vp, vp]
        L.pot_layout_scale_index.argtypes = [i64, i64, i32, i64, i64, vp]
        L.pot_dequant.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, vp]
        L.pot_gemv.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, vp, vp, sz, vp]
        L.pot_gemv_bf16.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, vp, vp, sz, vp]
        L.pot_gemm_bf16.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, i64, vp, vp, sz, vp]
        L.pot_gemv_host.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.pot_gemm.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, i64, vp, vp, sz, vp]
        L.uint_quantize_ref.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp, vp]
        L.uint_dequant.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, vp, vp]
        L.uint_gemv.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, vp, vp, vp, sz, vp]
        L.pot_layout_bit.argtypes = [i32, i32, i32, i32, vp, vp]
        L.pot_gemv_noalloc.argtypes = [vp, vp, i64, i64, i32, i32, vp, vp, vp]
        L.pot_gemv_noalloc_max_scratch_bytes.restype = sz
        L.pot_gemv_noalloc_max_scratch_bytes.argtypes = []
        for name in EXPORTS:
            fn = getattr(L, name)
            if fn.restype is ctypes.c_int and name not in ("pot_status_string",):
                fn.restype = i32
        _lib = L
    return _lib


def _check(status: int, what: str) -> None:
    if status != POT_OK:
        raise PotError(f"{what}: {lib().pot_status_string(status).decode()} (status {status})")


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def pot_status_string(status: int) -> str:
    return lib().pot_status_string(status).decode()


def pot_packed_bytes(N: int, K: int, bits: int) -> int:
    return int(lib().pot_packed_bytes(N, K, bits))


def pot_scales_bytes(N: int, K: int, group: int) -> int:
    return int(lib().pot_scales_bytes(N, K, group))


def pot_gemv_workspace_bytes(N: int, K: int, bits: int, group: int) -> int:
    return int(lib().pot_gemv_workspace_bytes(N, K, bits, group))


def pot_gemm_workspace_bytes(M: int, N: int, K: int, bits: int, group: int) -> int:
    return int(lib().pot_gemm_workspace_bytes(M, N, K, bits, group))


def pot_launch_count() -> int:
    return int(lib().pot_launch_count())


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor | None:
    """Zero-initialised scratch (the split-K arrival counters must start at zero; the kernels
    leave them at zero, so one workspace can be reused by consecutive calls on one stream)."""
    if nbytes == 0:
        return None
    return torch.zeros(nbytes, dtype=torch.uint8, device=device)


def pot_quantize_ref(W: torch.Tensor, bits: int, group: int, rule: int = SCALE_TOP,
                     scales: torch.Tensor | None = None, stream=None):
    """W [N,K] float16 cuda -> (packed uint8 [N, K*bits/8] canonical, scales float16 [N, K/group])."""
    N, K = W.shape
    assert W.dtype == torch.float16 and W.is_cuda and W.is_contiguous()
    if rule == SCALE_GIVEN:
        assert scales is not None and scales.dtype == torch.float16 and scales.is_contiguous()
    else:
        scales = torch.empty((N, K // group), dtype=torch.float16, device=W.device)
    packed = torch.empty((N, K * bits // 8), dtype=torch.uint8, device=W.device)
    _check(lib().pot_quantize_ref(_ptr(W), N, K, bits, group, rule, _ptr(scales), _ptr(packed), _stream(stream)),
           "pot_quantize_ref")
    return packed, scales


def pot_validate_scales(scales: torch.Tensor, bits: int, stream=None) -> torch.Tensor:
    """Returns a device int32 tensor holding the number of illegal scales (reading it synchronises)."""
    bad = torch.zeros(1, dtype=torch.int32, device=scales.device)
    _check(lib().pot_validate_scales(_ptr(scales), scales.numel(), bits, _ptr(bad), _stream(stream)), "pot_validate_scales")
    return bad


def pot_repack(packed: torch.Tensor, K: int, bits: int, direction: int = 0, stream=None) -> torch.Tensor:
    """canonical -> tiled (direction 0) or back (direction 1); same shape and size."""
    out = torch.empty_like(packed)
    _check(lib().pot_repack(_ptr(packed), _ptr(out), packed.shape[0], K, bits, direction, _stream(stream)), "pot_repack")
    return out


def pot_repack_scales(scales: torch.Tensor, K: int, group: int, direction: int = 0, stream=None) -> torch.Tensor:
    """Per-group parameters (scales, or the uniform twin's zero-points) [N, K/group]: row-major -> tiled
    (direction 0) or back (direction 1); same shape and size.  The tiled kernels take both codes and parameters tiled."""
    out = torch.empty_like(scales)
    _check(lib().pot_repack_scales(_ptr(scales), _ptr(out), scales.shape[0], K, group, direction, _stream(stream)),
           "pot_repack_scales")
    return out


def pot_layout_scale_index(N: int, K: int, group: int, row: int, g: int) -> int:
    idx = ctypes.c_int64(-1)
    _check(lib().pot_layout_scale_index(N, K, group, row, g, ctypes.byref(idx)), "pot_layout_scale_index")
    return idx.value


def uint_repack(packed: torch.Tensor, K: int, bits: int, direction: int = 0, stream=None) -> torch.Tensor:
    out = torch.empty_like(packed)
    _check(lib().uint_repack(_ptr(packed), _ptr(out), packed.shape[0], K, bits, direction, _stream(stream)), "uint_repack")
    return out


def pot_dequant(packed: torch.Tensor, scales: torch.Tensor, K: int, bits: int, group: int, out_dtype: int = F16,
                out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    N = packed.shape[0]
    if out is None:
        out = torch.empty((N, K), dtype=torch.float16 if out_dtype == F16 else torch.bfloat16, device=packed.device)
    _check(lib().pot_dequant(_ptr(packed), _ptr(scales), N, K, bits, group, out_dtype, _ptr(out), _stream(stream)), "pot_dequant")
    return out


def pot_gemv(packed, scales, K: int, bits: int, group: int, x: torch.Tensor, layout: int = CANONICAL,
             y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """x float16 -> pot_gemv, x bfloat16 -> pot_gemv_bf16 (the output has the activations' dtype)."""
    N = packed.shape[0]
    assert x.dtype in (torch.float16, torch.bfloat16)
    if y is None:
        y = torch.empty(N, dtype=x.dtype, device=x.device)
    assert y.dtype == x.dtype
    need = pot_gemv_workspace_bytes(N, K, bits, group) if layout == TILED else 0
    if need and workspace is None:
        workspace = new_workspace(need, x.device)
    fn = lib().pot_gemv if x.dtype == torch.float16 else lib().pot_gemv_bf16
    _check(fn(_ptr(packed), _ptr(scales), N, K, bits, group, layout, _ptr(x), _ptr(y), _ptr(workspace),
              0 if workspace is None else workspace.numel(), _stream(stream)), "pot_gemv")
    return y


def pot_gemv_host(packed, scales, K: int, bits: int, group: int, x_host: torch.Tensor, y_host: torch.Tensor,
                  d_x: torch.Tensor, d_y: torch.Tensor, layout: int = CANONICAL, workspace=None, stream=None) -> None:
    """x_host / y_host: CPU (pinned) float16 tensors; d_x / d_y: device staging.  Asynchronous."""
    N = packed.shape[0]
    assert not x_host.is_cuda and not y_host.is_cuda and d_x.is_cuda and d_y.is_cuda
    _check(lib().pot_gemv_host(_ptr(packed), _ptr(scales), N, K, bits, group, layout, _ptr(x_host), _ptr(y_host),
                               _ptr(d_x), _ptr(d_y), _ptr(workspace), 0 if workspace is None else workspace.numel(),
                               _stream(stream)), "pot_gemv_host")


def pot_gemm(packed, scales, K: int, bits: int, group: int, X: torch.Tensor, layout: int = CANONICAL,
             Y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    N, M = packed.shape[0], X.shape[0]
    assert X.dtype in (torch.float16, torch.bfloat16)
    if Y is None:
        Y = torch.empty((M, N), dtype=X.dtype, device=X.device)
    assert Y.dtype == X.dtype
    need = pot_gemm_workspace_bytes(M, N, K, bits, group) if layout == TILED else 0
    if need and workspace is None:
        workspace = new_workspace(need, X.device)
    fn = lib().pot_gemm if X.dtype == torch.float16 else lib().pot_gemm_bf16
    _check(fn(_ptr(packed), _ptr(scales), N, K, bits, group, layout, _ptr(X), M, _ptr(Y), _ptr(workspace),
              0 if workspace is None else workspace.numel(), _stream(stream)), "pot_gemm")
    return Y


def uint_quantize_ref(W: torch.Tensor, bits: int, group: int, stream=None):
    N, K = W.shape
    scales = torch.empty((N, K // group), dtype=torch.float16, device=W.device)
    zeros = torch.empty((N, K // group), dtype=torch.float16, device=W.device)
    packed = torch.empty((N, K * bits // 8), dtype=torch.uint8, device=W.device)
    _check(lib().uint_quantize_ref(_ptr(W), N, K, bits, group, _ptr(scales), _ptr(zeros), _ptr(packed), _stream(stream)),
           "uint_quantize_ref")
    return packed, scales, zeros


def uint_dequant(packed, scales, zeros, K: int, bits: int, group: int, kernel: int = UINT_FAST,
                 out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    N = packed.shape[0]
    if out is None:
        out = torch.empty((N, K), dtype=torch.float16, device=packed.device)
    _check(lib().uint_dequant(_ptr(packed), _ptr(scales), _ptr(zeros), N, K, bits, group, kernel, _ptr(out), _stream(stream)),
           "uint_dequant")
    return out


def uint_gemv(packed, scales, zeros, K: int, bits: int, group: int, x: torch.Tensor, layout: int = CANONICAL,
              y: torch.Tensor | None = None, workspace=None, stream=None) -> torch.Tensor:
    N = packed.shape[0]
    if y is None:
        y = torch.empty(N, dtype=torch.float16, device=x.device)
    need = pot_gemv_workspace_bytes(N, K, bits, group) if layout == TILED else 0
    if need and workspace is None:
        workspace = new_workspace(need, x.device)
    _check(lib().uint_gemv(_ptr(packed), _ptr(scales), _ptr(zeros), N, K, bits, group, layout, _ptr(x), _ptr(y),
                           _ptr(workspace), 0 if workspace is None else workspace.numel(), _stream(stream)), "uint_gemv")
    return y


def pot_layout_bit(bits: int, kind: int, q: int, b: int) -> tuple[int, int]:
    word, bit = ctypes.c_int(-1), ctypes.c_int(-1)
    _check(lib().pot_layout_bit(bits, kind, q, b, ctypes.byref(word), ctypes.byref(bit)), "pot_layout_bit")
    return word.value, bit.value


def pot_gemv_noalloc_max_scratch_bytes() -> int:
    return int(lib().pot_gemv_noalloc_max_scratch_bytes())


def pot_gemv_noalloc(packed_tiled, scales, K: int, bits: int, group: int, x: torch.Tensor, y: torch.Tensor,
                     stream=None) -> torch.Tensor:
    """pot_gemv on the tiled layout with the library's built-in scratch array instead of a caller
    workspace -- for callers that may not allocate device memory.  `y` must be supplied (this wrapper
    allocates nothing either).  Shapes that need more than pot_gemv_noalloc_max_scratch_bytes() raise."""
    _check(lib().pot_gemv_noalloc(_ptr(packed_tiled), _ptr(scales), packed_tiled.shape[0], K, bits, group, _ptr(x),
                                  _ptr(y), _stream(stream)), "pot_gemv_noalloc")
    return y


def pot_debug_gemv_plan(N: int, K: int, bits: int, group: int, uniform: bool = False) -> dict:
    """{'ctas_per_sm', 'row_block_split', 'ring_slots', 'units_per_slot', 'x_in_smem'} of the tiled GEMV launch."""
    v = [ctypes.c_int(-1) for _ in range(5)]
    _check(lib().pot_debug_gemv_plan(N, K, bits, group, 1 if uniform else 0, *[ctypes.byref(x) for x in v]), "pot_debug_gemv_plan")
    return dict(zip(("ctas_per_sm", "row_block_split", "ring_slots", "units_per_slot", "x_in_smem"), (x.value for x in v)))


def pot_debug_errors() -> tuple[int, int, int]:
    """(gemv, gemm, prefill) device error words, read and cleared; all 0 when every bounded wait completed."""
    return int(lib().pot_debug_gemv_error()), int(lib().pot_debug_gemm_error()), int(lib().pot_debug_prefill_error())
