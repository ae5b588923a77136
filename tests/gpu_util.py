"""Helpers shared by the GPU parity tests: seeded cases quantized by the ORACLE on the host (so that
no oracle input ever comes from the CUDA path), uploads, and the GEMV/GEMM tolerance gate."""
from __future__ import annotations

import numpy as np
import torch

from oracle import pot_oracle as oracle
from paper_2507_11959_b200 import synth

DEV = "cuda"


def to_dev(a: np.ndarray, dtype=None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.to(DEV)


def f16_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> float16 cuda tensor"""
    return to_dev(bits.view(np.int16), torch.float16)


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> bfloat16 cuda tensor"""
    return to_dev(bits.view(np.int16), torch.bfloat16)


def f16_bits_to_bf16_bits(bits: np.ndarray) -> np.ndarray:
    """FP16 bit patterns rounded to BF16 bit patterns (round to nearest even), by integer arithmetic on float32"""
    u = np.ascontiguousarray(bits).view(np.float16).astype(np.float32).view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    """16-bit float cuda tensor -> uint16 numpy bit patterns"""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class PotCase:
    """Weights quantized by the oracle; device copies of the canonical codes and scales."""

    def __init__(self, N, K, bits, G, dist="normal", sigma=0.02, rule=oracle.RULE_TOP, seed=(0, 0), W_bits=None):
        self.N, self.K, self.bits, self.G = N, K, bits, G
        self.W_bits = synth.weights(synth.rng_for(*seed), N, K, dist, sigma) if W_bits is None else W_bits
        self.codes, self.S = oracle.quantize(self.W_bits, bits, G, rule)
        self.packed = oracle.pack(self.codes, bits)
        self.d_packed = to_dev(self.packed)
        self.d_S = f16_dev(self.S)

    def tiled(self):
        from paper_2507_11959_b200 import binding
        return binding.pot_repack(self.d_packed, self.K, self.bits, 0)

    def tiled_S(self):
        """scales in the tiled order that goes with tiled()"""
        from paper_2507_11959_b200 import binding
        return binding.pot_repack_scales(self.d_S, self.K, self.G, 0)


class UintCase:
    def __init__(self, N, K, bits, G, dist="normal", sigma=0.02, seed=(0, 0), W_bits=None):
        self.N, self.K, self.bits, self.G = N, K, bits, G
        self.W_bits = synth.weights(synth.rng_for(*seed), N, K, dist, sigma) if W_bits is None else W_bits
        self.codes, self.S, self.Z = oracle.uint_quantize(self.W_bits, bits, G)
        self.packed = oracle.pack(self.codes, bits)
        self.d_packed = to_dev(self.packed)
        self.d_S = f16_dev(self.S)
        self.d_Z = f16_dev(self.Z)

    def tiled(self):
        from paper_2507_11959_b200 import binding
        return binding.uint_repack(self.d_packed, self.K, self.bits, 0)

    def tiled_S(self):
        from paper_2507_11959_b200 import binding
        return binding.pot_repack_scales(self.d_S, self.K, self.G, 0)

    def tiled_Z(self):
        from paper_2507_11959_b200 import binding
        return binding.pot_repack_scales(self.d_Z, self.K, self.G, 0)


def gate(y_gpu_bits: np.ndarray, Y: np.ndarray, A: np.ndarray, bf16: bool = False):
    """|y_gpu - y_ref| <= 1e-3 * sum|w x| + 1e-5 per element, against the FP64 oracle on the same
    dequantized weights.  Also returns the tight diagnostic |err| / (2^-10 |y| + 2^-20 A): FP16
    output rounding plus FP32 accumulation should keep it O(1)."""
    if bf16:
        y = (np.ascontiguousarray(y_gpu_bits).astype(np.uint32) << 16).view(np.float32).astype(np.float64).reshape(Y.shape)
    else:
        y = y_gpu_bits.view(np.float16).astype(np.float64).reshape(Y.shape)
    err = np.abs(y - Y)
    # BF16 output: rounding the result to 8 significant bits alone costs up to 2^-8 |y|, which exceeds 1e-3 sum|w x|
    # when the terms of a short row share a sign; the gate for the BF16 route adds that term
    tol = 1e-3 * A + 1e-5 + (2.0 ** -8 * np.abs(Y) if bf16 else 0.0)
    ok = err <= tol
    tight = err / (2.0 ** (-7 if bf16 else -10) * np.abs(Y) + 2.0 ** -20 * A + 1e-30)
    return bool(ok.all()), float((err / tol).max()), float(tight.max())


# ---- stray-write detection ------------------------------------------------------------------------------------
# compute-sanitizer is not available to these tests, so every output and workspace of a parity test sits between two
# pads of a seeded byte pattern that must still be intact after the call.
_PAD = 4096
_pattern = None


def _pad_pattern() -> torch.Tensor:
    global _pattern
    if _pattern is None:
        g = torch.Generator().manual_seed(2507119590)
        _pattern = torch.randint(0, 256, (_PAD,), dtype=torch.uint8, generator=g).to(DEV)
    return _pattern


class Guarded:
    """A device buffer of `shape` / `dtype` with a 4 KB canary pad on both sides."""

    def __init__(self, shape, dtype, zero: bool = False):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.n = (n + 15) // 16 * 16
        self.buf = torch.empty(self.n + 2 * _PAD, dtype=torch.uint8, device=DEV)
        self.buf[:_PAD] = _pad_pattern()
        self.buf[_PAD + self.n:] = _pad_pattern()
        self.view = self.buf[_PAD:_PAD + n].view(dtype).reshape(shape)
        if zero:
            self.buf[_PAD:_PAD + self.n] = 0

    def intact(self) -> bool:
        return bool(torch.equal(self.buf[:_PAD], _pad_pattern()) and torch.equal(self.buf[_PAD + self.n:], _pad_pattern()))


class GuardedBinding:
    """The binding with every output and workspace it allocates placed between canary pads; after each call the
    device is synchronised and the pads are checked.  Anything else is forwarded unchanged."""

    def __init__(self):
        from paper_2507_11959_b200 import binding
        binding.lib()
        self._b = binding

    def __getattr__(self, name):
        return getattr(self._b, name)

    def _finish(self, what, *guards):
        torch.cuda.synchronize()
        for g in guards:
            assert g is None or g.intact(), f"{what}: a write landed outside its buffer"
        # bounded waits that gave up, or (checked build) an index check that failed, leave a code in these words
        assert self._b.pot_debug_errors() == (0, 0, 0), what

    def _ws(self, nbytes):
        return Guarded((nbytes,), torch.uint8, zero=True) if nbytes else None

    def pot_dequant(self, packed, scales, K, bits, group, out_dtype=0, **kw):
        out = Guarded((packed.shape[0], K), torch.float16 if out_dtype == 0 else torch.bfloat16)
        self._b.pot_dequant(packed, scales, K, bits, group, out_dtype, out=out.view, **kw)
        self._finish("pot_dequant", out)
        return out.view

    def uint_dequant(self, packed, scales, zeros, K, bits, group, kernel=0, **kw):
        out = Guarded((packed.shape[0], K), torch.float16)
        self._b.uint_dequant(packed, scales, zeros, K, bits, group, kernel, out=out.view, **kw)
        self._finish("uint_dequant", out)
        return out.view

    def pot_gemv(self, packed, scales, K, bits, group, x, layout=0, workspace=None, **kw):
        N = packed.shape[0]
        y = Guarded((N,), x.dtype)
        ws = None
        if workspace is None and layout == self._b.TILED:
            ws = self._ws(self._b.pot_gemv_workspace_bytes(N, K, bits, group))
            workspace = None if ws is None else ws.view
        self._b.pot_gemv(packed, scales, K, bits, group, x, layout, y=y.view, workspace=workspace, **kw)
        self._finish("pot_gemv", y, ws)
        return y.view

    def uint_gemv(self, packed, scales, zeros, K, bits, group, x, layout=0, workspace=None, **kw):
        N = packed.shape[0]
        y = Guarded((N,), torch.float16)
        ws = None
        if workspace is None and layout == self._b.TILED:
            ws = self._ws(self._b.pot_gemv_workspace_bytes(N, K, bits, group))
            workspace = None if ws is None else ws.view
        self._b.uint_gemv(packed, scales, zeros, K, bits, group, x, layout, y=y.view, workspace=workspace, **kw)
        self._finish("uint_gemv", y, ws)
        return y.view

    def pot_gemm(self, packed, scales, K, bits, group, X, layout=0, workspace=None, **kw):
        N, M = packed.shape[0], X.shape[0]
        Y = Guarded((M, N), X.dtype)
        ws = None
        if workspace is None and layout == self._b.TILED:
            ws = self._ws(self._b.pot_gemm_workspace_bytes(M, N, K, bits, group))
            workspace = None if ws is None else ws.view
        self._b.pot_gemm(packed, scales, K, bits, group, X, layout, Y=Y.view, workspace=workspace, **kw)
        self._finish("pot_gemm", Y, ws)
        return Y.view

    def new_workspace(self, nbytes, device=DEV):
        """A zeroed, guarded workspace; keep the returned tensor's guard alive through `guard_of`."""
        if nbytes == 0:
            return None
        g = Guarded((nbytes,), torch.uint8, zero=True)
        g.view._guard = g
        return g.view
