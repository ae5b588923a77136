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


def gate(y_gpu_bits: np.ndarray, Y: np.ndarray, A: np.ndarray):
    """|y_gpu - y_ref| <= 1e-3 * sum|w x| + 1e-5 per element, against the FP64 oracle on the same
    dequantized weights.  Also returns the tight diagnostic |err| / (2^-10 |y| + 2^-20 A): FP16
    output rounding plus FP32 accumulation should keep it O(1)."""
    y = y_gpu_bits.view(np.float16).astype(np.float64).reshape(Y.shape)
    err = np.abs(y - Y)
    ok = err <= 1e-3 * A + 1e-5
    tight = err / (2.0 ** -10 * np.abs(Y) + 2.0 ** -20 * A + 1e-30)
    return bool(ok.all()), float((err / (1e-3 * A + 1e-5)).max()), float(tight.max())
