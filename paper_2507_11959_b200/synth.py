"""Seeded synthetic inputs for the five workloads.

This module only draws random tensors (numpy ``Generator(PCG64)``, FP64 rounded to FP16 by
numpy) and lists the workload shapes.  It contains none of the method's arithmetic: no
quantizer, no packing, no dequantization.  Both the CUDA path and the CPU oracle are fed
from here so that neither side owns the generator.

Weights stand in for LLaMA / Llama-2 projection matrices (bell-shaped, heavy-tailed; the
shapes are the public Llama-2 7B / 13B / 70B projection shapes); activations stand in for
decoder hidden states with a few large "outlier" channels.  FP16 tensors are returned as
``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 250711959 * 10


@dataclass(frozen=True)
class Projection:
    name: str
    K: int  # input features (reduction dimension; groups run along it)
    N: int  # output features


# config index -> description of the synthetic workload
LLAMA2_7B = (Projection("qkv", 4096, 12288), Projection("o", 4096, 4096), Projection("gate", 4096, 11008),
             Projection("up", 4096, 11008), Projection("down", 11008, 4096))
LLAMA2_13B = (Projection("qkv", 5120, 15360), Projection("gate_or_up", 5120, 13824), Projection("down", 13824, 5120))
LLAMA2_70B = (Projection("qkv_gqa", 8192, 10240), Projection("gate_or_up", 8192, 28672), Projection("down", 28672, 8192))
DEQUANT_SWEEP = ((4096, 4096), (8192, 8192), (28672, 8192))  # (N, K)
LLAMA2_7B_LAYERS = 32
SMALL_BATCH_M = (1, 4, 8, 16, 32)
PREFILL_M = 2048


def rng_for(config_index: int, tensor_index: int) -> np.random.Generator:
    """One independent stream per (config, tensor).  tensor_index is the position of the
    tensor in the config's fixed order (weights of projection 0, its activations, ...)."""
    ss = np.random.SeedSequence(BASE_SEED + int(config_index))
    child = ss.spawn(int(tensor_index) + 1)[int(tensor_index)]
    return np.random.Generator(np.random.PCG64(child))


def _to_f16_bits(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a.astype(np.float16)).view(np.uint16)


def weights(rng: np.random.Generator, N: int, K: int, dist: str = "normal", sigma: float = 0.02) -> np.ndarray:
    """[N,K] FP16 bit patterns.  dist 'normal': N(0, sigma^2); 't5': sigma * Student-t(nu=5)."""
    out = np.empty((N, K), dtype=np.uint16)
    step = max(1, (1 << 22) // max(K, 1))  # draw in row blocks to bound the FP64 temporaries
    for r0 in range(0, N, step):
        r1 = min(N, r0 + step)
        if dist == "normal":
            a = rng.standard_normal((r1 - r0, K)) * sigma
        elif dist == "t5":
            a = rng.standard_t(5, (r1 - r0, K)) * sigma
        else:
            raise ValueError(dist)
        out[r0:r1] = _to_f16_bits(a)
    return out


def activations(rng: np.random.Generator, M: int, K: int, outliers: bool = True) -> np.ndarray:
    """[M,K] FP16 bit patterns ~ N(0,1); with outliers, floor(0.01*K) channels (a seeded
    permutation, the same channels for every token) are multiplied by 20."""
    a = rng.standard_normal((M, K))
    if outliers:
        n_out = int(0.01 * K)
        ch = rng.permutation(K)[:n_out]
        a[:, ch] *= 20.0
    return _to_f16_bits(a)


def f16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(bits).view(np.float16).astype(np.float64)
