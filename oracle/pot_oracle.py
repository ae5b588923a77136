"""ctypes loader for the CPU oracle (``pot_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the bench's
CPU-baseline / reference legs.  Nothing in the product package imports this module and this
module imports nothing from the product package.  All arrays are numpy; FP16/BF16 tensors
travel as ``uint16`` bit patterns so that no conversion routine other than the oracle's own
is involved.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "pot_oracle.c"
_LIB = _HERE / "libpot_oracle.so"

RULE_TOP, RULE_PAPER_S0, RULE_GIVEN = 0, 1, 2
F16, BF16 = 0, 1


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP over rows/groups).  Returns the library path."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        i64, i32, vp, dbl = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_double
        u16 = ctypes.c_uint16
        L.po_num_threads.restype = i32
        L.po_f16_to_f64.restype = dbl
        L.po_f16_to_f64.argtypes = [u16]
        L.po_f64_to_f16.restype = u16
        L.po_f64_to_f16.argtypes = [dbl, vp]
        L.po_bf16_to_f64.restype = dbl
        L.po_bf16_to_f64.argtypes = [u16]
        L.po_f64_to_bf16.restype = u16
        L.po_f64_to_bf16.argtypes = [dbl, vp]
        L.po_clamp_scale_bits.restype = u16
        L.po_clamp_scale_bits.argtypes = [u16, i32]
        L.po_scale_in_range.restype = i32
        L.po_scale_in_range.argtypes = [u16, i32]
        L.po_quantize.restype = i32
        L.po_quantize.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp]
        L.po_pack.restype = None
        L.po_pack.argtypes = [vp, i64, i64, i32, vp]
        L.po_unpack.restype = None
        L.po_unpack.argtypes = [vp, i64, i64, i32, vp]
        L.po_dequant.restype = i64
        L.po_dequant.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp]
        L.po_matmul.restype = i32
        L.po_matmul.argtypes = [vp, vp, i64, i64, i32, i32, vp, i64, vp, i64, vp, vp]
        L.po_matmul_bf16.restype = i32
        L.po_matmul_bf16.argtypes = [vp, vp, i64, i64, i32, i32, vp, i64, vp, i64, vp, vp]
        L.po_scale_search.restype = i32
        L.po_scale_search.argtypes = [vp, i64, i64, i32, i32, vp, vp]
        L.pu_quantize.restype = i32
        L.pu_quantize.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp]
        L.pu_dequant.restype = i32
        L.pu_dequant.argtypes = [vp, vp, vp, i64, i64, i32, i32, vp]
        L.pu_matmul.restype = i32
        L.pu_matmul.argtypes = [vp, vp, vp, i64, i64, i32, i32, vp, i64, vp, i64, vp, vp]
        _lib = L
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == dtype, (a.dtype, dtype)
    return a


def num_threads() -> int:
    return int(lib().po_num_threads())


# ------------------------------------------------------------------ scalar helpers
def f16_to_f64(bits: int) -> float:
    return float(lib().po_f16_to_f64(int(bits)))


def f64_to_f16(v: float) -> tuple[int, bool]:
    flag = ctypes.c_int(0)
    b = lib().po_f64_to_f16(float(v), ctypes.byref(flag))
    return int(b), bool(flag.value)


def bf16_to_f64(bits: int) -> float:
    return float(lib().po_bf16_to_f64(int(bits)))


def f64_to_bf16(v: float) -> tuple[int, bool]:
    flag = ctypes.c_int(0)
    b = lib().po_f64_to_bf16(float(v), ctypes.byref(flag))
    return int(b), bool(flag.value)


def clamp_scale_bits(bits16: int, bits: int) -> int:
    return int(lib().po_clamp_scale_bits(int(bits16), int(bits)))


# ------------------------------------------------------------------ PoT
def quantize(W_bits: np.ndarray, bits: int, G: int, rule: int = RULE_TOP,
             scales: np.ndarray | None = None) -> tuple[np.ndarray, np.ndarray]:
    """W_bits [N,K] uint16 (FP16 patterns) -> (codes [N,K] uint8, scales [N,K/G] uint16)."""
    W_bits = _c(W_bits, np.uint16)
    N, K = W_bits.shape
    if rule == RULE_GIVEN:
        S = _c(scales, np.uint16).reshape(N, K // G).copy()
    else:
        S = np.zeros((N, K // G), dtype=np.uint16)
    codes = np.zeros((N, K), dtype=np.uint8)
    rc = lib().po_quantize(_p(W_bits), N, K, bits, G, rule, _p(S), _p(codes))
    if rc != 0:
        raise ValueError(f"po_quantize failed with {rc}")
    return codes, S


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    out = np.zeros((N, K * bits // 8), dtype=np.uint8)
    lib().po_pack(_p(codes), N, K, bits, _p(out))
    return out


def unpack(packed: np.ndarray, K: int, bits: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N = packed.shape[0]
    out = np.zeros((N, K), dtype=np.uint8)
    lib().po_unpack(_p(packed), N, K, bits, _p(out))
    return out


def dequant(packed: np.ndarray, scales: np.ndarray, K: int, bits: int, G: int,
            dtype: int = F16) -> tuple[np.ndarray, int]:
    """-> (out [N,K] uint16 bit patterns, number of outputs that needed rounding)."""
    packed = _c(packed, np.uint8)
    scales = _c(scales, np.uint16)
    N = packed.shape[0]
    out = np.zeros((N, K), dtype=np.uint16)
    rounded = lib().po_dequant(_p(packed), _p(scales), N, K, bits, G, dtype, _p(out))
    if rounded < 0:
        raise ValueError("po_dequant: bad arguments")
    return out, int(rounded)


def matmul(packed: np.ndarray, scales: np.ndarray, K: int, bits: int, G: int, X_bits: np.ndarray,
           rows: np.ndarray | None = None, dtype: int = F16) -> tuple[np.ndarray, np.ndarray]:
    """FP64 Y [M, n_rows] and A = sum|w*x| [M, n_rows] on the FP16 reconstruction with FP16 activations (dtype F16) or
    on the BF16 reconstruction with BF16 activations (dtype BF16; X_bits are then BF16 bit patterns)."""
    packed = _c(packed, np.uint8)
    scales = _c(scales, np.uint16)
    X_bits = _c(X_bits, np.uint16).reshape(-1, K)
    N, M = packed.shape[0], X_bits.shape[0]
    if rows is not None:
        rows = _c(np.asarray(rows, dtype=np.int64), np.int64)
    n_rows = N if rows is None else rows.shape[0]
    Y = np.zeros((M, n_rows), dtype=np.float64)
    A = np.zeros((M, n_rows), dtype=np.float64)
    fn = lib().po_matmul if dtype == F16 else lib().po_matmul_bf16
    rc = fn(_p(packed), _p(scales), N, K, bits, G, _p(X_bits), M, _p(rows), n_rows, _p(Y), _p(A))
    if rc != 0:
        raise ValueError(f"po_matmul failed with {rc}")
    return Y, A


def scale_search(W_bits: np.ndarray, bits: int, G: int) -> tuple[np.ndarray, np.ndarray]:
    """Algorithm 1 -> (scales [N,K/G] uint16, index i of b* = 0.01*i [N,K/G] int32)."""
    W_bits = _c(W_bits, np.uint16)
    N, K = W_bits.shape
    S = np.zeros((N, K // G), dtype=np.uint16)
    bstar = np.zeros((N, K // G), dtype=np.int32)
    rc = lib().po_scale_search(_p(W_bits), N, K, bits, G, _p(S), _p(bstar))
    if rc != 0:
        raise ValueError(f"po_scale_search failed with {rc}")
    return S, bstar


# ------------------------------------------------------------------ uniform twin
def uint_quantize(W_bits: np.ndarray, bits: int, G: int) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    W_bits = _c(W_bits, np.uint16)
    N, K = W_bits.shape
    S = np.zeros((N, K // G), dtype=np.uint16)
    Z = np.zeros((N, K // G), dtype=np.uint16)
    codes = np.zeros((N, K), dtype=np.uint8)
    rc = lib().pu_quantize(_p(W_bits), N, K, bits, G, _p(S), _p(Z), _p(codes))
    if rc != 0:
        raise ValueError(f"pu_quantize failed with {rc}")
    return codes, S, Z


def uint_dequant(packed: np.ndarray, scales: np.ndarray, zeros: np.ndarray, K: int, bits: int, G: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N = packed.shape[0]
    out = np.zeros((N, K), dtype=np.uint16)
    rc = lib().pu_dequant(_p(packed), _p(_c(scales, np.uint16)), _p(_c(zeros, np.uint16)), N, K, bits, G, _p(out))
    if rc != 0:
        raise ValueError("pu_dequant: bad arguments")
    return out


def uint_matmul(packed, scales, zeros, K, bits, G, X_bits, rows=None):
    packed = _c(packed, np.uint8)
    X_bits = _c(X_bits, np.uint16).reshape(-1, K)
    N, M = packed.shape[0], X_bits.shape[0]
    if rows is not None:
        rows = _c(np.asarray(rows, dtype=np.int64), np.int64)
    n_rows = N if rows is None else rows.shape[0]
    Y = np.zeros((M, n_rows), dtype=np.float64)
    A = np.zeros((M, n_rows), dtype=np.float64)
    rc = lib().pu_matmul(_p(packed), _p(_c(scales, np.uint16)), _p(_c(zeros, np.uint16)), N, K, bits, G,
                         _p(X_bits), M, _p(rows), n_rows, _p(Y), _p(A))
    if rc != 0:
        raise ValueError(f"pu_matmul failed with {rc}")
    return Y, A
