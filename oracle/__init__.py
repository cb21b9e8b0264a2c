"""CPU oracle for the tiled low-rank-binary-index layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy front end of ``lrbi_oracle.c`` (plain C, fp64, one byte per bit).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do, and this package
imports nothing from them.

Functions (citations are to the paper):
  decode_mask          Eq. 3 applied tile by tile (Section 3.1).
  masked_gemm          Y = X (W .* Ia)^T with Ia as the masking layer (Sections 2, 2.2).
  masked_gemm_samples  the same two definitions evaluated only at chosen outputs.
  bf16_to_f64          exact widening of bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lrbi_oracle.c")
_LIB = os.path.join(_HERE, "liblrbi_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP). Returns the path of the .so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        lib.lrbi_oracle_decode.argtypes = [i64] * 5 + [vp] * 3
        lib.lrbi_oracle_decode.restype = None
        lib.lrbi_oracle_masked_gemm.argtypes = [i64] * 3 + [vp] * 4
        lib.lrbi_oracle_masked_gemm.restype = None
        lib.lrbi_oracle_masked_gemm_samples.argtypes = [i64] * 5 + [vp] * 4 + [i64] + [vp] * 3
        lib.lrbi_oracle_masked_gemm_samples.restype = None
        lib.lrbi_oracle_bf16_to_f64.argtypes = [i64, vp, vp]
        lib.lrbi_oracle_bf16_to_f64.restype = None
        lib.lrbi_oracle_threads.argtypes = []
        lib.lrbi_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Threads the oracle's outer loops use on this machine."""
    return int(_load().lrbi_oracle_threads())


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _grid(rows, cols, tm, tn):
    return -(-rows // tm), -(-cols // tn)


def decode_mask(Ip: np.ndarray, Iz: np.ndarray, rows: int, cols: int) -> np.ndarray:
    """Tiled Boolean product (Eq. 3 per tile).

    Ip: uint8 [GR, GC, tm, k], Iz: uint8 [GR, GC, k, tn]; returns uint8 [rows, cols].
    """
    Ip = _c(Ip, np.uint8)
    Iz = _c(Iz, np.uint8)
    GR, GC, tm, k = Ip.shape
    GR2, GC2, k2, tn = Iz.shape
    if (GR, GC, k) != (GR2, GC2, k2) or (GR, GC) != _grid(rows, cols, tm, tn):
        raise ValueError("factor shapes do not match the tile grid")
    if Ip.max(initial=0) > 1 or Iz.max(initial=0) > 1:
        raise ValueError("factor entries must be 0 or 1")
    M = np.empty((rows, cols), dtype=np.uint8)
    _load().lrbi_oracle_decode(rows, cols, tm, tn, k, Ip.ctypes.data, Iz.ctypes.data, M.ctypes.data)
    return M


def masked_gemm(W_bits: np.ndarray, M: np.ndarray, X_bits: np.ndarray) -> np.ndarray:
    """Y[b, o] = sum over kept i of X[b, i] * W[o, i], in fp64.

    W_bits: uint16 [N, K] bf16 patterns, M: uint8 [N, K], X_bits: uint16 [B, K].
    """
    W_bits = _c(W_bits, np.uint16)
    X_bits = _c(X_bits, np.uint16)
    M = _c(M, np.uint8)
    N, K = W_bits.shape
    B, K2 = X_bits.shape
    if K2 != K or M.shape != (N, K):
        raise ValueError("shape mismatch")
    Y = np.empty((B, N), dtype=np.float64)
    _load().lrbi_oracle_masked_gemm(B, N, K, W_bits.ctypes.data, M.ctypes.data, X_bits.ctypes.data, Y.ctypes.data)
    return Y


def masked_gemm_samples(W_bits, Ip, Iz, X_bits, b_idx, o_idx) -> np.ndarray:
    """Y[b_idx[s], o_idx[s]] for each s, decoding only the mask rows that are needed."""
    W_bits = _c(W_bits, np.uint16)
    X_bits = _c(X_bits, np.uint16)
    Ip = _c(Ip, np.uint8)
    Iz = _c(Iz, np.uint8)
    b_idx = _c(b_idx, np.int64)
    o_idx = _c(o_idx, np.int64)
    N, K = W_bits.shape
    GR, GC, tm, k = Ip.shape
    tn = Iz.shape[3]
    if (GR, GC) != _grid(N, K, tm, tn) or Iz.shape[:3] != (GR, GC, k) or X_bits.shape[1] != K:
        raise ValueError("shape mismatch")
    if b_idx.shape != o_idx.shape or b_idx.ndim != 1:
        raise ValueError("sample index arrays must be 1-D and equal length")
    if len(b_idx) and (b_idx.min() < 0 or b_idx.max() >= X_bits.shape[0] or o_idx.min() < 0 or o_idx.max() >= N):
        raise ValueError("sample index out of range")
    out = np.empty(len(b_idx), dtype=np.float64)
    _load().lrbi_oracle_masked_gemm_samples(
        N, K, tm, tn, k, W_bits.ctypes.data, Ip.ctypes.data, Iz.ctypes.data,
        X_bits.ctypes.data, len(b_idx), b_idx.ctypes.data, o_idx.ctypes.data, out.ctypes.data)
    return out


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = _c(bits, np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().lrbi_oracle_bf16_to_f64(bits.size, bits.ctypes.data, out.ctypes.data)
    return out
