"""CPU oracle for the tiled low-rank-binary-index layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy front end of ``lrbi_oracle.c`` (plain C, fp64, one byte per bit).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do, and this package
imports nothing from them.

Functions (citations are to the paper):
  decode_mask          Eq. 3 applied tile by tile (Section 3.1).
  decode_mask_ranks    the same with one rank per tile (Section 3.1, last paragraph).
  masked_gemm          Y = X (W .* Ia)^T with Ia as the masking layer (Sections 2, 2.2).
  masked_gemm_samples  the same two definitions evaluated only at chosen outputs.
  masked_backward      dX = dY (W .* Ia), dW = (dY^T X) .* Ia: gradients of the masked layer (Section 2.2).
  bf16_to_f64          exact widening of bf16 bit patterns.
Inner loop of Algorithm 1 (Section 2.1), in lrbi_alg1_oracle.c and, for the search itself, below:
  threshold            binary conversion of NMF factors, entry = 1 iff value >= T (sentence under Eq. 4).
  index_cost           per tile: ones of I and of Ia, and Cost = sum of |W| where I = 1 and Ia = 0.
  sz_from_eq7          the inversion of Eq. 7 printed under it.
  threshold_for_sparsity, alg1_search   the S_p sweep with the S_z search, in the order of Algorithm 1.
  nmf_multiplicative   the NMF of |W| that Algorithm 1 starts from, tile by tile, by multiplicative updates.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lrbi_oracle.c")
_SRC2 = os.path.join(_HERE, "lrbi_alg1_oracle.c")
_LIB = os.path.join(_HERE, "liblrbi_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP). Returns the path of the .so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC2)):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, _SRC2, "-lm"],
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
        lib.lrbi_oracle_decode_ranks.argtypes = [i64] * 5 + [vp] * 4
        lib.lrbi_oracle_decode_ranks.restype = None
        lib.lrbi_oracle_masked_gemm.argtypes = [i64] * 3 + [vp] * 4
        lib.lrbi_oracle_masked_gemm.restype = None
        lib.lrbi_oracle_masked_backward.argtypes = [i64] * 3 + [vp] * 6
        lib.lrbi_oracle_masked_backward.restype = None
        lib.lrbi_oracle_masked_gemm_samples.argtypes = [i64] * 5 + [vp] * 4 + [i64] + [vp] * 3
        lib.lrbi_oracle_masked_gemm_samples.restype = None
        lib.lrbi_oracle_bf16_to_f64.argtypes = [i64, vp, vp]
        lib.lrbi_oracle_bf16_to_f64.restype = None
        lib.lrbi_oracle_threshold.argtypes = [i64, i64, vp, vp, vp]
        lib.lrbi_oracle_threshold.restype = None
        lib.lrbi_oracle_index_cost.argtypes = [i64] * 4 + [vp, ctypes.c_float] + [vp] * 5
        lib.lrbi_oracle_index_cost.restype = None
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


def decode_mask_ranks(Ip: np.ndarray, Iz: np.ndarray, ranks: np.ndarray, rows: int, cols: int) -> np.ndarray:
    """Tiled Boolean product with one rank per tile: tile t uses Ip[..., :ranks[t]] and Iz[..., :ranks[t], :].

    Ip: uint8 [GR, GC, tm, kmax], Iz: uint8 [GR, GC, kmax, tn], ranks: [GR*GC] (row-major grid order).
    """
    Ip = _c(Ip, np.uint8)
    Iz = _c(Iz, np.uint8)
    ranks = _c(ranks, np.int32).ravel()
    GR, GC, tm, kmax = Ip.shape
    tn = Iz.shape[3]
    if Iz.shape[:3] != (GR, GC, kmax) or (GR, GC) != _grid(rows, cols, tm, tn) or ranks.size != GR * GC:
        raise ValueError("factor shapes do not match the tile grid")
    if ranks.min(initial=0) < 0 or ranks.max(initial=0) > kmax:
        raise ValueError("a rank lies outside 0..kmax")
    M = np.empty((rows, cols), dtype=np.uint8)
    _load().lrbi_oracle_decode_ranks(rows, cols, tm, tn, kmax, ranks.ctypes.data, Ip.ctypes.data, Iz.ctypes.data, M.ctypes.data)
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


def masked_backward(W_bits: np.ndarray, M: np.ndarray, X_bits: np.ndarray, dY_bits: np.ndarray):
    """Gradients of Y = X (W .* M)^T for dY = dL/dY, in fp64: (dX [B, K], dW [N, K]); dW is zero where M is."""
    W_bits, X_bits, dY_bits, M = _c(W_bits, np.uint16), _c(X_bits, np.uint16), _c(dY_bits, np.uint16), _c(M, np.uint8)
    N, K = W_bits.shape
    B = X_bits.shape[0]
    if X_bits.shape != (B, K) or dY_bits.shape != (B, N) or M.shape != (N, K):
        raise ValueError("shape mismatch")
    dX = np.empty((B, K), dtype=np.float64)
    dW = np.empty((N, K), dtype=np.float64)
    _load().lrbi_oracle_masked_backward(B, N, K, W_bits.ctypes.data, M.ctypes.data, X_bits.ctypes.data, dY_bits.ctypes.data,
                                        dX.ctypes.data, dW.ctypes.data)
    return dX, dW


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


# ------------------------------------------------------------------------------------------------
# Inner loop of Algorithm 1 (Section 2.1)
# ------------------------------------------------------------------------------------------------
def threshold(values: np.ndarray, T) -> np.ndarray:
    """Binary conversion of NMF factors: entry = 1 iff value >= threshold (sentence under Eq. 4).

    values: float32 [ntiles, ...]; T: one threshold per tile (a scalar is used for every tile).
    """
    values = _c(values, np.float32)
    ntiles = values.shape[0]
    T = np.ascontiguousarray(np.broadcast_to(np.asarray(T, dtype=np.float32), (ntiles,)))
    out = np.empty(values.shape, dtype=np.uint8)
    _load().lrbi_oracle_threshold(ntiles, values[0].size, values.ctypes.data, T.ctypes.data, out.ctypes.data)
    return out


def index_cost(W_bits: np.ndarray, theta: float, Ia: np.ndarray, tm: int, tn: int):
    """Per tile (row-major grid order): ones of I = (|W| >= theta), ones of Ia, positions with I = 1 and
    Ia = 0, and Cost = the sum of |W| over those positions (the cost line of Algorithm 1)."""
    W_bits = _c(W_bits, np.uint16)
    Ia = _c(Ia, np.uint8)
    rows, cols = W_bits.shape
    if Ia.shape != (rows, cols):
        raise ValueError("shape mismatch")
    gr, gc = _grid(rows, cols, tm, tn)
    kept_i, kept_a, lost = (np.empty(gr * gc, dtype=np.int64) for _ in range(3))
    cost = np.empty(gr * gc, dtype=np.float64)
    _load().lrbi_oracle_index_cost(rows, cols, tm, tn, W_bits.ctypes.data, ctypes.c_float(np.float32(theta)), Ia.ctypes.data,
                                   kept_i.ctypes.data, kept_a.ctypes.data, lost.ctypes.data, cost.ctypes.data)
    return kept_i, kept_a, lost, cost


def sz_from_eq7(S: float, Sp: float, k: int) -> float:
    """S_z = (S^(1/k) - S_p) / (1 - S_p), the inversion of Eq. 7 printed under it."""
    return (S ** (1.0 / k) - Sp) / (1.0 - Sp)


def threshold_for_sparsity(values: np.ndarray, sparsity: float) -> np.float32:
    """The threshold that turns the fraction `sparsity` of the entries into zeros: with the entries sorted,
    z = round(sparsity * n) of them must fall below it, so it is the z-th smallest value (+inf if z = n).
    Ties at that value are all kept, so the sparsity reached can be lower.  (The paper converts "with
    (S_p, S_z)" and gives no rule; this is the reading taken.)"""
    v = np.sort(np.asarray(values, dtype=np.float32).ravel())
    z = int(round(float(sparsity) * v.size))
    z = min(max(z, 0), v.size)
    return np.float32(np.inf) if z == v.size else v[z]


def alg1_search(W_bits: np.ndarray, theta: float, Mp: np.ndarray, Mz: np.ndarray, sp_step: float = 0.05,
                tol: float = 1e-3, max_iter: int = 24):
    """Algorithm 1 for one matrix (one tile), from the NMF factors on: the S_p sweep, S_z from Eq. 7 then
    adjusted by bisection until S_a is within `tol` of S, the cost of each candidate, the best one kept.

    W_bits: uint16 [m, n]; Mp: float32 [m, k]; Mz: float32 [k, n]; the index I is |W| >= theta and the
    target sparsity S is the sparsity of I.  The paper gives neither the step of the sweep, nor the
    tolerance of "S_a ~ S", nor the number of adjustments: sp_step, tol and max_iter are this reading's.
    Returns a dict with the best (Sp, Sz, Tp, Tz, cost, Sa) and the list of all candidates.
    """
    W_bits = _c(W_bits, np.uint16)
    m, n = W_bits.shape
    k = Mp.shape[1]
    Mp = _c(Mp, np.float32).reshape(1, m, k)
    Mz = _c(Mz, np.float32).reshape(1, k, n)
    full = np.ones((m, n), dtype=np.uint8)
    kept_i = index_cost(W_bits, theta, full, m, n)[0][0]
    S = 1.0 - kept_i / float(m * n)
    best, tried = None, []
    nsteps = int(round(1.0 / sp_step))
    for step in range(nsteps + 1):                       # "for S_p = 0.0 to 1.0"
        Sp = min(step * sp_step, 1.0)
        if Sp >= 1.0:
            Sz0 = 0.0                                    # Ip empty: Ia is empty whatever Iz is
        else:
            Sz0 = min(max(sz_from_eq7(S, Sp, k), 0.0), 1.0)   # "compute S_z using Eq. 7"
        Tp = threshold_for_sparsity(Mp, Sp)
        Ip = threshold(Mp, Tp).reshape(1, 1, m, k)
        lo, hi, Sz = 0.0, 1.0, Sz0
        for it in range(max_iter):                       # "repeat ... until S_a ~ S"
            Tz = threshold_for_sparsity(Mz, Sz)
            Iz = threshold(Mz, Tz).reshape(1, 1, k, n)   # "convert (Mp, Mz) into (Ip, Iz) w/ (S_p, S_z)"
            Ia = decode_mask(Ip, Iz, m, n)
            _, kept_a, lost, cost = index_cost(W_bits, theta, Ia, m, n)
            Sa = 1.0 - kept_a[0] / float(m * n)
            if abs(Sa - S) <= tol:
                break
            if Sa > S:                                   # too sparse: keep more of Iz ("adjust S_z depending on S_a - S")
                hi = Sz
            else:
                lo = Sz
            Sz = 0.5 * (lo + hi)
        cand = {"Sp": Sp, "Sz": Sz, "Tp": float(Tp), "Tz": float(Tz), "cost": float(cost[0]), "Sa": Sa, "lost": int(lost[0])}
        tried.append(cand)
        if best is None or best["cost"] > cand["cost"]:  # "if Cost_min > Cost"
            best = cand
    return {"S": S, "best": best, "tried": tried}


def nmf_multiplicative(W_bits: np.ndarray, Mp0: np.ndarray, Mz0: np.ndarray, tm: int, tn: int, iterations: int,
                       eps: float = 1e-9):
    """NMF of the magnitude matrix M = |W|, every tile on its own (Section 3.1), from given starting factors.

    The paper hands M to "an NMF library" and names no solver; the reading taken is the multiplicative update
    rule for the Frobenius objective ||M - Mp Mz||^2 that the paper's NMF reference gives: per iteration, first
        Mz <- Mz * (Mp^T M) / (Mp^T Mp Mz + eps)      then, with the new Mz,      Mp <- Mp * (M Mz^T) / (Mp Mz Mz^T + eps).
    W_bits: uint16 [rows, cols]; Mp0: [tiles, tm, k]; Mz0: [tiles, k, tn] (tiles in row-major grid order); positions of
    an edge tile outside the matrix count as zeros of M.  Plain numpy in fp64.  Returns (Mp, Mz)."""
    W_bits = _c(W_bits, np.uint16)
    rows, cols = W_bits.shape
    gr, gc = _grid(rows, cols, tm, tn)
    M_all = np.abs(bf16_to_f64(W_bits))
    Mp = np.array(Mp0, dtype=np.float64).copy()
    Mz = np.array(Mz0, dtype=np.float64).copy()
    if Mp.shape[0] != gr * gc or Mz.shape[0] != gr * gc or Mp.shape[1] != tm or Mz.shape[2] != tn or Mp.shape[2] != Mz.shape[1]:
        raise ValueError("factor shapes do not match the tile grid")
    for t in range(gr * gc):
        tr, tc = divmod(t, gc)
        M = np.zeros((tm, tn))
        blk = M_all[tr * tm:(tr + 1) * tm, tc * tn:(tc + 1) * tn]
        M[:blk.shape[0], :blk.shape[1]] = blk
        P, Z = Mp[t], Mz[t]
        for _ in range(iterations):
            Z = Z * (P.T @ M) / (P.T @ P @ Z + eps)
            P = P * (M @ Z.T) / (P @ (Z @ Z.T) + eps)
        Mp[t], Mz[t] = P, Z
    return Mp, Mz
