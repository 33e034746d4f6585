"""ctypes front end of the CPU oracle (``fkv_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
CPU-baseline leg import this package.  It compiles the C file with gcc on
first use, takes numpy arrays (bf16 tensors as ``uint16`` bit patterns) and
does no arithmetic of its own.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fkv_oracle.c")
_SO = os.path.join(_HERE, "libfkv_oracle.so")
_lib = None

RELU, SILU, GELU_TANH, SIGMOID = 0, 1, 2, 3


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.fkv_oracle_select.restype = ctypes.c_int
        _lib.fkv_oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().fkv_oracle_num_threads())


def score(K, V, A, W1, b1, W2, b2, act=RELU):
    """K, V: [n][D] uint16 (bf16 bits); A: [n][F] fp32; W1: [2D+F][H]. Returns phi [n] fp32."""
    K, pK = _c(K, np.uint16)
    V, pV = _c(V, np.uint16)
    A, pA = _c(A, np.float32)
    W1, pW1 = _c(W1, np.float32)
    b1, pb1 = _c(b1, np.float32)
    W2, pW2 = _c(W2, np.float32)
    n, D = K.shape
    F = A.shape[1] if A.ndim == 2 else 0
    H = W1.shape[1]
    assert V.shape == (n, D) and W1.shape[0] == 2 * D + F and b1.shape == (H,) and W2.reshape(-1).shape == (H,)
    phi = np.empty(n, np.float32)
    lib().fkv_oracle_score(pK, pV, pA, n, D, F, H, pW1, pb1, pW2, ctypes.c_float(float(b2)), int(act),
                           phi.ctypes.data_as(ctypes.c_void_p))
    return phi


def select(phi, B, R=0):
    """Kept slots (ascending int32) of one segment."""
    phi, pphi = _c(phi, np.float32)
    n = phi.shape[0]
    kept = np.empty(max(1, min(B, n)), np.int32)
    nk = lib().fkv_oracle_select(pphi, n, int(B), int(R), kept.ctypes.data_as(ctypes.c_void_p))
    return kept[:nk].copy()


def select_sampled(phi, B, R, noise):
    """Sampled eviction action: kept slots (ascending int32) and the candidate slots (slot order).

    noise: standard Gumbel draws, one per candidate in slot order (at least min(2 (n - B), n - r) of them).
    """
    phi, pphi = _c(phi, np.float32)
    noise, pnoise = _c(noise, np.float32)
    n = phi.shape[0]
    kept = np.empty(max(1, min(B, n)), np.int32)
    cand = np.empty(max(1, n), np.int32)
    ncand = ctypes.c_int32(0)
    need = 0 if n <= B else min(2 * (n - B), n - min(R, B))
    assert noise.shape[0] >= need, (noise.shape, need)
    lib().fkv_oracle_select_sampled.restype = ctypes.c_int
    nk = lib().fkv_oracle_select_sampled(pphi, n, int(B), int(R), pnoise, kept.ctypes.data_as(ctypes.c_void_p),
                                         cand.ctypes.data_as(ctypes.c_void_p), ctypes.byref(ncand))
    return kept[:nk].copy(), cand[:ncand.value].copy()


H2O_COLUMN, SNAPKV_COLUMN = 4, 0


def score_feature(A, g, column):
    """Baseline score (H2O: column 4, SnapKV: column 0): mean over the g heads of one feature column, fp32."""
    A, pA = _c(A, np.float32)
    n = A.shape[0]
    assert A.shape == (n, 6 * g) and 0 <= column < 6
    phi = np.empty(n, np.float32)
    lib().fkv_oracle_score_feature(pA, n, int(g), int(column), phi.ctypes.data_as(ctypes.c_void_p))
    return phi


def score_rkv(K, A, g, lambda_a=0.1, lambda_s=0.9, column=SNAPKV_COLUMN, rows=None):
    """R-KV baseline score (Appendix E.2; the similarity term is the oracle's own reading, see fkv_oracle.c):
    lambda_a * (window-8 attention, mean over heads) - lambda_s * max_{j != i} cos(k_i, k_j).
    K: [n][D] bf16 bits; A: [n][6g].  rows: optional int32 list of pairs to compute (else all)."""
    K, pK = _c(K, np.uint16)
    A, pA = _c(A, np.float32)
    n, D = K.shape
    assert A.shape == (n, 6 * g)
    if rows is None:
        phi = np.empty(n, np.float32)
        prow, nrows = ctypes.c_void_p(0), 0
    else:
        rows, prow = _c(rows, np.int32)
        nrows = rows.shape[0]
        phi = np.empty(nrows, np.float32)
    lib().fkv_oracle_score_rkv(pK, pA, n, D, int(g), int(column), ctypes.c_double(float(lambda_a)),
                               ctypes.c_double(float(lambda_s)), prow, nrows, phi.ctypes.data_as(ctypes.c_void_p))
    return phi


def golden(A, B, L):
    """Golden Eviction labels of one attention group.  A: [g][T][T] fp32 attention probabilities.

    Returns (alpha [M][T] future scores, kept [M][B - L] retained positions per eviction step).
    """
    A, pA = _c(A, np.float32)
    g, T, T2 = A.shape
    assert T == T2 and 0 < L < B
    M = max(0, (T - B + L - 1) // L - 1)
    alpha = np.zeros((max(M, 1), T), np.float32)
    kept = np.zeros((max(M, 1), B - L), np.int32)
    lib().fkv_oracle_golden.restype = ctypes.c_int
    m = lib().fkv_oracle_golden(pA, g, T, int(B), int(L), alpha.ctypes.data_as(ctypes.c_void_p),
                                kept.ctypes.data_as(ctypes.c_void_p))
    assert m == M
    return alpha[:M], kept[:M]


def golden_select(alpha, B, L):
    """Retained sets [M][B - L] of Golden Eviction from given future scores alpha [M][T]."""
    alpha, pa = _c(alpha, np.float32)
    M, T = alpha.shape
    kept = np.zeros((M, B - L), np.int32)
    lib().fkv_oracle_golden_select(pa, T, int(B), int(L), M, kept.ctypes.data_as(ctypes.c_void_p))
    return kept


def features(K, q, nvalid, A, scale=None, decay=0.9):
    """Attention features refreshed at the end of a chunk (Appendix B.1).

    K: [n][D] bf16 bits; q: [nq][g][D] bf16 bits (chronological); nvalid: [nq] pairs each query saw;
    A: [n][6g] fp32 features before the chunk.  Returns the new [n][6g] array.
    """
    K, pK = _c(K, np.uint16)
    q, pq = _c(q, np.uint16)
    nvalid, pnv = _c(nvalid, np.int32)
    A = np.array(A, dtype=np.float32, order="C", copy=True)
    n, D = K.shape
    nq, g, _ = q.shape
    assert A.shape == (n, 6 * g) and nvalid.shape == (nq,)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    lib().fkv_oracle_features(pK, n, D, g, pq, nq, pnv, ctypes.c_double(float(scale)), ctypes.c_double(float(decay)),
                              A.ctypes.data_as(ctypes.c_void_p))
    return A


def compact(K, V, A, pos, kept):
    K, pK = _c(K, np.uint16)
    V, pV = _c(V, np.uint16)
    A, pA = _c(A, np.float32)
    pos, ppos = _c(pos, np.int32)
    kept, pkept = _c(kept, np.int32)
    n, D = K.shape
    F = A.shape[1]
    nk = kept.shape[0]
    K2, V2 = np.empty((nk, D), np.uint16), np.empty((nk, D), np.uint16)
    A2, pos2 = np.empty((nk, F), np.float32), np.empty(nk, np.int32)
    lib().fkv_oracle_compact(pK, pV, pA, ppos, D, F, pkept, nk, K2.ctypes.data_as(ctypes.c_void_p),
                             V2.ctypes.data_as(ctypes.c_void_p), A2.ctypes.data_as(ctypes.c_void_p),
                             pos2.ctypes.data_as(ctypes.c_void_p))
    return K2, V2, A2, pos2


def attend(q, K, V, scale=None):
    """q: [g][D] bf16 bits; K, V: [n][D]. Returns (out bf16 bits [g][D], out float64 [g][D])."""
    q, pq = _c(q, np.uint16)
    K, pK = _c(K, np.uint16)
    V, pV = _c(V, np.uint16)
    g, D = q.shape
    n = K.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty((g, D), np.uint16)
    out64 = np.empty((g, D), np.float64)
    lib().fkv_oracle_attend(pq, pK, pV, n, g, D, ctypes.c_double(float(scale)), out.ctypes.data_as(ctypes.c_void_p),
                            out64.ctypes.data_as(ctypes.c_void_p))
    return out, out64


def evict_batch(K, V, A, pos, off, n, B, R, W1, b1, W2, b2, act=RELU):
    """score -> select -> compact over many segments packed densely (offsets in pairs).

    Returns phi (packed), kept (packed, first nkept[i] entries of each segment valid),
    nkept, and the compacted K2, V2, A2, pos2 (packed the same way).
    """
    K, pK = _c(K, np.uint16)
    V, pV = _c(V, np.uint16)
    A, pA = _c(A, np.float32)
    pos, ppos = _c(pos, np.int32)
    off, poff = _c(off, np.int64)
    n, pn = _c(n, np.int32)
    B, pB = _c(B, np.int32)
    W1, pW1 = _c(W1, np.float32)
    b1, pb1 = _c(b1, np.float32)
    W2, pW2 = _c(W2, np.float32)
    b2, pb2 = _c(b2, np.float32)
    nseg = n.shape[0]
    total, D = K.shape
    F = A.shape[1]
    H = W1.shape[-1]
    assert W1.shape == (nseg, 2 * D + F, H)
    phi = np.empty(total, np.float32)
    kept = np.full(total, -1, np.int32)
    nkept = np.empty(nseg, np.int32)
    K2, V2 = np.zeros_like(K), np.zeros_like(V)
    A2, pos2 = np.zeros_like(A), np.zeros_like(pos)
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    lib().fkv_oracle_evict_batch(nseg, poff, pn, pB, int(R), D, F, H, int(act), pK, pV, pA, ppos, pW1, pb1, pW2, pb2,
                                 p(phi), p(kept), p(nkept), p(K2), p(V2), p(A2), p(pos2))
    return phi, kept, nkept, K2, V2, A2, pos2


def attend_batch(q, K, V, off, n, scale=None):
    """q: [nseg][g][D]; K, V packed [total][D]. Returns out bf16 bits [nseg][g][D]."""
    q, pq = _c(q, np.uint16)
    K, pK = _c(K, np.uint16)
    V, pV = _c(V, np.uint16)
    off, poff = _c(off, np.int64)
    n, pn = _c(n, np.int32)
    nseg, g, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty((nseg, g, D), np.uint16)
    lib().fkv_oracle_attend_batch(nseg, poff, pn, g, D, ctypes.c_double(float(scale)), pq, pK, pV,
                                  out.ctypes.data_as(ctypes.c_void_p))
    return out
