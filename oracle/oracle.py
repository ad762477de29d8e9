"""ctypes loader and numpy wrappers for the fp64 CPU oracle (oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's CPU-baseline
leg.  It imports nothing from the CUDA package and the CUDA package imports nothing from here.
All arithmetic lives in oracle.cpp; this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.cpp with g++ (-O2, OpenMP) into liboracle.so next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def bf16_to_f64(bits):
    b = _c(bits, np.uint16)
    out = np.empty(b.shape, np.float64)
    lib().orc_bf16_to_f64(C.c_int64(b.size), _p(b), _p(out))
    return out


def f16_to_f64(bits):
    b = _c(bits, np.uint16)
    out = np.empty(b.shape, np.float64)
    lib().orc_f16_to_f64(C.c_int64(b.size), _p(b), _p(out))
    return out


def f64_to_bf16(x):
    x = _c(x, np.float64)
    out = np.empty(x.shape, np.uint16)
    lib().orc_f64_to_bf16(C.c_int64(x.size), _p(x), _p(out))
    return out


def _wq(qbits, Wq):
    return _c(Wq, np.int8 if qbits == 8 else np.uint8)


def dequant(qbits, Wq, Ws):
    """Wq [N,K] int8 or [N,K/2] uint8, Ws fp16 bits [N,K/32] -> fp64 [N,K]."""
    Wq, Ws = _wq(qbits, Wq), _c(Ws, np.uint16)
    N = Wq.shape[0]
    K = Ws.shape[1] * 32
    w = np.empty((N, K), np.float64)
    lib().orc_dequant(C.c_int(qbits), C.c_int64(N), C.c_int64(K), _p(Wq), _p(Ws), _p(w))
    return w


def qgemm_dense(qbits, A, Wq, Ws):
    """A bf16 bits [M,K] -> fp64 C [M,N]."""
    A, Wq, Ws = _c(A, np.uint16), _wq(qbits, Wq), _c(Ws, np.uint16)
    M, K = A.shape
    N = Wq.shape[0]
    assert Ws.shape == (N, K // 32)
    out = np.empty((M, N), np.float64)
    lib().orc_qgemm_dense(C.c_int(qbits), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(A), _p(Wq), _p(Ws), _p(out))
    return out


def qgemm_dense_sample(qbits, A, Wq, Ws, rows, cols):
    A, Wq, Ws = _c(A, np.uint16), _wq(qbits, Wq), _c(Ws, np.uint16)
    rows, cols = _c(rows, np.int64), _c(cols, np.int64)
    M, K = A.shape
    N = Wq.shape[0]
    out = np.empty(rows.shape, np.float64)
    lib().orc_qgemm_dense_sample(C.c_int(qbits), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(A), _p(Wq), _p(Ws),
                                 C.c_int64(rows.size), _p(rows), _p(cols), _p(out))
    return out


def route(logits, k):
    """logits f32 [M,E] -> (idx int32 [M,k], w fp64 [M,k], w32 f32 [M,k])."""
    l = _c(logits, np.float32)
    M, E = l.shape
    idx = np.empty((M, k), np.int32)
    w = np.empty((M, k), np.float64)
    w32 = np.empty((M, k), np.float32)
    lib().orc_route(C.c_int64(M), C.c_int(E), C.c_int(k), _p(l), _p(idx), _p(w), _p(w32))
    return idx, w, w32


def counts_offsets(idx, E):
    idx = _c(idx, np.int32)
    counts = np.empty(E, np.int32)
    offsets = np.empty(E + 1, np.int32)
    lib().orc_counts_offsets(C.c_int64(idx.size), C.c_int(E), _p(idx), _p(counts), _p(offsets))
    return counts, offsets


def permutation(idx, offsets):
    idx, offsets = _c(idx, np.int32), _c(offsets, np.int32)
    R = idx.size
    row_pair = np.empty(R, np.int32)
    pair_row = np.empty(R, np.int32)
    lib().orc_permutation(C.c_int64(R), C.c_int(offsets.size - 1), _p(idx), _p(offsets), _p(row_pair), _p(pair_row))
    return row_pair, pair_row


def permute(X, row_pair, k):
    X, row_pair = _c(X, np.uint16), _c(row_pair, np.int32)
    H = X.shape[1]
    Xp = np.empty((row_pair.size, H), np.uint16)
    lib().orc_permute(C.c_int64(row_pair.size), C.c_int(k), C.c_int64(H), _p(X), _p(row_pair), _p(Xp))
    return Xp


def grouped_gemm(qbits, Ain, offsets, Wq, Ws):
    """Ain fp64 [R,K]; Wq [E,N,K(/2)]; Ws fp16 bits [E,N,K/32] -> fp64 [R,N]."""
    Ain, offsets, Wq, Ws = _c(Ain, np.float64), _c(offsets, np.int32), _wq(qbits, Wq), _c(Ws, np.uint16)
    R, K = Ain.shape
    E, N = Ws.shape[0], Ws.shape[1]
    assert Ws.shape[2] * 32 == K and offsets.size == E + 1
    out = np.zeros((R, N), np.float64)
    lib().orc_grouped_gemm(C.c_int(qbits), C.c_int64(R), C.c_int(E), C.c_int64(N), C.c_int64(K), _p(Ain),
                           _p(offsets), _p(Wq), _p(Ws), _p(out))
    return out


def silu_mul(GU):
    GU = _c(GU, np.float64)
    R, F2 = GU.shape
    out = np.empty((R, F2 // 2), np.float64)
    lib().orc_silu_mul(C.c_int64(R), C.c_int64(F2 // 2), _p(GU), _p(out))
    return out


def combine(D, pair_row, k, w=None):
    D, pair_row = _c(D, np.float64), _c(pair_row, np.int32)
    M = pair_row.size // k
    H = D.shape[1]
    y = np.empty((M, H), np.float64)
    wp = _p(_c(w, np.float64)) if w is not None else None
    lib().orc_combine(C.c_int64(M), C.c_int(k), C.c_int64(H), _p(D), _p(pair_row), wp, _p(y))
    return y


def combine_shared(D, pair_row, k, shared, w=None):
    """combine() plus the shared expert's output row (a dense FFN every token passes through), added last."""
    D, pair_row, shared = _c(D, np.float64), _c(pair_row, np.int32), _c(shared, np.float64)
    M = pair_row.size // k
    H = D.shape[1]
    y = np.empty((M, H), np.float64)
    wp = _p(_c(w, np.float64)) if w is not None else None
    lib().orc_combine_shared(C.c_int64(M), C.c_int(k), C.c_int64(H), _p(D), _p(pair_row), wp, _p(shared), _p(y))
    return y


def router_logits(X, Wr):
    """Router projection (hidden -> experts) that feeds route(): L = X Wr^T, X [M, H] and Wr [E, H] as doubles."""
    X, Wr = _c(X, np.float64), _c(Wr, np.float64)
    M, H = X.shape
    E = Wr.shape[0]
    L = np.empty((M, E), np.float64)
    lib().orc_router_logits(C.c_int64(M), C.c_int64(H), C.c_int64(E), _p(X), _p(Wr), _p(L))
    return L


def moe_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k):
    """End-to-end MoE layer with no intermediate rounding; returns a dict of every stage."""
    E = logits.shape[1]
    idx, w, w32 = route(logits, k)
    counts, offsets = counts_offsets(idx, E)
    row_pair, pair_row = permutation(idx, offsets)
    Xp = permute(X, row_pair, k)
    GU = grouped_gemm(qbits, bf16_to_f64(Xp), offsets, W1q, W1s)
    Hh = silu_mul(GU)
    Dn = grouped_gemm(qbits, Hh, offsets, W2q, W2s)
    y = combine(Dn, pair_row, k, w)
    return dict(idx=idx, w=w, w32=w32, counts=counts, offsets=offsets, row_pair=row_pair, pair_row=pair_row,
                Xp=Xp, GU=GU, Hh=Hh, Dn=Dn, y=y)


def attention(Q, K, V, Hq, Hkv, d, causal=True, scale=None, qpos=None):
    """Q bf16 bits [S, Hq*d], K / V bf16 bits [S, Hkv*d] (any row stride: pass 2-D views of a wider array) -> fp64
    [nq, Hq*d] for the query positions qpos (all if None).  softmax(scale * Q K^T) V per head, keys j <= i if causal,
    query head h uses key/value head h // (Hq // Hkv); scale defaults to 1 / sqrt(d)."""
    Q, K, V = (np.asarray(x) for x in (Q, K, V))
    assert Q.dtype == np.uint16 and K.dtype == np.uint16 and V.dtype == np.uint16
    S = Q.shape[0]
    for x in (Q, K, V):
        assert x.strides[1] == 2, "rows must be contiguous"
    qpos = np.arange(S, dtype=np.int64) if qpos is None else _c(qpos, np.int64)
    out = np.empty((qpos.size, Hq * d), np.float64)
    scale = 1.0 / np.sqrt(d) if scale is None else float(scale)
    lib().orc_attention(C.c_int64(S), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), _p(Q), C.c_int64(Q.strides[0] // 2), _p(K),
                        C.c_int64(K.strides[0] // 2), _p(V), C.c_int64(V.strides[0] // 2), C.c_double(scale),
                        C.c_int(1 if causal else 0), C.c_int64(qpos.size), _p(qpos), _p(out))
    return out


def e4m3_to_f64(codes):
    c = _c(codes, np.uint8)
    out = np.empty(c.shape, np.float64)
    lib().orc_e4m3_to_f64(C.c_int64(c.size), _p(c), _p(out))
    return out


def mx_quantize(x):
    """x fp64 [rows, K] -> (E4M3 codes uint8 [rows, K], E8M0 scale bytes uint8 [rows, K/32]); blocks of 32 along K."""
    x = _c(x, np.float64)
    rows, K = x.shape
    assert K % 32 == 0
    codes = np.empty((rows, K), np.uint8)
    sf = np.empty((rows, K // 32), np.uint8)
    lib().orc_mx_quantize(C.c_int64(rows), C.c_int64(K), _p(x), _p(codes), _p(sf))
    return codes, sf


def mx_gemm(a, asf, w, wsf):
    """C[m, n] = sum_k (a[m,k] 2^(asf[m,k/32]-127)) (w[n,k] 2^(wsf[n,k/32]-127)), fp64; scale bytes in plain layout."""
    a, asf, w, wsf = _c(a, np.uint8), _c(asf, np.uint8), _c(w, np.uint8), _c(wsf, np.uint8)
    M, K = a.shape
    N = w.shape[0]
    out = np.empty((M, N), np.float64)
    lib().orc_mx_gemm(C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(a), _p(asf), _p(w), _p(wsf), _p(out))
    return out


def mx_grouped_gemm(a, asf, offsets, w, wsf):
    """mx_gemm per expert segment: rows offsets[e] .. offsets[e+1] of (a, asf) against expert e's (w[e], wsf[e])."""
    a, asf = _c(a, np.uint8), _c(asf, np.uint8)
    E, N = w.shape[0], w.shape[1]
    out = np.zeros((a.shape[0], N), np.float64)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi > lo:
            out[lo:hi] = mx_gemm(a[lo:hi], asf[lo:hi], w[e], wsf[e])
    return out
