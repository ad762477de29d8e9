"""Seeded synthetic inputs for the quantised prefill GEMM path (dense and MoE).

This module is harness code shared by the CPU oracle's tests and by the CUDA
path's tests and benchmark, so that both sides see identical bits.  It holds no
arithmetic of the method itself (no dequantisation, no matrix product, no
routing): it only draws numbers and stores them in the interchange formats

* activations: bf16 bit patterns (uint16), N(0,1) rounded to nearest-even;
* Q8 weights : int8, uniform in [-127, 127], row-major [N, K];
* Q4 weights : uint8, two 4-bit codes per byte, every code uniform in [0, 15]
               (the code of a weight q in [-8, 7] is q + 8), row-major [N, K/2];
* scales     : fp16 bit patterns (uint16), |N(0, sigma=0.02)| / qmax, [N, K/32];
* router logits: float32 N(0,1), optionally with a constant added to a "hot"
               subset of experts so that the assignment histogram is skewed.

Every element is a pure function of (seed, tensor id, element index): a 64-bit
mixing hash (counter-based), so tensors can be generated in slices and in any
order.  Normals use the Box-Muller transform in fp64.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_TWO53 = float(1 << 53)

# Tensor ids used by the workload builders below (any distinct integers do).
TID_A, TID_WQ, TID_WS, TID_LOGITS, TID_X, TID_W1Q, TID_W1S, TID_W2Q, TID_W2S = range(1, 10)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def hash_u64(seed: int, tid: int, n: int, start: int = 0, lane: int = 0) -> np.ndarray:
    """n 64-bit words; word i depends only on (seed, tid, lane, start + i)."""
    with np.errstate(over="ignore"):
        key = _mix(np.array([(seed * 0x100000001B3 + tid * 0x1000193 + lane * 0x9E37 + 0x632BE59BD9B4E019)
                             & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))[0]
        idx = np.arange(start, start + n, dtype=np.uint64)
        return _mix(_mix(idx * _GOLDEN + key) + key)


def uniform01(seed: int, tid: int, n: int, start: int = 0, lane: int = 0) -> np.ndarray:
    """fp64 uniforms in (0, 1)."""
    u = hash_u64(seed, tid, n, start, lane) >> np.uint64(11)
    return (u.astype(np.float64) + 0.5) / _TWO53


def normal(seed: int, tid: int, n: int, start: int = 0) -> np.ndarray:
    """fp64 standard normals (Box-Muller, one normal per pair of uniforms)."""
    u1 = uniform01(seed, tid, n, start, lane=0)
    u2 = uniform01(seed, tid, n, start, lane=1)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def activations(M: int, K: int, seed: int = 0, tid: int = TID_A) -> np.ndarray:
    """bf16 bits [M, K], N(0,1)."""
    return f32_to_bf16_bits(normal(seed, tid, M * K).astype(np.float32)).reshape(M, K)


def weights_q8(N: int, K: int, seed: int = 0, tid: int = TID_WQ) -> np.ndarray:
    """int8 [N, K], uniform over the 255 values -127..127."""
    n = N * K
    words = hash_u64(seed, tid, (n + 3) // 4)
    lanes = words.view(np.uint16).astype(np.uint32)          # four 16-bit lanes per word
    q = ((lanes * np.uint32(255)) >> np.uint32(16)).astype(np.int16) - 127
    return q[:n].astype(np.int8).reshape(N, K)


def weights_q4(N: int, K: int, seed: int = 0, tid: int = TID_WQ) -> np.ndarray:
    """uint8 [N, K/2]; both 4-bit codes of every byte are uniform in 0..15."""
    assert K % 2 == 0
    n = N * (K // 2)
    words = hash_u64(seed, tid, (n + 7) // 8)
    return words.view(np.uint8)[:n].copy().reshape(N, K // 2)


def scales(N: int, KB: int, qmax: int, seed: int = 0, tid: int = TID_WS, sigma: float = 0.02) -> np.ndarray:
    """fp16 bits [N, KB]: |N(0, sigma)| / qmax rounded to fp16 (subnormals kept)."""
    s = np.abs(normal(seed, tid, N * KB) * sigma) / float(qmax)
    return s.astype(np.float16).view(np.uint16).reshape(N, KB)


def router_logits(M: int, E: int, seed: int = 0, tid: int = TID_LOGITS, hot_bias: float = 0.0,
                  hot_stride: int = 4) -> np.ndarray:
    """float32 [M, E] N(0,1); experts with e % hot_stride == 0 get +hot_bias."""
    l = normal(seed, tid, M * E).reshape(M, E)
    if hot_bias != 0.0:
        l[:, ::hot_stride] += hot_bias
    return l.astype(np.float32)


# Bias that makes the hot quarter of the experts receive about 60 % of the top-8-of-128 assignments.
SKEW_HOT_BIAS = 0.80


def dense_problem(qbits: int, M: int, N: int, K: int, seed: int = 0, tid_base: int = 0):
    """(A bf16 bits [M,K], Wq, Wscale fp16 bits [N,K/32]) for one dense projection."""
    assert K % 32 == 0 and qbits in (4, 8)
    A = activations(M, K, seed, TID_A + tid_base)
    if qbits == 8:
        Wq = weights_q8(N, K, seed, TID_WQ + tid_base)
        Ws = scales(N, K // 32, 127, seed, TID_WS + tid_base)
    else:
        Wq = weights_q4(N, K, seed, TID_WQ + tid_base)
        Ws = scales(N, K // 32, 7, seed, TID_WS + tid_base)
    return A, Wq, Ws


def moe_problem(qbits: int, M: int, H: int, E: int, F: int, seed: int = 0, skewed: bool = False):
    """Inputs of one MoE layer: logits f32 [M,E], X bf16 bits [M,H],
    W1 (gate rows 0..F-1, up rows F..2F-1) [E,2F,H] + scales [E,2F,H/32],
    W2 [E,H,F] + scales [E,H,F/32] (Q4 packs two codes per byte along the last axis)."""
    assert H % 32 == 0 and F % 32 == 0 and qbits in (4, 8)
    logits = router_logits(M, E, seed, TID_LOGITS, SKEW_HOT_BIAS if skewed else 0.0)
    X = activations(M, H, seed, TID_X)
    qmax = 127 if qbits == 8 else 7
    gen = weights_q8 if qbits == 8 else weights_q4
    W1q = gen(E * 2 * F, H, seed, TID_W1Q).reshape(E, 2 * F, -1)
    W1s = scales(E * 2 * F, H // 32, qmax, seed, TID_W1S).reshape(E, 2 * F, H // 32)
    W2q = gen(E * H, F, seed, TID_W2Q).reshape(E, H, -1)
    W2s = scales(E * H, F // 32, qmax, seed, TID_W2S).reshape(E, H, F // 32)
    return logits, X, W1q, W1s, W2q, W2s


def mx_scale_tiles(plain: np.ndarray) -> np.ndarray:
    """Scale bytes [rows, K/32] -> the library's tiled order (a pure permutation; rows padded to a multiple of 128 with
    the byte 127 = 2^0, K a multiple of 128): tile (rows 128 t .. 128 t + 127, four consecutive 32-blocks c) is 512
    contiguous bytes, byte (r % 32) * 16 + (r // 32) * 4 + c for row r of the tile."""
    rows, kb = plain.shape
    assert kb % 4 == 0
    rp = (rows + 127) // 128 * 128
    full = np.full((rp, kb), 127, np.uint8)
    full[:rows] = plain
    t = full.reshape(rp // 128, 4, 32, kb // 4, 4)            # [tile, q, r, chunk, c]
    return np.ascontiguousarray(t.transpose(0, 3, 2, 1, 4)).reshape(-1)    # [tile, chunk, r, q, c]


def mx_scale_tiles_grouped(plain: np.ndarray, offsets: np.ndarray) -> np.ndarray:
    """mx_scale_tiles per expert segment: the rows of segment e (offsets[e] .. offsets[e+1]) are tiled on their own, so a
    segment's tiles start at its first row; the tiles of all segments follow one another (empty segments have none)."""
    parts = [mx_scale_tiles(plain[offsets[e]:offsets[e + 1]]) for e in range(len(offsets) - 1) if offsets[e + 1] > offsets[e]]
    return np.concatenate(parts) if parts else np.zeros(0, np.uint8)


def mx_scale_plain(tiles: np.ndarray, rows: int, K: int) -> np.ndarray:
    """Inverse of mx_scale_tiles."""
    kb = K // 32
    rp = (rows + 127) // 128 * 128
    t = np.asarray(tiles, np.uint8).reshape(rp // 128, kb // 4, 32, 4, 4)   # [tile, chunk, r, q, c]
    return np.ascontiguousarray(t.transpose(0, 3, 2, 1, 4)).reshape(rp, kb)[:rows]
