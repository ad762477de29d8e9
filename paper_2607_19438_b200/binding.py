"""Thin ctypes binding of the C-ABI library declared in include/qgemm.h.

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is used
for device memory and the current stream.  There is no fallback: if the shared library is missing or a
call returns an error code, a QGemmError is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqgemm_b200.so")

QG_Q8, QG_Q4 = 8, 4
MODE_PLAIN, MODE_GATE_UP_SILU, MODE_DOWN_WEIGHTED, MODE_DOWN_ACCUM_F32 = 0, 1, 2, 3
D_BF16, D_F32_ACC = 0, 1

EXPORTS = ["qg_create", "qg_destroy", "qg_strerror", "qg_poll_status", "qg_test_inject", "qg_test_gemv_mode", "qg_plan_dense", "qg_set_schedule", "qg_route_workspace_bytes",
           "qgemm_dense", "qgemm_small_m", "qgemm_dense_gate_up_silu", "prefill_attention",
           "qg_mx_scale_bytes", "qg_mx_quantize", "qg_mx_pack_weights", "qgemm_mx_dense",
           "moe_route", "moe_route_static", "moe_permute", "moe_grouped_qgemm", "moe_grouped_qgemm_gather", "moe_combine",
           "moe_combine_shared", "moe_router_logits",
           "qg_mx_grouped_scale_bytes", "qg_mx_quantize_grouped", "moe_grouped_qgemm_mx"]


class QGemmError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: error {code} ({strerror(code)})")
        self.code = code


_lib = None
_ctx = {}


def load():
    """Loads libqgemm_b200.so (built by `python -m paper_2607_19438_b200.build` or __graft_entry__.build())."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise QGemmError(-6, f"CUDA library not built: {LIB_PATH} is missing (run __graft_entry__.build())")
        lib = C.CDLL(LIB_PATH)
        lib.qg_strerror.restype = C.c_char_p
        lib.qg_strerror.argtypes = [C.c_int]
        lib.qg_route_workspace_bytes.restype = C.c_size_t
        lib.qg_route_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        lib.qg_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
        lib.qg_destroy.argtypes = [C.c_void_p]
        lib.qg_poll_status.argtypes = [C.c_void_p, C.c_void_p]
        lib.qg_test_inject.argtypes = [C.c_void_p, C.c_uint, C.c_int]
        lib.qg_test_gemv_mode.argtypes = [C.c_void_p, C.c_int]
        lib.qg_plan_dense.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        lib.qg_set_schedule.argtypes = [C.c_void_p, C.c_int, C.c_int]
        vp, ci = C.c_void_p, C.c_int
        lib.qgemm_dense.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp, vp]
        lib.qgemm_small_m.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp, vp]
        lib.qgemm_dense_gate_up_silu.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp, vp]
        ll = C.c_longlong
        lib.prefill_attention.argtypes = [vp, ci, ci, ci, ci, vp, ll, vp, ll, vp, ll, vp, ll, ci, C.c_float, vp]
        lib.qg_mx_scale_bytes.restype = C.c_size_t
        lib.qg_mx_scale_bytes.argtypes = [ci, ci]
        lib.qg_mx_quantize.argtypes = [vp, ci, ci, vp, vp, vp, vp]
        lib.qg_mx_pack_weights.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, vp]
        lib.qgemm_mx_dense.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, vp, vp]
        lib.moe_route.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp, ci, vp, C.c_size_t, vp]
        lib.moe_route_static.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp, ci, vp]
        lib.moe_permute.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp]
        lib.moe_grouped_qgemm.argtypes = [vp, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, ci, vp, vp]
        lib.moe_grouped_qgemm_gather.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, vp, vp, ci, vp, vp, vp, vp, vp, vp]
        lib.moe_combine.argtypes = [vp, ci, ci, ci, vp, ci, vp, vp, vp, vp]
        lib.moe_combine_shared.argtypes = [vp, ci, ci, ci, vp, ci, vp, vp, vp, vp, vp]
        lib.moe_router_logits.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp]
        lib.qg_mx_grouped_scale_bytes.restype = C.c_size_t
        lib.qg_mx_grouped_scale_bytes.argtypes = [ci, ci, ci]
        lib.qg_mx_quantize_grouped.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, vp]
        lib.moe_grouped_qgemm_mx.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        _lib = lib
    return _lib


def strerror(code: int) -> str:
    try:
        return load().qg_strerror(code).decode()
    except Exception:
        return "?"


def context(device: int | None = None):
    """The per-device library context (created on first use)."""
    if device is None:
        device = torch.cuda.current_device()
    if device not in _ctx:
        h = C.c_void_p()
        rc = load().qg_create(C.byref(h), int(device))
        if rc != 0:
            raise QGemmError(rc, "qg_create")
        _ctx[device] = h
    return _ctx[device]


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _check(rc, what):
    if rc != 0:
        raise QGemmError(rc, what)


def poll_status():
    """Synchronises the current stream and raises if a kernel recorded a device-side error."""
    _check(load().qg_poll_status(context(), _stream()), "qg_poll_status")


def poll_status_code() -> int:
    """Synchronises the current stream; returns (and clears) the device status word instead of raising."""
    return int(load().qg_poll_status(context(), _stream()))


def test_inject(wait_limit_polls: int = 0, skip_kblock: int = -1):
    """Testing hook: bounded-wait limit in polls (0 = default) and the k-block whose activation load the next GEMM
    launch leaves out (-1 = none)."""
    _check(load().qg_test_inject(context(), wait_limit_polls, skip_kblock), "qg_test_inject")


def test_gemv_mode(mode: int = 0):
    """Testing hook: kernel choice of qgemm_small_m (bit 0 no clusters, bit 1 always the ring kernel, bit 2 never)."""
    _check(load().qg_test_gemv_mode(context(), mode), "qg_test_gemv_mode")


def plan_dense(qbits, M, N, K):
    """(token tile, stream-K flag) qgemm_dense would use for this shape."""
    bt, sk = C.c_int(0), C.c_int(0)
    _check(load().qg_plan_dense(context(), qbits, M, N, K, C.byref(bt), C.byref(sk)), "qg_plan_dense")
    return bt.value, bool(sk.value)


def set_schedule(token_tile: int = 0, streamk_mode: int = -1):
    """Overrides the launch configuration (0 / -1 = the library's cost model); for sweeps and tests."""
    _check(load().qg_set_schedule(context(), token_tile, streamk_mode), "qg_set_schedule")


def route_workspace_bytes(M, E, k) -> int:
    return int(load().qg_route_workspace_bytes(M, E, k))


def qgemm_dense(qbits, A, Wq, Wscale, out=None):
    """A bf16 [M,K]; Wq int8 [N,K] / uint8 [N,K/2]; Wscale fp16 [N,K/32] -> bf16 [M,N]."""
    M, K = A.shape
    N = Wq.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    _check(load().qgemm_dense(context(), qbits, M, N, K, _ptr(A), _ptr(Wq), _ptr(Wscale), _ptr(out), _stream()),
           "qgemm_dense")
    return out


def qgemm_small_m(qbits, A, Wq, Wscale, out=None):
    """qgemm_dense for 1..16 tokens: the weight-streaming kernel."""
    M, K = A.shape
    N = Wq.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    _check(load().qgemm_small_m(context(), qbits, M, N, K, _ptr(A), _ptr(Wq), _ptr(Wscale), _ptr(out), _stream()),
           "qgemm_small_m")
    return out


def qgemm_dense_gate_up_silu(qbits, A, Wq, Wscale, out=None):
    """A bf16 [M,K]; Wq [2F,K(/2)] (gate rows then up rows) -> silu(gate) * up, bf16 [M,F]."""
    M, K = A.shape
    F = Wq.shape[0] // 2
    if out is None:
        out = torch.empty((M, F), dtype=torch.bfloat16, device=A.device)
    _check(load().qgemm_dense_gate_up_silu(context(), qbits, M, F, K, _ptr(A), _ptr(Wq), _ptr(Wscale), _ptr(out),
                                           _stream()), "qgemm_dense_gate_up_silu")
    return out


def prefill_attention(Q, K, V, Hq, Hkv, d, causal=True, scale=0.0, out=None):
    """Q bf16 [S, Hq*d], K / V bf16 [S, Hkv*d] (2-D views with unit column stride and any row stride, e.g. column blocks
    of a fused QKV projection's output) -> O bf16 [S, Hq*d]."""
    S = Q.shape[0]
    for t in (Q, K, V):
        assert t.dim() == 2 and t.stride(1) == 1 and t.dtype == torch.bfloat16
    if out is None:
        out = torch.empty((S, Hq * d), dtype=torch.bfloat16, device=Q.device)
    _check(load().prefill_attention(context(), S, Hq, Hkv, d, _ptr(Q), Q.stride(0), _ptr(K), K.stride(0), _ptr(V),
                                    V.stride(0), _ptr(out), out.stride(0), 1 if causal else 0, float(scale), _stream()),
           "prefill_attention")
    return out


def mx_quantize(X):
    """bf16 [rows, K] -> (E4M3 codes uint8 [rows, K], E8M0 scale bytes in the library's tiled order)."""
    rows, K = X.shape
    codes = torch.empty((rows, K), dtype=torch.uint8, device=X.device)
    sf = torch.empty(max(16, int(load().qg_mx_scale_bytes(rows, K))), dtype=torch.uint8, device=X.device)
    _check(load().qg_mx_quantize(context(), rows, K, _ptr(X), _ptr(codes), _ptr(sf), _stream()), "qg_mx_quantize")
    return codes, sf


def mx_pack_weights(qbits, Wq, Wscale):
    """Q8 / Q4 weights + fp16 scales -> (E4M3 codes uint8 [N, K], E8M0 scale bytes, tiled)."""
    N = Wq.shape[0]
    K = Wscale.shape[1] * 32
    codes = torch.empty((N, K), dtype=torch.uint8, device=Wq.device)
    sf = torch.empty(max(16, int(load().qg_mx_scale_bytes(N, K))), dtype=torch.uint8, device=Wq.device)
    _check(load().qg_mx_pack_weights(context(), qbits, N, K, _ptr(Wq), _ptr(Wscale), _ptr(codes), _ptr(sf), _stream()),
           "qg_mx_pack_weights")
    return codes, sf


def qgemm_mx_dense(A_codes, A_sf, W_codes, W_sf, out=None):
    """Block-scaled FP8 GEMM: codes uint8 [M, K] / [N, K], scale bytes tiled -> bf16 [M, N]."""
    M, K = A_codes.shape
    N = W_codes.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A_codes.device)
    _check(load().qgemm_mx_dense(context(), M, N, K, _ptr(A_codes), _ptr(A_sf), _ptr(W_codes), _ptr(W_sf), _ptr(out),
                                 _stream()), "qgemm_mx_dense")
    return out


def mx_quantize_grouped(X, offsets):
    """Sorted rows X bf16 [R, K], int32 offsets [E + 1] -> (codes uint8 [R, K], scale tiles laid out per segment)."""
    R, K = X.shape
    E = offsets.numel() - 1
    codes = torch.empty((R, K), dtype=torch.uint8, device=X.device)
    sf = torch.zeros(max(16, load().qg_mx_grouped_scale_bytes(R, E, K)), dtype=torch.uint8, device=X.device)
    _check(load().qg_mx_quantize_grouped(context(), R, E, K, _ptr(X), _ptr(offsets), _ptr(codes), _ptr(sf), _stream()),
           "qg_mx_quantize_grouped")
    return codes, sf


def moe_grouped_qgemm_mx(mode, A_codes, A_sf, offsets, W_codes, W_sf, N, topk_w=None, row_pair=None, out=None):
    """A_codes uint8 [R, K] with per-segment scale tiles; W_codes uint8 [E * N, K] with scale tiles (mx_pack_weights)."""
    R, K = A_codes.shape
    E = offsets.numel() - 1
    if out is None:
        out = torch.empty((R, N // 2 if mode == MODE_GATE_UP_SILU else N), dtype=torch.bfloat16, device=A_codes.device)
    _check(load().moe_grouped_qgemm_mx(context(), mode, R, E, N, K, _ptr(A_codes), _ptr(A_sf), _ptr(offsets), _ptr(W_codes),
                                       _ptr(W_sf), _ptr(topk_w), _ptr(row_pair), _ptr(out), _stream()), "moe_grouped_qgemm_mx")
    return out


def _route_outputs(M, E, k, H, dev, X, out):
    """The output tensors of a routing call: the caller's (`out`, a dict with the same keys) or fresh ones."""
    if out is not None:
        return out
    i32 = dict(dtype=torch.int32, device=dev)
    o = dict(topk_idx=torch.empty((M, k), **i32), topk_w=torch.empty((M, k), dtype=torch.float32, device=dev),
             counts=torch.empty(E, **i32), offsets=torch.empty(E + 1, **i32),
             row_pair=torch.empty(M * k, **i32), pair_row=torch.empty(M * k, **i32))
    if X is not None:
        o["Xperm"] = torch.empty((M * k, H), dtype=torch.bfloat16, device=dev)
    return o


def moe_route(logits, k, X=None, ws=None, out=None):
    """logits f32 [M,E] -> dict(topk_idx, topk_w, counts, offsets, row_pair, pair_row[, Xperm])."""
    M, E = logits.shape
    H = X.shape[1] if X is not None else 0
    out = _route_outputs(M, E, k, H, logits.device, X, out)
    need = route_workspace_bytes(M, E, k)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=logits.device)
    _check(load().moe_route(context(), M, E, k, _ptr(logits), _ptr(out["topk_idx"]), _ptr(out["topk_w"]),
                            _ptr(out["counts"]), _ptr(out["offsets"]), _ptr(out["row_pair"]), _ptr(out["pair_row"]),
                            _ptr(X), _ptr(out.get("Xperm")), H, _ptr(ws), ws.numel(), _stream()), "moe_route")
    return out


def moe_route_static(logits, k, X=None, out=None):
    """moe_route for callers that cannot supply scratch memory: the block histograms live in a fixed array inside
    the library (limit ceil(M/32)*E <= 65536, else QGemmError -8).  The output tensors are still the caller's: pass
    them as `out` (a dict with the keys moe_route returns) and this wrapper allocates nothing either; without `out`
    it allocates them for convenience.  Calls that overlap on the GPU share the array and would race."""
    M, E = logits.shape
    H = X.shape[1] if X is not None else 0
    out = _route_outputs(M, E, k, H, logits.device, X, out)
    _check(load().moe_route_static(context(), M, E, k, _ptr(logits), _ptr(out["topk_idx"]), _ptr(out["topk_w"]),
                                   _ptr(out["counts"]), _ptr(out["offsets"]), _ptr(out["row_pair"]),
                                   _ptr(out["pair_row"]), _ptr(X), _ptr(out.get("Xperm")), H, _stream()),
           "moe_route_static")
    return out


def moe_permute(X, row_pair, k, out=None):
    M, H = X.shape
    if out is None:
        out = torch.empty((M * k, H), dtype=torch.bfloat16, device=X.device)
    _check(load().moe_permute(context(), M, k, H, _ptr(X), _ptr(row_pair), _ptr(out), _stream()), "moe_permute")
    return out


def moe_grouped_qgemm(mode, qbits, Ain, offsets, Wq, Wscale, topk_w=None, row_pair=None, k=1, out=None, M=None):
    """Ain bf16 [R,K]; Wq [E,N,K(/2)]; Wscale fp16 [E,N,K/32]; see include/qgemm.h for the modes."""
    R, K = Ain.shape
    E, N = Wscale.shape[0], Wscale.shape[1]
    dev = Ain.device
    if out is None:
        if mode == MODE_GATE_UP_SILU:
            out = torch.empty((R, N // 2), dtype=torch.bfloat16, device=dev)
        elif mode == MODE_DOWN_ACCUM_F32:
            out = torch.zeros((M if M is not None else R // k, N), dtype=torch.float32, device=dev)
        else:
            out = torch.empty((R, N), dtype=torch.bfloat16, device=dev)
    _check(load().moe_grouped_qgemm(context(), mode, qbits, R, E, N, K, _ptr(Ain), _ptr(offsets), _ptr(Wq),
                                    _ptr(Wscale), _ptr(topk_w), _ptr(row_pair), k, _ptr(out), _stream()),
           "moe_grouped_qgemm")
    return out


def moe_grouped_qgemm_gather(mode, qbits, X, row_pair, k, offsets, Wq, Wscale, topk_w=None, out=None):
    """moe_grouped_qgemm whose input row r is X[row_pair[r] // k] (X bf16 [M,K] in token order)."""
    M, K = X.shape
    R = row_pair.numel()
    E, N = Wscale.shape[0], Wscale.shape[1]
    dev = X.device
    if out is None:
        if mode == MODE_GATE_UP_SILU:
            out = torch.empty((R, N // 2), dtype=torch.bfloat16, device=dev)
        elif mode == MODE_DOWN_ACCUM_F32:
            out = torch.zeros((M, N), dtype=torch.float32, device=dev)
        else:
            out = torch.empty((R, N), dtype=torch.bfloat16, device=dev)
    _check(load().moe_grouped_qgemm_gather(context(), mode, qbits, M, R, E, N, K, _ptr(X), _ptr(row_pair), k,
                                           _ptr(offsets), _ptr(Wq), _ptr(Wscale), _ptr(topk_w), _ptr(out), _stream()),
           "moe_grouped_qgemm_gather")
    return out


def moe_combine(D, pair_row, k, topk_w=None, d_kind=D_BF16, out=None, shared=None):
    """shared (bf16 [M, H], the shared expert's output) is added last when given (moe_combine_shared)."""
    if d_kind == D_F32_ACC:
        M, H = D.shape
    else:
        H = D.shape[1]
        M = D.shape[0] // k
    if out is None:
        out = torch.empty((M, H), dtype=torch.bfloat16, device=D.device)
    if shared is None:
        _check(load().moe_combine(context(), M, k, H, _ptr(D), d_kind, _ptr(pair_row), _ptr(topk_w), _ptr(out), _stream()),
               "moe_combine")
    else:
        _check(load().moe_combine_shared(context(), M, k, H, _ptr(D), d_kind, _ptr(pair_row), _ptr(topk_w), _ptr(shared),
                                         _ptr(out), _stream()), "moe_combine_shared")
    return out


def moe_router_logits(X, Wr, out=None):
    """X bf16 [M, H], Wr bf16 [E, H] -> fp32 logits [M, E], the input of moe_route."""
    M, H = X.shape
    E = Wr.shape[0]
    if out is None:
        out = torch.empty((M, E), dtype=torch.float32, device=X.device)
    _check(load().moe_router_logits(context(), M, H, E, _ptr(X), _ptr(Wr), _ptr(out), _stream()), "moe_router_logits")
    return out
