"""Seeded random small shapes through every GPU entry point against the oracle: ragged sizes, odd segment layouts and
value patterns the hand-picked cases do not enumerate.  Sizes are small enough for the fp64 oracle to take well under a
second per case."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def _rng(i):
    return np.random.default_rng(1000 + i)


@pytest.mark.parametrize("i", range(12))
def test_fuzz_dense(i):
    r = _rng(i)
    qbits = int(r.choice([4, 8]))
    M = int(r.integers(1, 700)); N = 8 * int(r.integers(1, 120)); K = 256 * int(r.integers(1, 5))
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=i)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.qgemm_dense(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    util.assert_close(util.host_bf16_f64(g.t), orc.qgemm_dense(qbits, A, Wq, Ws), f"dense q{qbits} {M}x{N}x{K}")
    if M <= 16:
        out = qg.qgemm_small_m(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
        util.assert_close(util.host_bf16_f64(out), orc.qgemm_dense(qbits, A, Wq, Ws), "small-M")


@pytest.mark.parametrize("i", range(12))
def test_fuzz_grouped(i):
    """Random segment lengths (many empty, some longer than two token tiles), every epilogue, both token tiles."""
    r = _rng(100 + i)
    qbits = int(r.choice([4, 8]))
    E = int(r.integers(1, 12)); K = 256 * int(r.integers(1, 3))
    mode = int(r.choice([qg.MODE_PLAIN, qg.MODE_GATE_UP_SILU, qg.MODE_DOWN_WEIGHTED]))
    N = 128 * int(r.integers(1, 6)) if mode == qg.MODE_GATE_UP_SILU else 8 * int(r.integers(1, 60))
    counts = r.choice([0, 0, 1, 7, 33, 128, 129, 200, 450], size=E).astype(np.int32)
    if counts.sum() == 0:
        counts[0] = 5
    offsets = np.zeros(E + 1, np.int32); offsets[1:] = np.cumsum(counts)
    R = int(offsets[-1])
    A = synth.activations(R, K, seed=i, tid=61)
    gen = synth.weights_q8 if qbits == 8 else synth.weights_q4
    Wq = gen(E * N, K, i, 62).reshape(E, N, -1)
    Ws = synth.scales(E * N, K // 32, 127 if qbits == 8 else 7, i, 63).reshape(E, N, K // 32)
    row_pair = r.permutation(R).astype(np.int32)
    w = r.uniform(0.1, 1.0, R).astype(np.float32)
    qg.set_schedule(int(r.choice([0, 128, 192])), -1)
    try:
        cols = N // 2 if mode == qg.MODE_GATE_UP_SILU else N
        g = util.Guarded((R, cols), torch.bfloat16)
        qg.moe_grouped_qgemm(mode, qbits, util.dev_bf16(A), util.dev(offsets), util.dev(Wq), util.dev_f16(Ws),
                             topk_w=util.dev(w), row_pair=util.dev(row_pair), k=1, out=g.t)
        qg.poll_status()
    finally:
        qg.set_schedule(0, -1)
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.grouped_gemm(qbits, orc.bf16_to_f64(A), offsets, Wq, Ws)
    if mode == qg.MODE_GATE_UP_SILU:
        ref = orc.silu_mul(ref)
    elif mode == qg.MODE_DOWN_WEIGHTED:
        ref = ref * w[row_pair].astype(np.float64)[:, None]
    util.assert_close(util.host_bf16_f64(g.t), ref, f"grouped mode {mode} q{qbits} E={E} N={N} K={K} counts={counts.tolist()}")


@pytest.mark.parametrize("i", range(10))
def test_fuzz_attention(i):
    """Random lengths, head counts and masks; every third case has keys whose scores grow along the sequence, so the
    running maximum keeps moving (the exponent reference is moved and the output rescaled many times)."""
    r = _rng(200 + i)
    d = int(r.choice([64, 128])); Hkv = int(r.integers(1, 4)); Hq = Hkv * int(r.integers(1, 4))
    S = int(r.integers(1, 900)); causal = bool(r.integers(0, 2))
    W = (Hq + 2 * Hkv) * d
    x = synth.bf16_bits_to_f32(synth.activations(S, W, seed=i, tid=71)).copy()
    if i % 3 == 0:
        x[:, Hq * d:(Hq + Hkv) * d] *= np.linspace(0.2, 6.0, S, dtype=np.float32)[:, None]       # later keys score higher
    bits = synth.f32_to_bf16_bits(x)
    dev = util.dev_bf16(bits)
    sl = lambda t: (t[:, :Hq * d], t[:, Hq * d:(Hq + Hkv) * d], t[:, (Hq + Hkv) * d:])
    scale = float(r.choice([0.0, 0.05, 0.3]))
    g = util.Guarded((S, Hq * d), torch.bfloat16)
    qg.prefill_attention(*sl(dev), Hq, Hkv, d, causal=causal, scale=scale, out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.attention(*sl(bits), Hq, Hkv, d, causal=causal, scale=None if scale == 0.0 else scale)
    util.assert_close(util.host_bf16_f64(g.t), ref, f"attention S={S} Hq={Hq} Hkv={Hkv} d={d} causal={causal} scale={scale}")


@pytest.mark.parametrize("i", range(8))
def test_fuzz_mx(i):
    r = _rng(300 + i)
    M = int(r.integers(1, 600)); N = 8 * int(r.integers(1, 90)); K = 128 * int(r.integers(1, 9))
    a, asf = orc.mx_quantize(r.standard_normal((M, K)) * float(r.choice([1e-3, 1.0, 50.0])))
    w, wsf = orc.mx_quantize(r.standard_normal((N, K)) * 0.02)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.qgemm_mx_dense(util.dev(a), util.dev(synth.mx_scale_tiles(asf)), util.dev(w), util.dev(synth.mx_scale_tiles(wsf)), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    util.assert_close(util.host_bf16_f64(g.t), orc.mx_gemm(a, asf, w, wsf), f"mx {M}x{N}x{K}")


@pytest.mark.parametrize("i", range(8))
def test_fuzz_route_and_layer(i):
    r = _rng(400 + i)
    qbits = int(r.choice([4, 8])); E = int(r.choice([2, 5, 16, 40])); k = int(r.integers(1, min(E, 8) + 1))
    M = int(r.integers(1, 300)); H = 256 * int(r.integers(1, 3)); F = 256 * int(r.integers(1, 3))
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=i, skewed=bool(i % 2))
    if i % 4 == 0:
        logits[:, : E // 2] = logits[:, E - E // 2:]                  # exact ties between pairs of experts
    dX = util.dev_bf16(X)
    ro = qg.moe_route(util.dev(logits), k, X=dX)
    Hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, qbits, ro["Xperm"], ro["offsets"], util.dev(W1q), util.dev_f16(W1s))
    Dw = qg.moe_grouped_qgemm(qg.MODE_DOWN_WEIGHTED, qbits, Hh, ro["offsets"], util.dev(W2q), util.dev_f16(W2s),
                              topk_w=ro["topk_w"].view(-1), row_pair=ro["row_pair"], k=k)
    y = qg.moe_combine(Dw, ro["pair_row"], k)
    qg.poll_status()
    o = orc.moe_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k)
    assert np.array_equal(ro["topk_idx"].cpu().numpy().reshape(o["idx"].shape), o["idx"])
    assert np.array_equal(ro["row_pair"].cpu().numpy(), o["row_pair"]) and np.array_equal(ro["offsets"].cpu().numpy(), o["offsets"])
    util.assert_close(util.host_bf16_f64(y), o["y"], f"layer q{qbits} M={M} H={H} E={E} F={F} k={k}")


@pytest.mark.parametrize("i", range(24))
def test_fuzz_small_m(i):
    """Random ragged shapes through qgemm_small_m with the kernel choice forced in turn (library's choice, ring kernel
    with clusters, ring kernel with the scratch): tiles that end inside a 128-row block, K that does not divide into
    equal slices or phases, every token count."""
    r = _rng(500 + i)
    qbits = int(r.choice([4, 8]))
    M = int(r.integers(1, 17)); N = 8 * int(r.integers(1, 400)); K = 256 * int(r.integers(1, 25))
    mode = (0, 2, 3)[i % 3]
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=i)
    g = util.Guarded((M, N), torch.bfloat16)
    try:
        qg.test_gemv_mode(mode)
        qg.qgemm_small_m(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws), out=g.t)
        qg.poll_status()
    finally:
        qg.test_gemv_mode(0)
    assert g.intact() and not bool(g.untouched_inside().any().item())
    util.assert_close(util.host_bf16_f64(g.t), orc.qgemm_dense(qbits, A, Wq, Ws), f"small-M q{qbits} {M}x{N}x{K} mode {mode}")
