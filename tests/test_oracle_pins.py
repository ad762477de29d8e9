"""Pins of the CPU oracle against things other than itself: hand-computed cases (tests/golden),
exhaustive code tables, closed forms, brute force by a full library sort, an independent fp64 library
matmul, invariants and reductions of the MoE layer to dense products.  No GPU needed."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))


def f16bits(x):
    return np.asarray(x, dtype=np.float16).view(np.uint16)


def bf16bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# ----------------------------------------------------------------------------- decode
def test_fp16_decode_all_patterns_vs_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.f16_to_f64(bits)
    ref = bits.view(np.float16).astype(np.float64)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert got[1] == 2.0 ** -24 and got[0x0400] == 2.0 ** -14 and got[0x8001] == -(2.0 ** -24)


def test_bf16_decode_all_patterns_vs_torch():
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.bf16_to_f64(bits)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    nan = np.isnan(ref)
    assert np.array_equal(got[~nan], ref[~nan]) and np.array_equal(np.isnan(got), nan)


def test_bf16_rounding_vs_torch_and_ties():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    got = orc.f64_to_bf16(x.astype(np.float64))
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, ref)
    # ties: 1 + 2^-8 is halfway between 1 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert orc.f64_to_bf16(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 1e-12]))[:].tolist() == \
        [0x3F80, 0x3F82, 0x3F81]


def test_q4_code_table_exhaustive():
    # every byte value at every position of a 32-block; scale 1: weight 2j = (byte & 15) - 8, 2j+1 = (byte >> 4) - 8
    for byte in range(256):
        Wq = np.full((1, 16), 0x88, np.uint8)  # 0x88 = two zeros
        for j in (0, 5, 15):
            W = Wq.copy()
            W[0, j] = byte
            w = orc.dequant(4, W, f16bits([[1.0]]))[0]
            exp = np.zeros(32)
            exp[2 * j] = (byte % 16) - 8
            exp[2 * j + 1] = (byte // 16) - 8
            assert np.array_equal(w, exp)


def test_q8_code_table_exhaustive():
    q = np.arange(-128, 128, dtype=np.int8).reshape(1, 256)
    s = f16bits(np.array([[0.5, 1, 2, -1, 0.25, 3, 1, 1]]))
    w = orc.dequant(8, q, s)[0]
    exp = np.arange(-128, 128).astype(np.float64) * np.repeat([0.5, 1, 2, -1, 0.25, 3, 1, 1], 32)
    assert np.array_equal(w, exp)


# ----------------------------------------------------------------------------- dense hand cases
def _build_dense_case(c):
    K = c["K"]
    k = np.arange(K)
    A = {"ones": np.ones(K), "kmod4": (k % 4).astype(float), "first16": (k < 16).astype(float),
         "onehot1": (k == 1).astype(float)}[c["A"]]
    if c["qbits"] == 8:
        q = {"k-16": k - 16, "const127": np.full(K, 127), "constm128": np.full(K, -128), "const3": np.full(K, 3),
             "t2": np.where(k < 32, 1, -2)}[c["q"]].astype(np.int8).reshape(1, K)
    else:
        assert c["q"] == "t3"
        q = np.array([0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE] * 2, np.uint8).reshape(1, 16)
    s = np.array(c["scale_bits"], np.uint16) if "scale_bits" in c else f16bits(c["scale"])
    return bf16bits(A).reshape(1, K), q, s.reshape(1, K // 32)


@pytest.mark.parametrize("case", GOLD["dense"], ids=lambda c: c["name"].split(":")[0])
def test_dense_hand_cases(case):
    A, q, s = _build_dense_case(case)
    out = orc.qgemm_dense(case["qbits"], A, q, s)
    assert out.shape == (1, 1) and out[0, 0] == case["expect"]
    assert orc.qgemm_dense_sample(case["qbits"], A, q, s, [0], [0])[0] == case["expect"]


def _np_dequant(qbits, Wq, Ws):
    """Independent numpy route to the dequantised matrix (used only together with the hand cases above)."""
    s = np.repeat(Ws.view(np.float16).astype(np.float64), 32, axis=1)
    if qbits == 8:
        return Wq.astype(np.float64) * s
    lo = (Wq & 0xF).astype(np.float64) - 8
    hi = (Wq >> 4).astype(np.float64) - 8
    return np.stack([lo, hi], axis=-1).reshape(Wq.shape[0], -1) * s


@pytest.mark.parametrize("qbits,M,N,K", [(8, 128, 2048, 2048), (4, 37, 264, 320), (8, 5, 40, 96)])
def test_dense_vs_library_matmul_fp64(qbits, M, N, K):
    """Config-0 size (and ragged, non-square shapes that expose a transposed operand) against torch.matmul in
    fp64 over numpy-dequantised weights: an independent routine, different summation order -> 1e-12 relative."""
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=0)
    C = orc.qgemm_dense(qbits, A, Wq, Ws)
    a64 = torch.from_numpy(synth.bf16_bits_to_f32(A).astype(np.float64))
    ref = (a64 @ torch.from_numpy(_np_dequant(qbits, Wq, Ws)).T).numpy()
    assert C.shape == (M, N)
    assert np.max(np.abs(C - ref)) <= 1e-12 * np.max(np.abs(ref))
    rows = np.array([0, M - 1, M // 2, 3 % M]); cols = np.array([N - 1, 0, N // 3, 7])
    assert np.array_equal(orc.qgemm_dense_sample(qbits, A, Wq, Ws, rows, cols), C[rows, cols])


def test_dense_linearity_and_block_structure():
    # doubling one block's scale changes the result by exactly that block's partial sum
    A, Wq, Ws = synth.dense_problem(8, 3, 4, 128, seed=3)
    s = np.array([[1.0, 0.5, 2.0, 1.0]] * 4); s2 = s.copy(); s2[:, 2] = 4.0
    C1 = orc.qgemm_dense(8, A, Wq, f16bits(s)); C2 = orc.qgemm_dense(8, A, Wq, f16bits(s2))
    a = synth.bf16_bits_to_f32(A).astype(np.float64)
    part = a[:, 64:96] @ Wq[:, 64:96].astype(np.float64).T
    assert np.allclose(C2 - C1, 2.0 * part, rtol=0, atol=1e-9)


# ----------------------------------------------------------------------------- routing
@pytest.mark.parametrize("case", GOLD["route"], ids=lambda c: c["name"].split(":")[0])
def test_route_hand_cases(case):
    idx, w, w32 = orc.route(np.array([case["logits"]], np.float32), case["k"])
    assert idx[0].tolist() == case["idx"]
    assert np.allclose(w[0], case["w"], rtol=0, atol=1e-15)
    assert np.array_equal(w32[0], w[0].astype(np.float32))


def test_segments_hand_case():
    g = GOLD["segments"]
    logits = np.array([c["logits"] for c in GOLD["route"]], np.float32)
    idx, _, _ = orc.route(logits, g["k"])
    counts, offsets = orc.counts_offsets(idx, g["E"])
    row_pair, pair_row = orc.permutation(idx, offsets)
    assert counts.tolist() == g["counts"] and offsets.tolist() == g["offsets"]
    assert row_pair.tolist() == g["row_pair"] and pair_row.tolist() == g["pair_row"]


def _ties_logits(M, E, seed):
    rng = np.random.default_rng(seed)
    l = rng.standard_normal((M, E)).astype(np.float32)
    l[0::5] = np.round(l[0::5] * 2) / 2            # many equal values
    l[1::7, :] = 0.25                              # all equal
    l[2::11, ::2] = 0.0; l[2::11, 1::4] = -0.0     # signed zeros compare equal
    return l


@pytest.mark.parametrize("M,E,k", [(64, 128, 8), (33, 16, 16), (20, 8, 1), (50, 5, 3), (7, 1024, 8)])
def test_route_vs_full_stable_sort(M, E, k):
    l = _ties_logits(M, E, seed=E + k)
    idx, w, _ = orc.route(l, k)
    brute = np.argsort(-(l + np.float32(0.0)), axis=1, kind="stable")[:, :k]   # +0.0 folds -0 into +0
    assert np.array_equal(idx, brute.astype(np.int32))
    assert np.allclose(w.sum(1), 1.0, atol=1e-14)
    assert np.all(np.diff(w, axis=1) <= 1e-16)
    assert all(len(set(r)) == k for r in idx.tolist())
    sel = np.take_along_axis(l.astype(np.float64), idx.astype(np.int64), 1)
    ref = torch.softmax(torch.from_numpy(sel), dim=1).numpy()                  # library softmax of the selected
    assert np.allclose(w, ref, rtol=0, atol=1e-15)
    if k == E:
        full = torch.softmax(torch.from_numpy(l.astype(np.float64)), dim=1).numpy()
        assert np.allclose(np.sort(w, 1), np.sort(full, 1), atol=1e-15)
    if k == 1:
        assert np.all(w == 1.0)


def test_renormalised_full_softmax_equals_softmax_of_selected():
    l = synth.router_logits(40, 128, seed=2)
    idx, w, _ = orc.route(l, 8)
    p = torch.softmax(torch.from_numpy(l.astype(np.float64)), 1).numpy()
    sel = np.take_along_axis(p, idx.astype(np.int64), 1)
    assert np.allclose(w, sel / sel.sum(1, keepdims=True), rtol=1e-13, atol=0)


@pytest.mark.parametrize("skewed", [False, True])
def test_permutation_invariants(skewed):
    M, E, k = 256, 128, 8
    l = synth.router_logits(M, E, seed=0, hot_bias=synth.SKEW_HOT_BIAS if skewed else 0.0)
    idx, _, _ = orc.route(l, k)
    counts, offsets = orc.counts_offsets(idx, E)
    row_pair, pair_row = orc.permutation(idx, offsets)
    R = M * k
    assert np.array_equal(counts, np.bincount(idx.ravel(), minlength=E))
    assert offsets[0] == 0 and offsets[-1] == R and np.array_equal(np.diff(offsets), counts)
    assert np.array_equal(np.sort(row_pair), np.arange(R))
    assert np.array_equal(pair_row[row_pair], np.arange(R))
    assert np.array_equal(np.bincount(row_pair // k, minlength=M), np.full(M, k))   # every token exactly k times
    flat = idx.ravel()
    for e in range(E):
        seg = row_pair[offsets[e]:offsets[e + 1]]
        assert np.all(flat[seg] == e) and np.all(np.diff(seg) > 0)
    assert np.array_equal(row_pair, np.argsort(flat, kind="stable").astype(np.int32))  # library stable sort
    if skewed:
        hot = counts[::4].sum() / R
        assert 0.55 < hot < 0.65


def test_permute_is_row_gather():
    X = synth.activations(10, 64, seed=5)
    row_pair = np.array([5, 0, 19, 7, 3, 12], np.int32)
    assert np.array_equal(orc.permute(X, row_pair, 2), X[row_pair // 2])


# ----------------------------------------------------------------------------- MoE stages
def test_silu_closed_forms():
    for c in GOLD["silu"]:
        out = orc.silu_mul(np.array([[c["g"], c["u"]]]))
        assert abs(out[0, 0] - c["expect"]) <= 1e-15 * max(1.0, abs(c["expect"]))
    g = np.linspace(-30, 30, 61)
    out = orc.silu_mul(np.stack([g, np.ones_like(g)], 1).reshape(61, 2))[:, 0]
    assert np.allclose(out, g * torch.sigmoid(torch.from_numpy(g)).numpy(), rtol=1e-14, atol=0)
    # gate columns come first, up columns second: F = 2
    assert orc.silu_mul(np.array([[0.0, 1.0, 5.0, 7.0]]))[0].tolist() == [0.0, 7.0 / (1 + np.exp(-1.0))]


def _small_moe(qbits, M=24, H=64, E=4, F=32, k=2, seed=1):
    return synth.moe_problem(qbits, M, H, E, F, seed=seed), k


@pytest.mark.parametrize("qbits", [4, 8])
def test_grouped_gemm_is_per_segment_library_matmul(qbits):
    (logits, X, W1q, W1s, W2q, W2s), k = _small_moe(qbits)
    E = logits.shape[1]
    idx, w, _ = orc.route(logits, k)
    counts, offsets = orc.counts_offsets(idx, E)
    row_pair, _ = orc.permutation(idx, offsets)
    Xp = synth.bf16_bits_to_f32(orc.permute(X, row_pair, k)).astype(np.float64)
    GU = orc.grouped_gemm(qbits, Xp, offsets, W1q, W1s)
    for e in range(E):
        w_e = _np_dequant(qbits, W1q[e], W1s[e])
        seg = slice(offsets[e], offsets[e + 1])
        assert np.allclose(GU[seg], Xp[seg] @ w_e.T, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("qbits", [4, 8])
def test_moe_single_expert_reduces_to_three_dense_products(qbits):
    M, H, F = 9, 64, 32
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, 1, F, seed=4)
    r = orc.moe_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k=1)
    assert np.all(r["w"] == 1.0) and np.array_equal(r["row_pair"], np.arange(M))
    GU = orc.qgemm_dense(qbits, X, W1q[0], W1s[0])
    G, U = GU[:, :F], GU[:, F:]
    Hh = G / (1 + np.exp(-G)) * U
    y = Hh @ _np_dequant(qbits, W2q[0], W2s[0]).T
    assert np.allclose(r["y"], y, rtol=1e-12, atol=1e-14)


def test_moe_identical_experts_equal_single_ffn_for_any_routing():
    M, H, E, F, k = 16, 64, 8, 32, 3
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(8, M, H, E, F, seed=6)
    W1q[:] = W1q[0]; W1s[:] = W1s[0]; W2q[:] = W2q[0]; W2s[:] = W2s[0]
    r = orc.moe_layer(8, logits, X, W1q, W1s, W2q, W2s, k)
    one = orc.moe_layer(8, np.zeros((M, 1), np.float32), X, W1q[:1], W1s[:1], W2q[:1], W2s[:1], 1)
    assert np.allclose(r["y"], one["y"], rtol=1e-12, atol=1e-14)     # weights sum to 1


def test_combine_definition():
    D = np.arange(12, dtype=np.float64).reshape(6, 2)
    pair_row = np.array([3, 0, 5, 1, 2, 4], np.int32)
    w = np.array([[0.5, 0.5], [1.0, 0.0], [0.25, 0.75]])
    y = orc.combine(D, pair_row, 2, w)
    assert y.tolist() == [[0.5 * 6 + 0.5 * 0, 0.5 * 7 + 0.5 * 1], [10.0, 11.0], [0.25 * 4 + 0.75 * 8, 0.25 * 5 + 0.75 * 9]]
    assert orc.combine(D, pair_row, 2).tolist() == [[6.0, 8.0], [12.0, 14.0], [12.0, 14.0]]


def test_combine_shared_adds_the_shared_row_last():
    """Hand case: the routed sums of test_combine_definition plus a shared row; a zero shared expert changes nothing;
    with no routed weight (w = 0) the result is the shared row itself."""
    D = np.arange(12, dtype=np.float64).reshape(6, 2)
    pair_row = np.array([3, 0, 5, 1, 2, 4], np.int32)
    w = np.array([[0.5, 0.5], [1.0, 0.0], [0.25, 0.75]])
    shared = np.array([[100.0, -1.0], [0.5, 0.25], [-7.0, 2.0]])
    y = orc.combine_shared(D, pair_row, 2, shared, w)
    assert y.tolist() == [[3.0 + 100.0, 4.0 - 1.0], [10.5, 11.25], [7.0 - 7.0, 8.0 + 2.0]]
    assert np.array_equal(orc.combine_shared(D, pair_row, 2, np.zeros((3, 2)), w), orc.combine(D, pair_row, 2, w))
    assert np.array_equal(orc.combine_shared(D, pair_row, 2, shared, np.zeros((3, 2))), shared)


def test_router_logits_definition():
    """Hand case (a transposed operand or a swapped index gives other numbers), one-hot rows that pick out single
    weights, and an fp64 library matmul on a ragged shape."""
    X = np.array([[1.0, 2.0, 3.0], [0.0, -1.0, 0.5]])
    Wr = np.array([[1.0, 0.0, 0.0], [0.0, 1.0, 1.0], [2.0, 2.0, 2.0], [-1.0, 0.5, 0.25]])
    L = orc.router_logits(X, Wr)
    assert L.tolist() == [[1.0, 5.0, 12.0, 0.75], [0.0, -0.5, -1.0, -0.375]]
    rng = np.random.default_rng(3)
    Wr = rng.standard_normal((7, 5))
    assert np.array_equal(orc.router_logits(np.eye(5), Wr), Wr.T)
    X = rng.standard_normal((33, 129)); Wr = rng.standard_normal((10, 129))
    np.testing.assert_allclose(orc.router_logits(X, Wr), X @ Wr.T, rtol=1e-12, atol=1e-12)


def test_one_hot_logits_select_one_expert():
    M, H, E, F, k = 6, 64, 4, 32, 2
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(4, M, H, E, F, seed=8)
    logits[:] = -50.0
    logits[np.arange(M), np.arange(M) % E] = 50.0
    r = orc.moe_layer(4, logits, X, W1q, W1s, W2q, W2s, k)
    assert np.array_equal(r["idx"][:, 0], np.arange(M) % E) and np.all(r["w"][:, 1] < 1e-40)
    e = 1; t = 1
    GU = orc.qgemm_dense(4, X[t:t + 1], W1q[e], W1s[e])
    Hh = orc.silu_mul(GU)
    y = Hh @ _np_dequant(4, W2q[e], W2s[e]).T
    assert np.allclose(r["y"][t], y[0], rtol=1e-12, atol=1e-16)


# ---------------------------------------------------------------------------------------------- attention
def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, np.float32))


def test_attention_closed_forms():
    """Pins that need no other implementation.  Zero queries give uniform weights, so a causal row i is the mean of
    V[0..i] and a full row the mean of all V; a query aligned with exactly one key by a huge margin returns that
    key's value; row 0 of a causal problem is V[0]."""
    S, Hq, Hkv, d = 7, 2, 1, 8
    rng = np.random.default_rng(0)
    V = _bf16(rng.standard_normal((S, Hkv * d)))
    K = _bf16(rng.standard_normal((S, Hkv * d)))
    Q0 = _bf16(np.zeros((S, Hq * d)))
    Vf = orc.bf16_to_f64(V)
    out = orc.attention(Q0, K, V, Hq, Hkv, d, causal=True)
    for i in range(S):
        want = Vf[:i + 1].mean(axis=0)
        assert np.allclose(out[i, :d], want, atol=1e-12) and np.allclose(out[i, d:], want, atol=1e-12)
    full = orc.attention(Q0, K, V, Hq, Hkv, d, causal=False)
    assert np.allclose(full, np.tile(Vf.mean(axis=0), (S, Hq)), atol=1e-12)
    # one-hot keys, query = 64 * e_j: score gap of 64 * scale * 1 = 22.6, weights of the others below 2e-10
    Ke = _bf16(np.eye(S, d)); Qe = _bf16(np.tile(64.0 * np.eye(S, d)[::-1], (1, Hq)))   # query i looks for key S-1-i
    pick = orc.attention(Qe, Ke, V, Hq, Hkv, d, causal=False)
    assert np.allclose(pick[:, :d], Vf[::-1], atol=1e-8)
    assert np.array_equal(orc.attention(Qe, Ke, V, Hq, Hkv, d, causal=True)[0, :d], Vf[0])


def test_attention_hand_case():
    """S = 2, d = 2, one head, scale 1: scores [[q0.k0], [q1.k0, q1.k1]] = [[1], [0, ln 3]] -> weights [1], [1/4, 3/4];
    values v0 = (4, 0), v1 = (0, 8)  ->  O = [(4, 0), (1, 6)]."""
    ln3 = np.log(3.0)
    Q = np.array([[1.0, 0.0], [0.0, 1.0]], np.float32)
    K = np.array([[1.0, 0.0], [0.0, ln3]], np.float32)
    V = np.array([[4.0, 0.0], [0.0, 8.0]], np.float32)
    out = orc.attention(_bf16(Q), _bf16(K), _bf16(V), 1, 1, 2, causal=True, scale=1.0)
    k11 = float(orc.bf16_to_f64(_bf16(K))[1, 1])                 # ln 3 rounded to bf16
    w1 = np.exp(k11) / (1.0 + np.exp(k11))
    assert np.allclose(out[0], [4.0, 0.0], atol=1e-15)
    assert np.allclose(out[1], [4.0 * (1 - w1), 8.0 * w1], atol=1e-13)
    assert abs(out[1, 1] - 6.0) < 0.02                            # 3/4 * 8 up to the rounding of ln 3


@pytest.mark.parametrize("causal", [True, False])
def test_attention_against_library_softmax_and_matmul(causal):
    """torch fp64 matmul + softmax as an independent routine, grouped-query heads expanded explicitly, inputs taken as
    strided views of one wide [S, (Hq + 2 Hkv) d] buffer (the layout a fused QKV projection leaves behind)."""
    S, Hq, Hkv, d = 37, 6, 2, 16
    rng = np.random.default_rng(1)
    qkv = _bf16(rng.standard_normal((S, (Hq + 2 * Hkv) * d)))
    Q, K, V = qkv[:, :Hq * d], qkv[:, Hq * d:(Hq + Hkv) * d], qkv[:, (Hq + Hkv) * d:]
    out = orc.attention(Q, K, V, Hq, Hkv, d, causal=causal)
    f = lambda x, h: torch.from_numpy(orc.bf16_to_f64(np.ascontiguousarray(x))).view(S, h, d).permute(1, 0, 2)
    q, k, v = f(Q, Hq), f(K, Hkv).repeat_interleave(Hq // Hkv, 0), f(V, Hkv).repeat_interleave(Hq // Hkv, 0)
    sc = q @ k.transpose(1, 2) / np.sqrt(d)
    if causal:
        sc = sc.masked_fill(torch.triu(torch.ones(S, S, dtype=torch.bool), 1), float("-inf"))
    want = (torch.softmax(sc, -1) @ v).permute(1, 0, 2).reshape(S, Hq * d).numpy()
    assert np.allclose(out, want, atol=1e-12)
    # a sample of query rows equals the same rows of the full result
    qpos = np.array([0, 5, S - 1])
    assert np.array_equal(orc.attention(Q, K, V, Hq, Hkv, d, causal=causal, qpos=qpos), out[qpos])


# ---------------------------------------------------------------------------------------------- MX (block-scaled FP8)
def test_e4m3_table_matches_the_library_type_and_known_values():
    codes = np.arange(256, dtype=np.uint8)
    mine = orc.e4m3_to_f64(codes)
    lib_vals = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    finite = ~np.isnan(lib_vals)
    assert np.array_equal(np.isnan(mine), ~finite) and np.array_equal(mine[finite], lib_vals[finite])
    assert mine[0x38] == 1.0 and mine[0x7E] == 448.0 and mine[0x01] == 2.0 ** -9 and mine[0xC0] == -2.0 and mine[0x08] == 2.0 ** -6


def test_mx_quantize_hand_cases_and_library_rounding():
    """Block max 448 -> e = 0, codes are the values themselves; max 1.0 -> e = -8, 1.0 becomes 256 (0x78); a value of 449
    in a block whose max is 449 (e = 0) clamps to 448; ties go to the even code (13 is half-way between 12 and 14 at
    this binade: 12 = 0x54 has an even mantissa... checked against the table itself); zero block -> scale byte 0."""
    x = np.zeros((4, 32))
    x[0, :4] = [448.0, 1.0, -3.5, 0.0625]
    x[1, :3] = [1.0, 0.5, -0.75]
    x[2, :2] = [449.0, 300.0]
    codes, sf = orc.mx_quantize(x)
    assert sf[0, 0] == 127 and sf[1, 0] == 127 - 8 and sf[2, 0] == 127 and sf[3, 0] == 0
    v = orc.e4m3_to_f64(codes)
    assert list(v[0, :4]) == [448.0, 1.0, -3.5, 0.0625]
    assert list(v[1, :3]) == [256.0, 128.0, -192.0]
    assert v[2, 0] == 448.0 and v[2, 1] == 288.0 or v[2, 1] == 320.0      # 300 lies between 288 and 320: nearest is 288
    assert v[2, 1] == 288.0
    assert not np.any(v[3])
    # in-range values against the library's round-to-nearest-even conversion
    rng = np.random.default_rng(0)
    y = rng.standard_normal((64, 64)) * rng.choice([1e-3, 1.0, 30.0], (64, 1))
    c, s = orc.mx_quantize(y)
    scaled = y.reshape(64, 2, 32) * (2.0 ** (127.0 - s.astype(np.float64)))[:, :, None]
    assert np.max(np.abs(scaled)) < 512.0
    inr = np.abs(scaled) <= 448.0
    want = torch.from_numpy(scaled).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(c.reshape(64, 2, 32)[inr], want[inr])
    # dequantised blocks reproduce the input to within half an E4M3 step of the block maximum's binade
    deq = orc.e4m3_to_f64(c).reshape(64, 2, 32) * (2.0 ** (s.astype(np.float64) - 127.0))[:, :, None]
    amax = np.abs(y.reshape(64, 2, 32)).max(axis=2, keepdims=True)
    assert np.all(np.abs(deq - y.reshape(64, 2, 32)) <= amax / 8.0 + 1e-300)


def test_mx_gemm_against_library_matmul_and_scale_tiling_roundtrip():
    rng = np.random.default_rng(1)
    M, N, K = 9, 13, 256
    a, asf = orc.mx_quantize(rng.standard_normal((M, K)))
    w, wsf = orc.mx_quantize(rng.standard_normal((N, K)) * 0.01)
    A = orc.e4m3_to_f64(a).reshape(M, K // 32, 32) * (2.0 ** (asf.astype(np.float64) - 127))[:, :, None]
    W = orc.e4m3_to_f64(w).reshape(N, K // 32, 32) * (2.0 ** (wsf.astype(np.float64) - 127))[:, :, None]
    want = (torch.from_numpy(A.reshape(M, K)) @ torch.from_numpy(W.reshape(N, K)).T).numpy()
    assert np.allclose(orc.mx_gemm(a, asf, w, wsf), want, rtol=1e-13, atol=1e-300)
    # hand case: one block, a = 1.0 (code 0x38) with scale 2^1, w = 0.5 (0x30) with scale 2^-2: 32 * 2 * 0.125 = 8
    one = np.full((1, 32), 0x38, np.uint8); half = np.full((1, 32), 0x30, np.uint8)
    assert orc.mx_gemm(one, np.array([[128]], np.uint8), half, np.array([[125]], np.uint8))[0, 0] == 8.0
    plain = rng.integers(0, 255, (300, 8)).astype(np.uint8)
    tiles = synth.mx_scale_tiles(plain)
    assert tiles.size == 384 * 8 and np.array_equal(synth.mx_scale_plain(tiles, 300, 256), plain)
    assert tiles[100] == plain[38, 0] and tiles[511] == plain[127, 3] and tiles[512 + 17] == plain[1, 5]


def test_mx_grouped_gemm_is_the_per_segment_product():
    """Two experts with different weights: each output row equals the dense MX product of its row with its own expert's
    weights (checked against mx_gemm on single rows), an empty expert contributes nothing, and the grouped scale tiling
    restarts at every segment (the first row of segment 1 sits at row 0 of a new tile)."""
    rng = np.random.default_rng(11)
    K, N = 128, 5
    offsets = np.array([0, 3, 3, 7], np.int32)
    a, asf = orc.mx_quantize(rng.standard_normal((7, K)))
    w = np.zeros((3, N, K), np.uint8); wsf = np.zeros((3, N, K // 32), np.uint8)
    for e in range(3):
        w[e], wsf[e] = orc.mx_quantize(rng.standard_normal((N, K)) * (e + 1))
    out = orc.mx_grouped_gemm(a, asf, offsets, w, wsf)
    for r, e in [(0, 0), (2, 0), (3, 2), (6, 2)]:
        assert np.array_equal(out[r], orc.mx_gemm(a[r:r + 1], asf[r:r + 1], w[e], wsf[e])[0])
    tiles = synth.mx_scale_tiles_grouped(asf, offsets)
    assert tiles.size == 2 * 512                               # one tile per non-empty segment
    assert tiles[512 + 0 * 16 + 0 * 4 + 1] == asf[3, 1] and tiles[2 * 16 + 3] == asf[2, 3]
