"""GPU parity: routing, segment offsets, stable permutation, row gather and combine against the CPU oracle.
Integer outputs must match bit for bit; routing weights within 1e-6 of the fp64 value."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def _ties_logits(M, E, seed):
    rng = np.random.default_rng(seed)
    l = rng.standard_normal((M, E)).astype(np.float32)
    l[0::5] = np.round(l[0::5] * 2) / 2
    l[1::7, :] = 0.25
    l[2::11, ::2] = 0.0
    l[2::11, 1::4] = -0.0
    return l


def _extreme_logits(M, E, seed):
    """Finite extremes: huge magnitudes of both signs, subnormals, both zeros, ordinary values, many ties."""
    rng = np.random.default_rng(seed)
    pool = np.array([3.0e38, -3.0e38, 1.0e-45, -1.0e-45, 0.0, -0.0, 1.5, -1.5, 1.17549435e-38, -7.0, 65504.0],
                    dtype=np.float32)
    return pool[rng.integers(0, pool.size, size=(M, E))]


CASES = [
    ("uniform-2048", 2048, 128, 8, "uniform"), ("skewed-2048", 2048, 128, 8, "skewed"),
    ("skewed-128", 128, 128, 8, "skewed"), ("ties", 257, 128, 8, "ties"), ("ragged", 33, 16, 16, "ties"),
    ("k1", 100, 8, 1, "uniform"), ("odd-E", 77, 5, 3, "ties"), ("E1024", 40, 1024, 8, "uniform"),
    ("k40", 65, 64, 40, "uniform"), ("one-token", 1, 128, 8, "uniform"), ("uniform-8192", 8192, 128, 8, "uniform"),
    ("extremes", 200, 96, 6, "extremes"),
    # more histogram blocks than the scan kernel has warps, with a ragged last block
    ("blocks-257", 8193, 16, 2, "skewed"), ("blocks-256-ragged", 8161, 24, 3, "ties"),
]


@pytest.mark.parametrize("name,M,E,k,kind", CASES, ids=[c[0] for c in CASES])
def test_route_bit_exact(name, M, E, k, kind):
    if kind == "ties":
        logits = _ties_logits(M, E, seed=M + E)
    elif kind == "extremes":
        logits = _extreme_logits(M, E, seed=M + E)
    else:
        logits = synth.router_logits(M, E, seed=0, hot_bias=synth.SKEW_HOT_BIAS if kind == "skewed" else 0.0)
    H = 64
    X = synth.activations(M, H, seed=1)
    r = qg.moe_route(util.dev(logits), k, X=util.dev_bf16(X))
    qg.poll_status()
    idx, w, _ = orc.route(logits, k)
    counts, offsets = orc.counts_offsets(idx, E)
    row_pair, pair_row = orc.permutation(idx, offsets)
    assert np.array_equal(r["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(r["counts"].cpu().numpy(), counts)
    assert np.array_equal(r["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(r["row_pair"].cpu().numpy(), row_pair)
    assert np.array_equal(r["pair_row"].cpu().numpy(), pair_row)
    gw = r["topk_w"].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(gw - w)) <= util.TOPK_W_ATOL
    assert np.max(np.abs(gw.sum(1) - 1.0)) <= util.TOPK_W_ATOL
    assert np.array_equal(util.host_bf16_bits(r["Xperm"]), orc.permute(X, row_pair, k))


def test_route_is_reproducible_and_empty_input_is_a_noop():
    logits = util.dev(synth.router_logits(512, 128, seed=3))
    a = qg.moe_route(logits, 8)
    b = qg.moe_route(logits, 8)
    for key in ("topk_idx", "row_pair", "pair_row", "offsets"):
        assert torch.equal(a[key], b[key])
    z = qg.moe_route(torch.empty((0, 16), dtype=torch.float32, device="cuda"), 2)
    assert z["offsets"].cpu().tolist() == [0] * 17 and z["counts"].cpu().tolist() == [0] * 16


def test_permute_standalone_and_combine():
    M, E, k, H = 300, 32, 4, 520
    logits = synth.router_logits(M, E, seed=5)
    X = synth.activations(M, H, seed=6)
    idx, w, w32 = orc.route(logits, k)
    counts, offsets = orc.counts_offsets(idx, E)
    row_pair, pair_row = orc.permutation(idx, offsets)
    Xp = qg.moe_permute(util.dev_bf16(X), util.dev(row_pair), k)
    assert np.array_equal(util.host_bf16_bits(Xp), orc.permute(X, row_pair, k))
    # combine over bf16 rows: the oracle consumes exactly the rows the GPU consumed
    D = synth.activations(M * k, H, seed=7)
    Dd = util.dev_bf16(D)
    y_w = qg.moe_combine(Dd, util.dev(pair_row), k, topk_w=util.dev(w32))
    y_1 = qg.moe_combine(Dd, util.dev(pair_row), k)
    qg.poll_status()
    D64 = orc.bf16_to_f64(D)
    util.assert_close(util.host_bf16_f64(y_w), orc.combine(D64, pair_row, k, w32.astype(np.float64)), "combine weighted")
    util.assert_close(util.host_bf16_f64(y_1), orc.combine(D64, pair_row, k), "combine unweighted")
    # f32 accumulator flavour: plain rounding
    acc = torch.randn(M, H, device="cuda", dtype=torch.float32)
    y_a = qg.moe_combine(acc, None, k, d_kind=qg.D_F32_ACC)
    assert torch.equal(y_a, acc.to(torch.bfloat16))


def test_error_codes_are_returned_before_any_launch():
    l = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(qg.QGemmError) as e:
        qg.moe_route(l, 9)
    assert e.value.code == -2
    with pytest.raises(qg.QGemmError) as e:
        qg.moe_route(l, 2, ws=torch.empty(4, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -4
    A = torch.zeros((4, 100), dtype=torch.bfloat16, device="cuda")
    Wq = torch.zeros((8, 100), dtype=torch.int8, device="cuda")
    Ws = torch.zeros((8, 4), dtype=torch.float16, device="cuda")
    with pytest.raises(qg.QGemmError) as e:
        qg.qgemm_dense(8, A, Wq, Ws)
    assert e.value.code == -2
    A = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    Wq = torch.zeros((8, 256), dtype=torch.int8, device="cuda")
    Ws = torch.zeros((8, 8), dtype=torch.float16, device="cuda")
    big = torch.zeros(8 * 256 + 16, dtype=torch.int8, device="cuda")
    with pytest.raises(qg.QGemmError) as e:
        qg.qgemm_dense(8, A, big[1:1 + 8 * 256].view(8, 256), Ws)     # misaligned weight pointer
    assert e.value.code == -3
    with pytest.raises(qg.QGemmError) as e:
        qg.qgemm_dense(5, A, Wq, Ws)
    assert e.value.code == -2
    assert qg.qgemm_dense(8, A[:0], Wq, Ws).shape == (0, 8)
