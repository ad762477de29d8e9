"""GPU parity of the MoE path: every call alone against an oracle fed with exactly the tensors the GPU call
consumed, and the whole layer against the unrounded fp64 layer."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def gpu_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k, fused_combine=False):
    d = dict(logits=util.dev(logits), X=util.dev_bf16(X), W1q=util.dev(W1q), W1s=util.dev_f16(W1s),
             W2q=util.dev(W2q), W2s=util.dev_f16(W2s))
    M = logits.shape[0]
    r = qg.moe_route(d["logits"], k, X=d["X"])
    Hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, qbits, r["Xperm"], r["offsets"], d["W1q"], d["W1s"])
    wflat = r["topk_w"].view(-1)
    if fused_combine:
        acc = qg.moe_grouped_qgemm(qg.MODE_DOWN_ACCUM_F32, qbits, Hh, r["offsets"], d["W2q"], d["W2s"], topk_w=wflat,
                                   row_pair=r["row_pair"], k=k, M=M)
        y = qg.moe_combine(acc, None, k, d_kind=qg.D_F32_ACC)
        Dw = None
    else:
        Dw = qg.moe_grouped_qgemm(qg.MODE_DOWN_WEIGHTED, qbits, Hh, r["offsets"], d["W2q"], d["W2s"], topk_w=wflat,
                                  row_pair=r["row_pair"], k=k)
        y = qg.moe_combine(Dw, r["pair_row"], k)
    qg.poll_status()
    return r, Hh, Dw, y, d


CASES = [
    ("small-q4", 4, 96, 256, 8, 256, 2, False), ("small-q8", 8, 96, 256, 8, 256, 2, False),
    ("empty-experts-q4", 4, 5, 256, 16, 256, 2, False), ("k-eq-E-q8", 8, 40, 512, 4, 256, 4, False),
    ("long-segments-q4", 4, 700, 256, 2, 256, 1, False), ("long-segments-q8", 8, 650, 256, 3, 512, 2, False),
    ("skewed-q4", 4, 512, 512, 32, 256, 8, True),
]


@pytest.mark.parametrize("name,qbits,M,H,E,F,k,skewed", CASES, ids=[c[0] for c in CASES])
def test_moe_stages_and_layer(name, qbits, M, H, E, F, k, skewed):
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=1, skewed=skewed)
    r, Hh, Dw, y, d = gpu_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k)
    o = orc.moe_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k)
    for key, okey in (("topk_idx", "idx"), ("counts", "counts"), ("offsets", "offsets"), ("row_pair", "row_pair"),
                      ("pair_row", "pair_row")):
        assert np.array_equal(r[key].cpu().numpy().reshape(o[okey].shape), o[okey]), key
    assert np.array_equal(util.host_bf16_bits(r["Xperm"]), o["Xp"])
    # stage: gate/up + SiLU (inputs identical to the oracle's because Xperm is bit exact)
    util.assert_close(util.host_bf16_f64(Hh), o["Hh"], "gate/up+silu")
    # stage: down projection on the GPU's own bf16 Hh and fp32 routing weights
    Hh64 = util.host_bf16_f64(Hh)
    w_gpu = r["topk_w"].cpu().numpy().astype(np.float64).reshape(-1)
    Dn = orc.grouped_gemm(qbits, Hh64, o["offsets"], W2q, W2s)
    util.assert_close(util.host_bf16_f64(Dw), Dn * w_gpu[o["row_pair"]][:, None], "down weighted")
    # stage: plain mode on the same input
    Dp = qg.moe_grouped_qgemm(qg.MODE_PLAIN, qbits, Hh, r["offsets"], d["W2q"], d["W2s"])
    util.assert_close(util.host_bf16_f64(Dp), Dn, "down plain")
    # stage: combine on the GPU's own weighted rows
    util.assert_close(util.host_bf16_f64(y), orc.combine(util.host_bf16_f64(Dw), o["pair_row"], k), "combine")
    # whole layer against the unrounded fp64 layer
    util.assert_close(util.host_bf16_f64(y), o["y"], "layer")
    # fused accumulate flavour
    _, _, _, y2, _ = gpu_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k, fused_combine=True)
    util.assert_close(util.host_bf16_f64(y2), o["y"], "layer (atomic accumulate)")


def test_moe_config3_shape_reduced_tokens():
    """Config 3 geometry (H=2048, E=128, k=8, F=768, Q4) at M=128 with skewed routing: 8 rows per expert on average,
    segments from at most 2 rows to at least 20 in one launch; every stage output against the oracle."""
    qbits, M, H, E, F, k = 4, 128, 2048, 128, 768, 8
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=0, skewed=True)
    r, Hh, Dw, y, d = gpu_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k)
    o = orc.moe_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k)
    assert np.array_equal(r["row_pair"].cpu().numpy(), o["row_pair"])
    assert o["counts"].min() <= 2 and o["counts"].max() >= 20      # short and long segments in one launch
    util.assert_close(util.host_bf16_f64(Hh), o["Hh"], "gate/up+silu cfg3")
    util.assert_close(util.host_bf16_f64(y), o["y"], "layer cfg3")


def test_grouped_more_tiles_per_pair_than_the_tile_table():
    """512 experts x 20 pairs of weight tiles = about 10,000 pair tiles, i.e. more per SM pair (about 138) than the
    128 entries of the kernel's shared-memory tile table: the tiles past the table are decoded on the fly.  Ragged
    segments, some experts empty; plain grouped mode, every output row against the oracle."""
    qbits, E, N, K = 4, 512, 5120, 256
    rng = np.random.default_rng(5)
    counts = rng.integers(1, 12, size=E).astype(np.int32)
    counts[rng.integers(0, E, size=6)] = 0
    offsets = np.zeros(E + 1, np.int32)
    offsets[1:] = np.cumsum(counts)
    R = int(offsets[-1])
    A = synth.activations(R, K, 3, 21)
    Wq = synth.weights_q4(E * N, K, 3, 22).reshape(E, N, K // 2)
    Ws = synth.scales(E * N, K // 32, 7, 3, 23).reshape(E, N, K // 32)
    n_tiles = int(np.count_nonzero(counts)) * ((N // 128 + 1) // 2)
    assert n_tiles > 128 * 74
    out = qg.moe_grouped_qgemm(qg.MODE_PLAIN, qbits, util.dev_bf16(A), util.dev(offsets), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    ref = orc.grouped_gemm(qbits, orc.bf16_to_f64(A), offsets, Wq, Ws)
    util.assert_close(util.host_bf16_f64(out), ref, "grouped plain, tiles beyond the table")


@pytest.mark.parametrize("qbits,E,rows,K,N,mode", [
    (4, 2, 600, 256, 8192, qg.MODE_PLAIN), (8, 2, 600, 512, 8192, qg.MODE_DOWN_WEIGHTED),
    (4, 16, 96, 256, 8192, qg.MODE_PLAIN), (8, 16, 96, 512, 8192, qg.MODE_DOWN_WEIGHTED),
    (4, 3, 500, 256, 4096, qg.MODE_GATE_UP_SILU)],
    ids=["q4-192tile-k256", "q8-192tile-k512-weighted", "q4-128tile-k256", "q8-128tile-k512-weighted", "q4-gateup-k256"])
def test_grouped_short_k_many_tiles_per_pair(qbits, E, rows, K, N, mode):
    """Grouped calls with K = 256 / 512 and several token tiles of real length per SM pair (long segments -> 192-token
    tiles, 96-row segments -> 128-token tiles): every output row against the oracle."""
    counts = np.full(E, rows, np.int32)
    counts[-1] = rows - 37                                      # one ragged segment
    offsets = np.zeros(E + 1, np.int32)
    offsets[1:] = np.cumsum(counts)
    R = int(offsets[-1])
    A = synth.activations(R, K, 8, 51)
    gen = synth.weights_q8 if qbits == 8 else synth.weights_q4
    Wq = gen(E * N, K, 8, 52).reshape(E, N, -1)
    Ws = synth.scales(E * N, K // 32, 127 if qbits == 8 else 7, 8, 53).reshape(E, N, K // 32)
    rng = np.random.default_rng(3)
    row_pair = rng.permutation(R).astype(np.int32)
    w = rng.uniform(0.1, 1.0, R).astype(np.float32)
    out = qg.moe_grouped_qgemm(mode, qbits, util.dev_bf16(A), util.dev(offsets), util.dev(Wq), util.dev_f16(Ws),
                               topk_w=util.dev(w), row_pair=util.dev(row_pair), k=1)
    qg.poll_status()
    ref = orc.grouped_gemm(qbits, orc.bf16_to_f64(A), offsets, Wq, Ws)
    if mode == qg.MODE_GATE_UP_SILU:
        ref = orc.silu_mul(ref)
    elif mode == qg.MODE_DOWN_WEIGHTED:
        ref = ref * w[row_pair].astype(np.float64)[:, None]
    util.assert_close(util.host_bf16_f64(out), ref, "grouped short K")


GATHER = [("small-q4", 4, 96, 256, 8, 256, 2, False), ("ragged-q8", 8, 333, 512, 5, 256, 3, False),
          ("skewed-q4", 4, 512, 512, 32, 256, 8, True), ("long-q4", 4, 700, 256, 2, 256, 1, False),
          ("cfg3-128", 4, 128, 2048, 128, 768, 8, True)]


@pytest.mark.parametrize("name,qbits,M,H,E,F,k,skewed", GATHER, ids=[c[0] for c in GATHER])
def test_gather_in_load_equals_permute_then_gemm(name, qbits, M, H, E, F, k, skewed):
    """moe_grouped_qgemm_gather reads the token rows through the routing table instead of from a permuted copy: its
    gate/up output must match the oracle, and the whole layer built on it (no Xperm, accumulate epilogue, rounding)
    must match the unrounded fp64 layer."""
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=2, skewed=skewed)
    dX, dW1q, dW1s, dW2q, dW2s = util.dev_bf16(X), util.dev(W1q), util.dev_f16(W1s), util.dev(W2q), util.dev_f16(W2s)
    r = qg.moe_route(util.dev(logits), k)                                   # no row gather here
    Hh = qg.moe_grouped_qgemm_gather(qg.MODE_GATE_UP_SILU, qbits, dX, r["row_pair"], k, r["offsets"], dW1q, dW1s)
    Gp = qg.moe_grouped_qgemm_gather(qg.MODE_PLAIN, qbits, dX, r["row_pair"], k, r["offsets"], dW1q, dW1s)
    acc = qg.moe_grouped_qgemm(qg.MODE_DOWN_ACCUM_F32, qbits, Hh, r["offsets"], dW2q, dW2s, topk_w=r["topk_w"].view(-1),
                               row_pair=r["row_pair"], k=k, M=M)
    y = qg.moe_combine(acc, None, k, d_kind=qg.D_F32_ACC)
    qg.poll_status()
    o = orc.moe_layer(qbits, logits, X, W1q, W1s, W2q, W2s, k)
    assert np.array_equal(r["row_pair"].cpu().numpy(), o["row_pair"])
    util.assert_close(util.host_bf16_f64(Gp), o["GU"], "gathered plain")
    util.assert_close(util.host_bf16_f64(Hh), o["Hh"], "gathered gate/up+silu")
    util.assert_close(util.host_bf16_f64(y), o["y"], "layer (gather + accumulate)")
    # and the two ways of feeding the kernel agree to the last bit on a stage with one k-block order per tile
    Xp = qg.moe_permute(dX, r["row_pair"], k)
    Hh2 = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, qbits, Xp, r["offsets"], dW1q, dW1s)
    qg.poll_status()
    util.assert_close(util.host_bf16_f64(Hh2), o["Hh"], "permute + gemm")
