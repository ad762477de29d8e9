"""Out-of-bounds guard: every output sits inside a larger buffer filled with a sentinel; after the call the sentinel
around it must be intact, every element that the call owns must have been written, and (for the grouped calls)
rows past the last expert segment must be untouched.  Ragged tails, odd weight-tile counts and segment ends in the
middle of a token tile are the cases whose stores rest on hand-written predicates."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu

DENSE = [(8, 17, 200, 256), (4, 513, 136, 768), (8, 300, 384, 512), (4, 1, 128, 256), (8, 129, 8, 256),
         (4, 191, 392, 512), (8, 257, 648, 256)]


@pytest.mark.parametrize("qbits,M,N,K", DENSE, ids=[f"q{c[0]}-{c[1]}x{c[2]}x{c[3]}" for c in DENSE])
def test_dense_writes_nothing_outside_its_output(qbits, M, N, K):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=3)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.qgemm_dense(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws), out=g.t)
    qg.poll_status()
    assert g.intact(), "store outside C[M, N]"
    assert not bool(g.untouched_inside().any().item()), "an element of C was never written"
    util.assert_close(util.host_bf16_f64(g.t), orc.qgemm_dense(qbits, A, Wq, Ws), "guarded dense")


def _segments(counts):
    off = np.zeros(len(counts) + 1, np.int32)
    off[1:] = np.cumsum(counts)
    return off


# expert segments that end in the middle of a token tile, followed by empty experts or by nothing at all
LAYOUTS = [("tail-then-empty", [100, 0, 0, 0]), ("mixed", [50, 0, 100, 0, 37]), ("long-then-short", [333, 1, 0, 7]),
           ("single-row", [0, 0, 1])]


@pytest.mark.parametrize("mode", [qg.MODE_PLAIN, qg.MODE_GATE_UP_SILU, qg.MODE_DOWN_WEIGHTED], ids=["plain", "gateup", "weighted"])
@pytest.mark.parametrize("name,counts", LAYOUTS, ids=[l[0] for l in LAYOUTS])
@pytest.mark.parametrize("qbits", [4, 8])
def test_grouped_stores_stay_inside_their_segments(qbits, name, counts, mode):
    E = len(counts)
    off = _segments(counts)
    R = int(off[-1])
    K = 256
    N = 512 if mode == qg.MODE_GATE_UP_SILU else 392          # 392 = three weight tiles and a ragged fourth
    A = synth.activations(R, K, 5, 31)
    gen = synth.weights_q8 if qbits == 8 else synth.weights_q4
    Wq = gen(E * N, K, 5, 32).reshape(E, N, -1)
    Ws = synth.scales(E * N, K // 32, 127 if qbits == 8 else 7, 5, 33).reshape(E, N, K // 32)
    n_out = N // 2 if mode == qg.MODE_GATE_UP_SILU else N
    extra = 40                                                  # rows past the last segment: nobody may write them
    g = util.Guarded((R + extra, n_out), torch.bfloat16)
    rng = np.random.default_rng(1)
    row_pair = rng.permutation(R).astype(np.int32)
    w = rng.uniform(0.1, 1.0, R).astype(np.float32)
    qg.moe_grouped_qgemm(mode, qbits, util.dev_bf16(A), util.dev(off), util.dev(Wq), util.dev_f16(Ws),
                         topk_w=util.dev(w), row_pair=util.dev(row_pair), k=1, out=g.t[:R])
    qg.poll_status()
    assert g.intact(), "store outside the output buffer"
    inside = g.untouched_inside()
    assert bool(inside[R:].all().item()), "store into rows past the last segment"
    assert not bool(inside[:R].any().item()), "a row of a segment was never written"
    ref = orc.grouped_gemm(qbits, orc.bf16_to_f64(A), off, Wq, Ws)
    if mode == qg.MODE_GATE_UP_SILU:
        ref = orc.silu_mul(ref)
    elif mode == qg.MODE_DOWN_WEIGHTED:
        ref = ref * w[row_pair].astype(np.float64)[:, None]
    util.assert_close(util.host_bf16_f64(g.t[:R]), ref, f"guarded grouped mode {mode}")


@pytest.mark.parametrize("qbits", [4, 8])
def test_accumulating_epilogue_touches_only_routed_tokens(qbits):
    """Mode 3 adds into y[token] with atomics: rows of tokens that no routed row points at must stay exactly zero and
    nothing may land outside y."""
    k, M_tok, E, K, N = 2, 90, 3, 256, 264
    routed = np.arange(0, M_tok, 2)                              # even tokens only
    pairs = np.concatenate([routed * k, routed * k + 1]).astype(np.int32)
    rng = np.random.default_rng(2)
    row_pair = rng.permutation(pairs).astype(np.int32)
    R = row_pair.size
    off = _segments([30, 0, R - 30])
    A = synth.activations(R, K, 6, 41)
    gen = synth.weights_q8 if qbits == 8 else synth.weights_q4
    Wq = gen(E * N, K, 6, 42).reshape(E, N, -1)
    Ws = synth.scales(E * N, K // 32, 127 if qbits == 8 else 7, 6, 43).reshape(E, N, K // 32)
    w = rng.uniform(0.1, 1.0, M_tok * k).astype(np.float32)
    g = util.Guarded((M_tok, N), torch.float32, fill_inside=False)
    qg.moe_grouped_qgemm(qg.MODE_DOWN_ACCUM_F32, qbits, util.dev_bf16(A), util.dev(off), util.dev(Wq), util.dev_f16(Ws),
                         topk_w=util.dev(w), row_pair=util.dev(row_pair), k=k, out=g.t)
    qg.poll_status()
    assert g.intact(), "atomic add outside y"
    y = g.t.cpu().numpy().astype(np.float64)
    assert np.all(y[1::2] == 0.0) and np.all(g.t[1::2].view(torch.int32).cpu().numpy() == 0), "an unrouted token's row was touched"
    Dn = orc.grouped_gemm(qbits, orc.bf16_to_f64(A), off, Wq, Ws)
    ref = np.zeros((M_tok, N))
    np.add.at(ref, row_pair // k, Dn * w[row_pair].astype(np.float64)[:, None])
    util.assert_close(y, ref, "guarded accumulate")


def test_route_permute_combine_write_nothing_outside_their_outputs():
    M, E, k, H = 333, 24, 3, 136
    logits = synth.router_logits(M, E, seed=9)
    X = synth.activations(M, H, seed=10)
    G = util.Guarded
    i32, f32, b16 = torch.int32, torch.float32, torch.bfloat16
    gs = dict(topk_idx=G((M, k), i32), topk_w=G((M, k), f32), counts=G((E,), i32), offsets=G((E + 1,), i32),
              row_pair=G((M * k,), i32), pair_row=G((M * k,), i32), Xperm=G((M * k, H), b16))
    out = {key: g.t for key, g in gs.items()}
    for fn in (qg.moe_route, qg.moe_route_static):
        for g in gs.values():
            g.buf.fill_(g.sent)
        fn(util.dev(logits), k, X=util.dev_bf16(X), out=out)
        qg.poll_status()
        for key, g in gs.items():
            assert g.intact(), f"{fn.__name__}: store outside {key}"
        idx, w, _ = orc.route(logits, k)
        counts, offsets = orc.counts_offsets(idx, E)
        row_pair, pair_row = orc.permutation(idx, offsets)
        assert np.array_equal(out["topk_idx"].cpu().numpy(), idx)
        assert np.array_equal(out["offsets"].cpu().numpy(), offsets)
        assert np.array_equal(out["row_pair"].cpu().numpy(), row_pair)
        assert np.array_equal(out["pair_row"].cpu().numpy(), pair_row)
        assert np.array_equal(util.host_bf16_bits(out["Xperm"]), orc.permute(X, row_pair, k))
    gp = G((M * k, H), b16)
    qg.moe_permute(util.dev_bf16(X), out["row_pair"], k, out=gp.t)
    gy = G((M, H), b16)
    qg.moe_combine(out["Xperm"], out["pair_row"], k, out=gy.t)
    gz = G((M, H), b16)
    acc = torch.randn(M, H, device="cuda")
    qg.moe_combine(acc, None, k, d_kind=qg.D_F32_ACC, out=gz.t)
    qg.poll_status()
    assert gp.intact() and gy.intact() and gz.intact()
    assert torch.equal(gp.t, out["Xperm"]) and torch.equal(gz.t, acc.to(torch.bfloat16))
    util.assert_close(util.host_bf16_f64(gy.t), orc.combine(util.host_bf16_f64(out["Xperm"]), pair_row, k), "guarded combine")
