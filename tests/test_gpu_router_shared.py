"""GPU parity of the router projection (hidden -> experts) and of the combine that adds a shared expert."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,H,E", [(1, 64, 1), (64, 64, 64), (70, 128, 130), (333, 2048, 128), (2048, 2048, 128),
                                   (129, 3072, 8), (500, 256, 1000)],
                         ids=lambda v: str(v))
def test_router_logits_parity(M, H, E):
    """Several tiles with ragged tails in both directions; fp32 logits against the fp64 sum of the same bf16 inputs
    (products exact, so only the fp32 accumulation differs: far inside the float tolerance)."""
    xb = synth.activations(M, H, seed=M + E, tid=31)
    wb = synth.f32_to_bf16_bits((synth.bf16_bits_to_f32(synth.activations(E, H, seed=H, tid=32)) * 0.05).astype(np.float32))
    g = util.Guarded((M, E), torch.float32)
    qg.moe_router_logits(util.dev_bf16(xb), util.dev_bf16(wb), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.router_logits(orc.bf16_to_f64(xb), orc.bf16_to_f64(wb))
    out = g.t.detach().cpu().numpy().astype(np.float64)
    mx, rmax, fro = util.errors(out, ref)
    assert np.all(np.isfinite(out)) and fro < 1e-5 and mx < 1e-4 * max(rmax, 1.0), (mx, rmax, fro)


def test_router_logits_are_reproducible_and_feed_route():
    """Two runs give the same bits; routing the GPU's logits on the GPU equals the oracle's routing of the same logits."""
    M, H, E, k = 300, 512, 64, 4
    xb = synth.activations(M, H, seed=9, tid=33)
    wb = synth.activations(E, H, seed=10, tid=34)
    X, Wr = util.dev_bf16(xb), util.dev_bf16(wb)
    l1 = qg.moe_router_logits(X, Wr)
    l2 = qg.moe_router_logits(X, Wr)
    assert torch.equal(l1, l2)
    r = qg.moe_route(l1, k)
    qg.poll_status()
    idx, _, w32 = orc.route(l1.cpu().numpy(), k)
    assert np.array_equal(r["topk_idx"].cpu().numpy().reshape(idx.shape), idx)
    assert np.allclose(r["topk_w"].cpu().numpy().reshape(w32.shape), w32, atol=1e-6, rtol=0)


def test_router_logits_rejects_bad_shapes():
    X = torch.zeros((4, 96), dtype=torch.bfloat16, device="cuda")
    Wr = torch.zeros((8, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(qg.QGemmError):
        qg.moe_router_logits(X, Wr)                     # H % 64 != 0
    out = qg.moe_router_logits(torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda"),
                               torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda"))
    assert out.shape == (0, 8)


@pytest.mark.parametrize("M,H,k,weighted", [(1, 8, 1, True), (37, 264, 3, True), (512, 2048, 8, False), (100, 1024, 8, True)])
def test_combine_shared_parity(M, H, k, weighted):
    rng = np.random.default_rng(M + H)
    Db = synth.activations(M * k, H, seed=3, tid=35)
    Sb = synth.activations(M, H, seed=4, tid=36)
    pair_row = rng.permutation(M * k).astype(np.int32)
    w = rng.uniform(0.0, 1.0, (M, k)).astype(np.float32) if weighted else None
    g = util.Guarded((M, H), torch.bfloat16)
    qg.moe_combine(util.dev_bf16(Db), util.dev(pair_row), k, topk_w=util.dev(w) if weighted else None, out=g.t,
                   shared=util.dev_bf16(Sb))
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.combine_shared(orc.bf16_to_f64(Db), pair_row, k, orc.bf16_to_f64(Sb),
                             w.astype(np.float64) if weighted else None)
    util.assert_close(util.host_bf16_f64(g.t), ref, "combine + shared expert")
    # a zero shared expert gives the plain combine, bit for bit
    y0 = qg.moe_combine(util.dev_bf16(Db), util.dev(pair_row), k, topk_w=util.dev(w) if weighted else None)
    yz = qg.moe_combine(util.dev_bf16(Db), util.dev(pair_row), k, topk_w=util.dev(w) if weighted else None,
                        shared=torch.zeros((M, H), dtype=torch.bfloat16, device="cuda"))
    assert torch.equal(y0, yz)


def test_layer_with_router_and_shared_expert():
    """The whole routed layer from the hidden states: router projection, routing, expert FFNs, plus a shared dense FFN,
    against the oracle's unrounded fp64 composition of the same steps (the oracle routes the GPU's logits, since a
    one-ulp difference in a logit may legitimately flip a near-tie)."""
    qbits, M, H, E, F, k, Fs = 4, 200, 512, 16, 256, 4, 512
    _, Xb, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=12)
    wrb = synth.f32_to_bf16_bits((synth.bf16_bits_to_f32(synth.activations(E, H, seed=13, tid=37)) * 0.05).astype(np.float32))
    _, S1q, S1s = synth.dense_problem(qbits, 1, 2 * Fs, H, seed=14)
    _, S2q, S2s = synth.dense_problem(qbits, 1, H, Fs, seed=15)
    X = util.dev_bf16(Xb)
    logits = qg.moe_router_logits(X, util.dev_bf16(wrb))
    r = qg.moe_route(logits, k, X=X)
    Hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, qbits, r["Xperm"], r["offsets"], util.dev(W1q), util.dev_f16(W1s))
    Dw = qg.moe_grouped_qgemm(qg.MODE_DOWN_WEIGHTED, qbits, Hh, r["offsets"], util.dev(W2q), util.dev_f16(W2s),
                              topk_w=r["topk_w"].view(-1), row_pair=r["row_pair"], k=k)
    sh = qg.qgemm_dense(qbits, qg.qgemm_dense_gate_up_silu(qbits, X, util.dev(S1q), util.dev_f16(S1s)), util.dev(S2q),
                        util.dev_f16(S2s))
    y = qg.moe_combine(Dw, r["pair_row"], k, shared=sh)
    qg.poll_status()
    # logits against the oracle's, then the rest of the layer from the GPU's logits
    lg = logits.cpu().numpy()
    ref_l = orc.router_logits(orc.bf16_to_f64(Xb), orc.bf16_to_f64(wrb))
    assert np.max(np.abs(lg - ref_l)) < 1e-4 * max(1.0, np.max(np.abs(ref_l)))
    o = orc.moe_layer(qbits, lg, Xb, W1q, W1s, W2q, W2s, k)
    one = np.array([0, M], np.int32)                                 # the shared expert: one segment over all tokens
    shared64 = orc.grouped_gemm(qbits, orc.silu_mul(orc.qgemm_dense(qbits, Xb, S1q, S1s)), one, S2q[None], S2s[None])
    util.assert_close(util.host_bf16_f64(y), o["y"] + shared64, "layer with router and shared expert")
