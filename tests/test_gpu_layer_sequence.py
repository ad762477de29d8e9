"""A model-like sequence on one context and one stream without a host synchronisation in between: many layers, each with
its own weight buffers, every layer running the dense projection, attention, the output projection, the router, routing,
both expert GEMMs and the combine, with a small-batch call on the side.  What it is for: the kernels follow each other
with programmatic dependent launch (a kernel's prologue overlaps the tail of the one before), they share the context's
scratch, counters and tensor-map cache, and a model has far more buffers than any single-operator test.  Checked: each
operator of sampled layers against the oracle on the inputs the GPU itself produced for it (so errors do not add up
along the chain), routing bit for bit, and a second pass over all layers (every cache and counter in the state the first
pass left) agreeing with the first where its inputs are the same."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu

M, H, F, E, TOPK = 96, 256, 256, 8, 2
HQ, HKV, D = 4, 2, 64
NQKV = (HQ + 2 * HKV) * D
LAYERS = 48


def _layer_weights(l):
    gen8, gen4 = synth.weights_q8, synth.weights_q4
    w = {
        "qkv": (gen8(NQKV, H, l, 1), synth.scales(NQKV, H // 32, 127, l, 2)),
        "o": (gen4(H, HQ * D, l, 3), synth.scales(H, HQ * D // 32, 7, l, 4)),
        "router": synth.activations(E, H, seed=l, tid=5),
        "w1": (gen4(E * 2 * F, H, l, 6).reshape(E, 2 * F, -1), synth.scales(E * 2 * F, H // 32, 7, l, 7).reshape(E, 2 * F, H // 32)),
        "w2": (gen8(E * H, F, l, 8).reshape(E, H, F), synth.scales(E * H, F // 32, 127, l, 9).reshape(E, H, F // 32)),
        "head": (gen4(512, H, l, 10), synth.scales(512, H // 32, 7, l, 11)),
    }
    return w


def _to_dev(w):
    d = {}
    for k, v in w.items():
        if k == "router":
            d[k] = util.dev_bf16(v)
        else:
            d[k] = (util.dev(v[0]), util.dev_f16(v[1]))
    return d


def _forward(x0, dw, keep):
    """One pass over all layers; returns {layer: tensors} for the layers in `keep` (clones taken on the stream)."""
    kept = {}
    x = x0
    for l, w in enumerate(dw):
        qkv = qg.qgemm_dense(8, x, *w["qkv"])
        q, k, v = qkv[:, :HQ * D], qkv[:, HQ * D:(HQ + HKV) * D], qkv[:, (HQ + HKV) * D:]
        att = qg.prefill_attention(q, k, v, HQ, HKV, D, causal=True)
        y = qg.qgemm_dense(4, att, *w["o"])
        logits = qg.moe_router_logits(y, w["router"])
        ro = qg.moe_route(logits, TOPK, X=y)
        hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, 4, ro["Xperm"], ro["offsets"], *w["w1"])
        dwt = qg.moe_grouped_qgemm(qg.MODE_DOWN_WEIGHTED, 8, hh, ro["offsets"], *w["w2"], topk_w=ro["topk_w"].view(-1),
                                   row_pair=ro["row_pair"], k=TOPK)
        out = qg.moe_combine(dwt, ro["pair_row"], TOPK)
        head = qg.qgemm_small_m(4, out[:5], *w["head"])            # a decode-sized call between the prefill calls
        if l in keep:
            kept[l] = {"x": x, "qkv": qkv, "att": att, "y": y, "logits": logits, "idx": ro["topk_idx"], "tw": ro["topk_w"],
                       "row_pair": ro["row_pair"], "pair_row": ro["pair_row"], "offsets": ro["offsets"], "xperm": ro["Xperm"],
                       "hh": hh, "dw": dwt, "out": out, "head": head}
        x = (out.float() * (1.0 / out.float().std().clamp_min(1e-30))).to(torch.bfloat16)   # unit scale for the next layer (plumbing)
    return kept


def test_many_layers_back_to_back_match_the_oracle_and_repeat():
    host = [_layer_weights(l) for l in range(LAYERS)]
    dw = [_to_dev(w) for w in host]
    x0 = util.dev_bf16(synth.activations(M, H, seed=77, tid=1))
    keep = (0, 17, LAYERS - 1)
    a = _forward(x0, dw, keep)
    b = _forward(x0, dw, keep)
    qg.poll_status()
    f64 = util.host_bf16_f64
    bits = util.host_bf16_bits
    for l in keep:
        t, w = a[l], host[l]
        name = f"layer {l}"
        util.assert_close(f64(t["qkv"]), orc.qgemm_dense(8, bits(t["x"]), *w["qkv"]), name + " qkv")
        qkvb = bits(t["qkv"])
        util.assert_close(f64(t["att"]), orc.attention(qkvb[:, :HQ * D], qkvb[:, HQ * D:(HQ + HKV) * D], qkvb[:, (HQ + HKV) * D:],
                                                      HQ, HKV, D, causal=True), name + " attention")
        util.assert_close(f64(t["y"]), orc.qgemm_dense(4, bits(t["att"]), *w["o"]), name + " o")
        ref_logits = orc.router_logits(orc.bf16_to_f64(bits(t["y"])), orc.bf16_to_f64(w["router"]))
        assert np.max(np.abs(t["logits"].cpu().numpy().astype(np.float64) - ref_logits)) <= 1e-4 * max(1.0, np.abs(ref_logits).max())
        gl = t["logits"].cpu().numpy()
        idx, tw, _ = orc.route(gl, TOPK)                              # routing of the logits the GPU produced: bit for bit
        counts, offsets = orc.counts_offsets(idx, E)
        row_pair, pair_row = orc.permutation(idx, offsets)
        assert np.array_equal(t["idx"].cpu().numpy(), idx) and np.array_equal(t["offsets"].cpu().numpy(), offsets)
        assert np.array_equal(t["row_pair"].cpu().numpy(), row_pair) and np.array_equal(t["pair_row"].cpu().numpy(), pair_row)
        assert np.array_equal(bits(t["xperm"]), orc.permute(bits(t["y"]), row_pair, TOPK))
        gu = orc.grouped_gemm(4, orc.bf16_to_f64(bits(t["xperm"])), offsets, *w["w1"])
        util.assert_close(f64(t["hh"]), orc.silu_mul(gu), name + " gate/up")
        dn = orc.grouped_gemm(8, orc.bf16_to_f64(bits(t["hh"])), offsets, *w["w2"])
        gw = t["tw"].cpu().numpy().reshape(-1).astype(np.float64)
        util.assert_close(f64(t["dw"]), dn * gw[row_pair][:, None], name + " down")
        util.assert_close(f64(t["out"]), orc.combine(orc.bf16_to_f64(bits(t["dw"])), pair_row, TOPK), name + " combine")
        util.assert_close(f64(t["head"]), orc.qgemm_dense(4, bits(t["out"])[:5], *w["head"]), name + " small batch")
        # the second pass ran on the same inputs with every cache and counter in the state the first pass left
        if l == 0:
            util.assert_close(f64(b[l]["qkv"]), f64(t["qkv"]), name + " second pass")
            util.assert_close(f64(b[l]["att"]), f64(t["att"]), name + " second pass, attention")
