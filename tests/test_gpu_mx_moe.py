"""GPU parity of the grouped block-scaled FP8 path: qg_mx_quantize_grouped bit for bit against the oracle's encoding,
moe_grouped_qgemm_mx against the oracle's per-segment product of the same encoded operands."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def _segments(counts):
    offsets = np.zeros(len(counts) + 1, np.int32)
    offsets[1:] = np.cumsum(counts)
    return offsets


@pytest.mark.parametrize("counts,K", [([5], 128), ([0, 130, 0, 1, 128, 300], 256), ([64] * 9, 512)])
def test_quantize_grouped_bit_exact(counts, K):
    offsets = _segments(counts)
    R = int(offsets[-1])
    bits = synth.activations(R, K, seed=R + K, tid=81)
    codes, sf = qg.mx_quantize_grouped(util.dev_bf16(bits), util.dev(offsets))
    qg.poll_status()
    ref_codes, ref_sf = orc.mx_quantize(orc.bf16_to_f64(bits))
    assert np.array_equal(codes.cpu().numpy(), ref_codes)
    want = synth.mx_scale_tiles_grouped(ref_sf, offsets)
    got = sf.cpu().numpy()[:want.size]
    # padding rows of a segment's last tile: the library writes 0 (2^-127), the host helper 127; compare real rows only
    tiles = 0
    for e, c in enumerate(counts):
        if c == 0:
            continue
        nt = (c + 127) // 128
        g = synth.mx_scale_plain(got[tiles * (K // 128) * 512:(tiles + nt) * (K // 128) * 512], nt * 128, K)
        assert np.array_equal(g[:c], ref_sf[offsets[e]:offsets[e + 1]]), f"segment {e}"
        assert np.all(g[c:] == 0)
        tiles += nt


CASES = [
    ("plain-small", qg.MODE_PLAIN, [5, 0, 130], 192, 128), ("plain-ragged-n", qg.MODE_PLAIN, [200, 64, 1], 448, 256),
    ("gate-up", qg.MODE_GATE_UP_SILU, [128, 129, 0, 7], 2 * 320, 256), ("gate-up-one-tile", qg.MODE_GATE_UP_SILU, [40], 2 * 64, 128),
    ("weighted", qg.MODE_DOWN_WEIGHTED, [300, 10, 128, 128], 384, 384),
    ("many-tiles", qg.MODE_PLAIN, [96] * 40, 1152, 128),          # 240 tiles: every CTA reuses both accumulators
]


@pytest.mark.parametrize("name,mode,counts,N,K", CASES, ids=[c[0] for c in CASES])
def test_grouped_mx_gemm_parity(name, mode, counts, N, K):
    rng = np.random.default_rng(len(counts) + N)
    offsets = _segments(counts)
    R, E = int(offsets[-1]), len(counts)
    a, asf = orc.mx_quantize(synth.bf16_bits_to_f32(synth.activations(R, K, seed=7, tid=82)).astype(np.float64))
    w = np.zeros((E, N, K), np.uint8); wsf = np.zeros((E, N, K // 32), np.uint8)
    for e in range(E):
        w[e], wsf[e] = orc.mx_quantize(rng.standard_normal((N, K)) * 0.05)
    row_pair = rng.permutation(R).astype(np.int32)
    tw = rng.uniform(0.1, 1.0, R).astype(np.float32)
    cols = N // 2 if mode == qg.MODE_GATE_UP_SILU else N
    g = util.Guarded((R, cols), torch.bfloat16)
    qg.moe_grouped_qgemm_mx(mode, util.dev(a), util.dev(synth.mx_scale_tiles_grouped(asf, offsets)), util.dev(offsets),
                            util.dev(w.reshape(E * N, K)), util.dev(synth.mx_scale_tiles(wsf.reshape(E * N, K // 32))), N,
                            topk_w=util.dev(tw), row_pair=util.dev(row_pair), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.mx_grouped_gemm(a, asf, offsets, w, wsf)
    if mode == qg.MODE_GATE_UP_SILU:
        ref = orc.silu_mul(ref)
    elif mode == qg.MODE_DOWN_WEIGHTED:
        ref = ref * tw[row_pair].astype(np.float64)[:, None]
    util.assert_close(util.host_bf16_f64(g.t), ref, f"grouped mx {name}")


def test_grouped_mx_layer_on_the_gpu_against_the_q4_layer():
    """The routed layer with both expert projections on the block-scaled path (weights packed from Q4, activations
    re-encoded on the GPU) against the fp64 layer over the original operands: bounds the format's own error."""
    qbits, M, H, E, F, k = 4, 256, 512, 8, 384, 2
    logits, Xb, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=21)
    r = qg.moe_route(util.dev(logits), k, X=util.dev_bf16(Xb))
    w1c, w1s = qg.mx_pack_weights(qbits, util.dev(W1q.reshape(E * 2 * F, -1)), util.dev_f16(W1s.reshape(E * 2 * F, -1)))
    w2c, w2s = qg.mx_pack_weights(qbits, util.dev(W2q.reshape(E * H, -1)), util.dev_f16(W2s.reshape(E * H, -1)))
    ac, asf = qg.mx_quantize_grouped(r["Xperm"], r["offsets"])
    Hh = qg.moe_grouped_qgemm_mx(qg.MODE_GATE_UP_SILU, ac, asf, r["offsets"], w1c, w1s, 2 * F)
    hc, hsf = qg.mx_quantize_grouped(Hh, r["offsets"])
    Dw = qg.moe_grouped_qgemm_mx(qg.MODE_DOWN_WEIGHTED, hc, hsf, r["offsets"], w2c, w2s, H, topk_w=r["topk_w"].view(-1),
                                 row_pair=r["row_pair"])
    y = qg.moe_combine(Dw, r["pair_row"], k)
    qg.poll_status()
    o = orc.moe_layer(qbits, logits, Xb, W1q, W1s, W2q, W2s, k)
    mx, rmax, fro = util.errors(util.host_bf16_f64(y), o["y"])
    assert np.all(np.isfinite(util.host_bf16_f64(y))) and fro < 8e-2 and mx < 0.4 * rmax, (mx, rmax, fro)
