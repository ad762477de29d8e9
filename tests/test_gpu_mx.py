"""GPU parity of the block-scaled FP8 path: the two re-encoding kernels bit for bit against the oracle's definition
(codes and scale bytes), the GEMM against the oracle's exact product of the same encoded operands, and the end-to-end
error of the re-encoded path against the bf16 x Q8 product it replaces (reported, with a loose bound)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def _check_encoding(codes, sf_tiles, x64, rows, K):
    want_c, want_s = orc.mx_quantize(x64)
    got_s = synth.mx_scale_plain(sf_tiles.cpu().numpy(), rows, K)
    assert np.array_equal(got_s, want_s), "scale bytes"
    assert np.array_equal(codes.cpu().numpy(), want_c), "element codes"
    # padding rows of the last scale tile carry 2^0
    full = sf_tiles.cpu().numpy()[:((rows + 127) // 128) * (K // 128) * 512]
    assert np.array_equal(synth.mx_scale_tiles(want_s), full)


@pytest.mark.parametrize("rows,K", [(128, 128), (300, 256), (1, 384), (257, 2048)])
def test_quantize_rows_bit_exact(rows, K):
    bits = synth.activations(rows, K, seed=rows + K)
    x = synth.bf16_bits_to_f32(bits)
    x[0, :32] = 0.0                                          # an all-zero block
    if rows > 2:
        x[1, :64] *= 1e-30; x[2, 5] = 3.0e38                 # tiny and huge blocks
        x[2, 40:44] = [448.0, 449.0, 480.0, 511.0]           # clamping inside a block whose maximum is below 512
    bits = synth.f32_to_bf16_bits(x)
    codes, sf = qg.mx_quantize(util.dev_bf16(bits))
    qg.poll_status()
    _check_encoding(codes, sf, orc.bf16_to_f64(bits), rows, K)


@pytest.mark.parametrize("qbits,N,K", [(8, 256, 256), (4, 200, 512), (8, 72, 1024)])
def test_pack_weights_bit_exact(qbits, N, K):
    _, Wq, Ws = synth.dense_problem(qbits, 1, N, K, seed=3)
    Ws = Ws.copy(); Ws[1, :] = 0; Ws[2, 0] = 1                # zero scales, a subnormal scale
    codes, sf = qg.mx_pack_weights(qbits, util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    _check_encoding(codes, sf, orc.dequant(qbits, Wq, Ws), N, K)


# the last two give every CTA pair three or more tiles (both accumulators reused), one of them with a single chunk per tile
SHAPES = [(128, 256, 128), (300, 392, 512), (1, 8, 128), (129, 264, 1024), (512, 2048, 2048), (2048, 2560, 2048),
          (2048, 4224, 256), (1000, 9216, 128),
          (2048, 2048, 2048), (1999, 2040, 2304)]       # one wave of 256-wide tiles: the single-accumulator shape


@pytest.mark.parametrize("M,N,K", SHAPES, ids=[f"{s[0]}x{s[1]}x{s[2]}" for s in SHAPES])
def test_mx_gemm_parity(M, N, K):
    """Operands encoded by the oracle (so the GEMM is tested on its own), product against the oracle's fp64 sum."""
    rng = np.random.default_rng(M + N)
    a, asf = orc.mx_quantize(synth.bf16_bits_to_f32(synth.activations(M, K, seed=5)).astype(np.float64))
    w, wsf = orc.mx_quantize(rng.standard_normal((N, K)) * 0.02)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.qgemm_mx_dense(util.dev(a), util.dev(synth.mx_scale_tiles(asf)), util.dev(w), util.dev(synth.mx_scale_tiles(wsf)), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    out = util.host_bf16_f64(g.t)
    if M * N * K <= 2 ** 28:
        ref = orc.mx_gemm(a, asf, w, wsf)
        mx, rmax, fro = util.assert_close(out, ref, f"mx gemm {M}x{N}x{K}")
        assert fro < 3e-3                                   # only the bf16 rounding of the output is left
    else:
        rows = np.unique(np.concatenate([[0, M - 1, 127, 128], rng.integers(0, M, 28)]))
        ref = orc.mx_gemm(a[rows], asf[rows], w, wsf)
        util.assert_close(out[rows], ref, f"mx gemm {M}x{N}x{K} (sampled rows)")


def test_mx_path_end_to_end_error_against_the_q8_product():
    """quantise activations + pack Q8 weights + GEMM, all on the GPU, against the fp64 product of the original
    operands: the re-encoding costs about 3 % relative Frobenius error (E4M3 has 3 mantissa bits on both operands)."""
    M, N, K = 256, 512, 1024
    A, Wq, Ws = synth.dense_problem(8, M, N, K, seed=7)
    ac, asf = qg.mx_quantize(util.dev_bf16(A))
    wc, wsf = qg.mx_pack_weights(8, util.dev(Wq), util.dev_f16(Ws))
    out = qg.qgemm_mx_dense(ac, asf, wc, wsf)
    qg.poll_status()
    ref = orc.qgemm_dense(8, A, Wq, Ws)
    mx, rmax, fro = util.errors(util.host_bf16_f64(out), ref)
    assert fro < 6e-2 and mx < 0.3 * rmax, (mx, rmax, fro)
    # and exactly the oracle's product of the GPU's own encoded operands
    ref2 = orc.mx_gemm(ac.cpu().numpy(), synth.mx_scale_plain(asf.cpu().numpy(), M, K), wc.cpu().numpy(),
                       synth.mx_scale_plain(wsf.cpu().numpy(), N, K))
    util.assert_close(util.host_bf16_f64(out), ref2, "mx gemm on the GPU's own encodings")
