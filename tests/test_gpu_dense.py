"""GPU parity: qgemm_dense against the fp64 oracle (max|err| <= 2e-2 max|ref|, relative Frobenius <= 5e-3),
plus integer-exact cases that must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def run_dense(qbits, A, Wq, Ws):
    out = qg.qgemm_dense(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    return out


SHAPES = [
    (8, 128, 2048, 2048),    # config 0
    (4, 128, 2048, 2048),
    (8, 300, 384, 512),      # ragged token tail, three weight tiles
    (4, 300, 384, 512),
    (8, 1, 128, 256), (4, 1, 128, 256),
    (8, 17, 200, 256),       # N not a multiple of the weight tile
    (4, 513, 136, 768),      # three token tiles of 256 with a tail of 1
    (8, 257, 2560, 2048), (4, 1024, 3072, 1024),
]


@pytest.mark.parametrize("qbits,M,N,K", SHAPES, ids=[f"q{s[0]}-{s[1]}x{s[2]}x{s[3]}" for s in SHAPES])
def test_dense_parity(qbits, M, N, K):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=0)
    out = run_dense(qbits, A, Wq, Ws)
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    mx, rmax, fro = util.assert_close(util.host_bf16_f64(out), ref, f"dense q{qbits} {M}x{N}x{K}")
    assert fro > 1e-4, "suspiciously exact: is the reference rounded?"


@pytest.mark.parametrize("qbits", [8, 4])
def test_dense_integer_exact_is_bit_exact(qbits):
    """A in {-1,0,1}, small codes, power-of-two scales, K=256: every dequantised weight is exact in bf16 and every
    partial sum is exact in fp32 whatever the order, so the only rounding left is the final one to bf16 and the
    GPU must reproduce round-to-nearest-even of the oracle's exact value bit for bit."""
    M, N, K = 200, 256, 256
    rng = np.random.default_rng(11)
    A = synth.f32_to_bf16_bits(rng.integers(-1, 2, (M, K)).astype(np.float32))
    if qbits == 8:
        Wq = rng.integers(-3, 4, (N, K)).astype(np.int8)
        Wq[0, :] = 0; Wq[0, 5] = -128; Wq[1, :] = 0; Wq[1, 255] = 127
    else:
        Wq = rng.integers(0, 256, (N, K // 2)).astype(np.uint8)
        Wq[:, 8:] = 0x88                     # only the first 16 weights of each row are non-zero
    Ws = (2.0 ** rng.integers(-3, 2, (N, K // 32))).astype(np.float16).view(np.uint16)
    out = run_dense(qbits, A, Wq, Ws)
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    assert np.array_equal(ref, ref.astype(np.float32).astype(np.float64)), "case is not exact in fp32"
    assert np.array_equal(util.host_bf16_bits(out), orc.f64_to_bf16(ref))


@pytest.mark.parametrize("qbits", [8, 4])
def test_dense_extreme_codes_and_scales(qbits):
    """q = -128 / -8, negative, zero and subnormal fp16 scales (never flushed)."""
    M, N, K = 64, 128, 512
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=2)
    Ws = Ws.copy()
    if qbits == 8:
        Wq = Wq.copy(); Wq[::3, ::5] = -128
    else:
        Wq = Wq.copy(); Wq[::3, ::5] = 0x00      # both codes 0 -> q = -8
    s = Ws.view(np.float16)
    s[0::4, :] = -s[0::4, :]
    s[1::4, 0] = 0.0
    Ws[2::4, :] = np.arange(1, K // 32 + 1, dtype=np.uint16)      # subnormals 2^-24 .. 16 * 2^-24
    out = run_dense(qbits, A, Wq, Ws)
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    util.assert_close(util.host_bf16_f64(out), ref, "extreme")
    sub = util.host_bf16_f64(out)[:, 2::4]
    assert np.any(sub != 0.0), "subnormal scales were flushed to zero"
    util.assert_close(sub, ref[:, 2::4], "subnormal rows")


def test_dense_full_size_sampled_config1_gate_up():
    """Config 1 gate/up projection at M = 2048 (the bench's launch configuration), checked on sampled outputs that
    hit every 128-column and every 256-row tile."""
    qbits, M, N, K = 8, 2048, 16384, 2048
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=0)
    out = util.host_bf16_f64(run_dense(qbits, A, Wq, Ws))
    rng = np.random.default_rng(0)
    rows, cols = [], []
    for rt in range(M // 128):
        for ct in range(N // 128):
            rows.append(rt * 128 + rng.integers(0, 128, 2)); cols.append(ct * 128 + rng.integers(0, 128, 2))
    rows = np.concatenate(rows); cols = np.concatenate(cols)
    ref = orc.qgemm_dense_sample(qbits, A, Wq, Ws, rows, cols)
    util.assert_close(out[rows, cols], ref, "config 1 gate/up sampled")
    assert np.all(np.isfinite(out))


def _sampled_on_device(qbits, A, Wq, Ws, out, per_tile, seed, tile=128):
    """Compares `out` (device bf16 [M, N]) with the oracle on per_tile random elements of every 128 x 128 tile and on
    the four corners; only the sampled elements leave the device."""
    M, N = out.shape
    rng = np.random.default_rng(seed)
    rt, ct = np.meshgrid(np.arange((M + tile - 1) // tile), np.arange((N + tile - 1) // tile), indexing="ij")
    rows = np.minimum(rt.reshape(-1, 1) * tile + rng.integers(0, tile, (rt.size, per_tile)), M - 1).reshape(-1)
    cols = np.minimum(ct.reshape(-1, 1) * tile + rng.integers(0, tile, (ct.size, per_tile)), N - 1).reshape(-1)
    rows = np.concatenate([rows, [0, M - 1, M - 1, 0]]); cols = np.concatenate([cols, [0, N - 1, 0, N - 1]])
    got = out[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].to(torch.float64).cpu().numpy()
    assert bool(torch.isfinite(out.float()).all().item())
    ref = orc.qgemm_dense_sample(qbits, A, Wq, Ws, rows, cols)
    return util.assert_close(got, ref, f"sampled q{qbits} {M}x{N}x{A.shape[1]}")


# Short K with several full token tiles per SM pair: the tile boundary logic (accumulator hand-over, the helpers
# of the last epilogue) runs with fewer k-blocks per tile than the rings are deep.  2048 x 8192 runs as 192-token
# tiles (about five per pair), 128 x 57344 as 128-token tiles (three per pair).
SHORT_K = [(8, 2048, 8192, 256), (4, 2048, 8192, 256), (8, 2048, 8192, 512), (4, 2048, 8192, 512),
           (8, 128, 57344, 256), (4, 128, 57344, 512), (8, 1536, 8192, 256)]


@pytest.mark.parametrize("qbits,M,N,K", SHORT_K, ids=[f"q{c[0]}-{c[1]}x{c[2]}x{c[3]}" for c in SHORT_K])
def test_dense_short_k_many_tiles_per_pair(qbits, M, N, K):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=4)
    out = run_dense(qbits, A, Wq, Ws)
    _sampled_on_device(qbits, A, Wq, Ws, out, per_tile=8, seed=K + M)
    # and every element of the last token tile and of a middle one, where a stale accumulator would show
    for r0 in (M - 128, (M // 2) & ~127):
        ref = orc.qgemm_dense(qbits, A[r0:r0 + 128], Wq[:2048], Ws[:2048])
        util.assert_close(util.host_bf16_f64(out[r0:r0 + 128, :2048]), ref, f"rows {r0}..")


@pytest.mark.parametrize("qbits,M,F,K", [(8, 300, 256, 512), (4, 1000, 1024, 768), (8, 64, 64, 256), (4, 2048, 2048, 1024)],
                         ids=["q8-300", "q4-1000", "q8-64", "q4-2048"])
def test_dense_gate_up_with_fused_silu(qbits, M, F, K):
    A, Wq, Ws = synth.dense_problem(qbits, M, 2 * F, K, seed=9)
    g = util.Guarded((M, F), torch.bfloat16)
    qg.qgemm_dense_gate_up_silu(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    util.assert_close(util.host_bf16_f64(g.t), orc.silu_mul(orc.qgemm_dense(qbits, A, Wq, Ws)), "dense gate/up + silu")


def test_dense_many_distinct_weight_buffers_through_one_context():
    """A model has hundreds of weight matrices and one set of activation buffers: the activation map is found in the
    context's tensor-map cache on every call while weight maps keep replacing older entries.  Every call must use the
    maps of its own arguments (a cached entry handed out by reference and then replaced made the kernel copy with
    another buffer's map and run into its wait limit)."""
    qbits, M, N, K = 4, 16, 256, 256
    A, _, _ = synth.dense_problem(qbits, M, N, K, seed=11)
    dA = util.dev_bf16(A)
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    n_weights = 2600                                             # more than the cache holds
    Wq0 = synth.weights_q4(N, K, 11, 1)
    Ws = util.dev_f16(synth.scales(N, K // 32, 7, 11, 2))
    pool = torch.empty((n_weights, N, K // 2), dtype=torch.uint8, device="cuda")
    pool[:] = util.dev(Wq0)[None]
    marks = {0: 0x11, 1037: 0x5A, n_weights - 1: 0xC3}            # three buffers with their own codes in row 0
    for i, byte in marks.items():
        pool[i, 0, :] = byte
    results = {}
    for rep in range(2):
        for i in range(n_weights):
            qg.qgemm_dense(qbits, dA, pool[i], Ws, out=out)
            if i in marks:
                results[(rep, i)] = out.clone()
    qg.poll_status()
    for (rep, i), got in results.items():
        Wq = Wq0.copy(); Wq[0, :] = marks[i]
        util.assert_close(util.host_bf16_f64(got), orc.qgemm_dense(qbits, A, Wq, synth.scales(N, K // 32, 7, 11, 2)), f"buffer {i} pass {rep}")
