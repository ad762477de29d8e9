"""GPU parity of qgemm_small_m (1..16 tokens, the weight-streaming call) against the fp64 oracle, through each of the
kernels that can serve it: the TMA-fed ring kernel with its K slices added through a thread-block cluster or through
the scratch, the small-block kernel, and the library's own choice."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu

SHAPES = [
    (8, 1, 2048, 2048), (4, 1, 2048, 2048), (8, 16, 2048, 2048), (4, 16, 3072, 3072),
    (8, 5, 200, 256),          # N not a multiple of the row tile, a single K slice
    (4, 3, 136, 768), (8, 7, 2560, 2048), (4, 16, 72, 4096), (8, 2, 2048, 8192), (4, 9, 1536, 2304),
    (8, 8, 1096, 5120),        # K slices of unequal length, a ragged last tile
]
# qg_test_gemv_mode: the library's choice, the ring kernel with and without clusters, the other kernels
MODES = [(0, "auto"), (2, "ring"), (3, "ring-scratch"), (4, "no-ring")]


@pytest.fixture(autouse=True)
def _restore_mode():
    yield
    qg.test_gemv_mode(0)


@pytest.mark.parametrize("mode,mname", MODES, ids=[m[1] for m in MODES])
@pytest.mark.parametrize("qbits,M,N,K", SHAPES, ids=[f"q{s[0]}-{s[1]}x{s[2]}x{s[3]}" for s in SHAPES])
def test_small_m_parity_and_guards(qbits, M, N, K, mode, mname):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=6)
    g = util.Guarded((M, N), torch.bfloat16)
    dA, dWq, dWs = util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws)
    qg.test_gemv_mode(mode)
    qg.qgemm_small_m(qbits, dA, dWq, dWs, out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    mx, rmax, fro = util.assert_close(util.host_bf16_f64(g.t), ref, f"small-M q{qbits} {M}x{N}x{K} {mname}")
    assert fro > 1e-4
    # fixed-order sums over the K phases and slices: a second run gives the same bits
    again = qg.qgemm_small_m(qbits, dA, dWq, dWs)
    qg.poll_status()
    assert torch.equal(again, g.t)


@pytest.mark.parametrize("qbits,M,N,K", [(4, 3, 19200, 4096), (8, 8, 19072, 6144), (8, 12, 18944, 2304)],
                         ids=["q4-two-phases", "q8-three-phases", "q8-16-tokens-two-phases"])
def test_small_m_ring_kernel_many_tiles_and_k_phases(qbits, M, N, K):
    """As many row tiles as SMs and K longer than the token slice a CTA keeps in shared memory: every CTA walks its
    tiles once per K phase and carries fp32 sums from phase to phase.  Sampled rows against the oracle, guards, and
    the same bits on a second run."""
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=9)
    dA, dWq, dWs = util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.test_gemv_mode(2)
    qg.qgemm_small_m(qbits, dA, dWq, dWs, out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([rng.integers(0, N, 600), np.arange(0, 300), np.arange(N - 300, N)]))
    ref = orc.qgemm_dense(qbits, A, Wq[rows], Ws[rows])
    util.assert_close(util.host_bf16_f64(g.t)[:, rows], ref, f"ring kernel q{qbits} {M}x{N}x{K}")
    again = qg.qgemm_small_m(qbits, dA, dWq, dWs)
    qg.poll_status()
    assert torch.equal(again, g.t)


@pytest.mark.parametrize("qbits,M,N,K,mode,skip", [(8, 4, 2048, 2048, 2, 1), (4, 16, 3072, 8192, 3, 0), (8, 3, 19072, 4096, 2, 5)],
                         ids=["cluster", "scratch-and-tickets", "phases"])
def test_small_m_ring_kernel_wait_that_runs_out(qbits, M, N, K, mode, skip):
    """The ring kernel's bounded waits: its first CTA never loads one weight stage, the consumers' wait for it expires,
    the launch ends with QG_ERR_TIMEOUT in the status word (every warp walks through the remaining barriers, the other
    CTAs of its cluster are not left waiting), and the next call on the context is correct."""
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=14)
    dA, dWq, dWs = util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws)
    qg.test_gemv_mode(mode)
    try:
        qg.test_inject(wait_limit_polls=2048, skip_kblock=skip)
        qg.qgemm_small_m(qbits, dA, dWq, dWs)
        assert qg.poll_status_code() == -7
        assert qg.poll_status_code() == 0
    finally:
        qg.test_inject(0, -1)
    out = qg.qgemm_small_m(qbits, dA, dWq, dWs)
    assert qg.poll_status_code() == 0
    rows = np.arange(0, N, max(1, N // 512))
    util.assert_close(util.host_bf16_f64(out)[:, rows], orc.qgemm_dense(qbits, A, Wq[rows], Ws[rows]), "after a timeout")


@pytest.mark.parametrize("mode", [2, 4], ids=["ring", "no-ring"])
@pytest.mark.parametrize("qbits", [8, 4])
def test_small_m_integer_exact_is_bit_exact(qbits, mode):
    M, N, K = 11, 264, 512
    rng = np.random.default_rng(17)
    A = synth.f32_to_bf16_bits(rng.integers(-1, 2, (M, K)).astype(np.float32))
    if qbits == 8:
        Wq = rng.integers(-3, 4, (N, K)).astype(np.int8)
        Wq[0, :] = 0; Wq[0, 5] = -128; Wq[1, :] = 0; Wq[1, 511] = 127
    else:
        Wq = rng.integers(0, 256, (N, K // 2)).astype(np.uint8)
        Wq[:, 16:] = 0x88
    Ws = (2.0 ** rng.integers(-3, 2, (N, K // 32))).astype(np.float16).view(np.uint16)
    qg.test_gemv_mode(mode)
    out = qg.qgemm_small_m(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    assert np.array_equal(ref, ref.astype(np.float32).astype(np.float64))
    assert np.array_equal(util.host_bf16_bits(out), orc.f64_to_bf16(ref))


@pytest.mark.parametrize("mode", [2, 4], ids=["ring", "no-ring"])
@pytest.mark.parametrize("qbits", [8, 4])
def test_small_m_extreme_scales_and_argument_checks(qbits, mode):
    M, N, K = 4, 128, 512
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=2)
    Ws = Ws.copy(); Wq = Wq.copy()
    Wq[::3, ::5] = -128 if qbits == 8 else 0x0F                # the most negative code (Q4: codes 15 and 0 in one byte)
    s = Ws.view(np.float16)
    s[0::4, :] = -s[0::4, :]
    s[1::4, 0] = 0.0
    Ws[2::4, :] = np.arange(1, K // 32 + 1, dtype=np.uint16)      # subnormal scales
    qg.test_gemv_mode(mode)
    out = qg.qgemm_small_m(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    util.assert_close(util.host_bf16_f64(out), ref, "extreme")
    assert np.any(util.host_bf16_f64(out)[:, 2::4] != 0.0), "subnormal scales were flushed to zero"
    A17 = torch.zeros((17, K), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(qg.QGemmError) as e:
        qg.qgemm_small_m(qbits, A17, util.dev(Wq), util.dev_f16(Ws))
    assert e.value.code == -2
    assert qg.qgemm_small_m(qbits, A17[:0], util.dev(Wq), util.dev_f16(Ws)).shape == (0, N)


@pytest.mark.parametrize("qbits,M,N,K", [(8, 16, 16384, 2048), (4, 16, 6144, 8192), (8, 12, 4096, 14336)],
                         ids=["q8-many-rows", "q4-48M-weights", "q8-long-k"])
def test_small_m_large_matrices_take_the_prefill_kernel(qbits, M, N, K):
    """With more than eight tokens, at 16384 rows or 48 M weights and more, the call is served by qgemm_dense's kernel (same numerics; the last bf16
    place may differ between runs, so only the oracle comparison and the guards are asserted)."""
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=7)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.qgemm_small_m(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws), out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    util.assert_close(util.host_bf16_f64(g.t), orc.qgemm_dense(qbits, A, Wq, Ws), f"small-M via prefill kernel q{qbits} {M}x{N}x{K}")


def test_gemv_mode_hook_rejects_contradictory_bits():
    for bad in (-1, 6, 7, 8):
        with pytest.raises(qg.QGemmError) as e:
            qg.test_gemv_mode(bad)
        assert e.value.code == -2
    qg.test_gemv_mode(5)          # never the ring kernel, and no clusters: accepted
    qg.test_gemv_mode(0)
