"""GPU parity at the benchmark's full sizes, in the launch configurations bench.py times, on sampled outputs the oracle
can compute one by one (dense) or on whole expert segments (MoE)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def _sampled_dense(qbits, M, N, K, seed, per_tile=2, tile=128):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=seed)
    out = qg.qgemm_dense(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    out = util.host_bf16_f64(out)
    rng = np.random.default_rng(seed)
    rows, cols = [], []
    for rt in range((M + tile - 1) // tile):
        for ct in range((N + tile - 1) // tile):
            rows.append(np.minimum(rt * tile + rng.integers(0, tile, per_tile), M - 1))
            cols.append(np.minimum(ct * tile + rng.integers(0, tile, per_tile), N - 1))
    # plus the last row / column (ragged edges) and the first ones
    rows.append(np.array([0, M - 1, M - 1, 0])); cols.append(np.array([0, N - 1, 0, N - 1]))
    rows = np.concatenate(rows); cols = np.concatenate(cols)
    ref = orc.qgemm_dense_sample(qbits, A, Wq, Ws, rows, cols)
    assert np.all(np.isfinite(out))
    return util.assert_close(out[rows, cols], ref, f"q{qbits} {M}x{N}x{K}")


# config 1 (2B-class Q8), config 2 (Llama-3.2-3B-shaped Q4), config 4 (8B-class Q8): one GEMM of each kind
FULL = [
    (8, 2048, 2560, 2048), (8, 2048, 2048, 8192), (8, 1024, 16384, 2048), (8, 1000, 2048, 2048),
    (4, 2048, 5120, 3072), (4, 2048, 3072, 8192), (4, 512, 16384, 3072),
    (8, 2048, 6144, 4096), (8, 4096, 4096, 14336), (8, 8192, 4096, 4096),
]


@pytest.mark.parametrize("qbits,M,N,K", FULL, ids=[f"q{c[0]}-{c[1]}x{c[2]}x{c[3]}" for c in FULL])
def test_dense_full_size_sampled(qbits, M, N, K):
    _sampled_dense(qbits, M, N, K, seed=0, per_tile=1 if M * N > 2 ** 24 else 2)


@pytest.mark.parametrize("M,skewed", [(2048, False), (2048, True), (1024, False), (4096, False), (8192, False), (8192, True)],
                         ids=["uniform-2048", "skewed-2048", "uniform-1024", "uniform-4096", "uniform-8192", "skewed-8192"])
def test_moe_config3_full_size_selected_experts(M, skewed):
    """Config 3 (H=2048, E=128, top-8, F=768, Q4) at the bench's token counts.  Routing and permutation are compared in
    full (bit exact); the two GEMM stages are compared on every row of a few experts (the busiest, the least busy and
    two others), each stage fed with exactly what the GPU stage consumed; the layer output is then checked through
    the combine stage on the GPU's own weighted rows."""
    qbits, H, E, F, k = 4, 2048, 128, 768, 8
    logits, X, W1q, W1s, W2q, W2s = synth.moe_problem(qbits, M, H, E, F, seed=0, skewed=skewed)
    d = dict(logits=util.dev(logits), X=util.dev_bf16(X), W1q=util.dev(W1q), W1s=util.dev_f16(W1s),
             W2q=util.dev(W2q), W2s=util.dev_f16(W2s))
    r = qg.moe_route(d["logits"], k, X=d["X"])
    Hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, qbits, r["Xperm"], r["offsets"], d["W1q"], d["W1s"])
    Dw = qg.moe_grouped_qgemm(qg.MODE_DOWN_WEIGHTED, qbits, Hh, r["offsets"], d["W2q"], d["W2s"],
                              topk_w=r["topk_w"].view(-1), row_pair=r["row_pair"], k=k)
    y = qg.moe_combine(Dw, r["pair_row"], k)
    qg.poll_status()
    idx, w, _ = orc.route(logits, k)
    counts, offsets = orc.counts_offsets(idx, E)
    row_pair, pair_row = orc.permutation(idx, offsets)
    assert np.array_equal(r["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(r["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(r["row_pair"].cpu().numpy(), row_pair)
    assert np.array_equal(r["pair_row"].cpu().numpy(), pair_row)
    Xp = orc.permute(X, row_pair, k)
    assert np.array_equal(util.host_bf16_bits(r["Xperm"]), Xp)
    w_gpu = r["topk_w"].cpu().numpy().astype(np.float64).reshape(-1)
    experts = sorted({int(np.argmax(counts)), int(np.argmin(counts)), 5, 64})
    for e in experts:
        seg = slice(int(offsets[e]), int(offsets[e + 1]))
        if seg.stop == seg.start:
            continue
        off1 = np.array([0, seg.stop - seg.start], np.int32)
        Hh_e = util.host_bf16_f64(Hh[seg])
        GU = orc.grouped_gemm(qbits, orc.bf16_to_f64(Xp[seg]), off1, W1q[e:e + 1], W1s[e:e + 1])
        util.assert_close(Hh_e, orc.silu_mul(GU), f"gate/up expert {e}")
        Dn = orc.grouped_gemm(qbits, Hh_e, off1, W2q[e:e + 1], W2s[e:e + 1])
        util.assert_close(util.host_bf16_f64(Dw[seg]), Dn * w_gpu[row_pair[seg]][:, None], f"down expert {e}")
    assert bool(torch.isfinite(Hh.float()).all().item()) and bool(torch.isfinite(Dw.float()).all().item())
    # combine on the GPU's own weighted rows: all tokens up to M = 2048, else the first and the last 512 tokens
    yh = util.host_bf16_f64(y)
    assert np.all(np.isfinite(yh))
    toks = np.arange(M) if M <= 2048 else np.concatenate([np.arange(512), np.arange(M - 512, M)])
    rows_needed = pair_row.reshape(M, k)[toks].reshape(-1)
    D_sub = util.host_bf16_f64(Dw[torch.from_numpy(rows_needed.astype(np.int64)).cuda()])
    sub_pair_row = np.arange(rows_needed.size, dtype=np.int32)            # token i of the subset owns rows i k .. i k + k - 1
    util.assert_close(yh[toks], orc.combine(D_sub, sub_pair_row, k), "combine")
    # the fused flavour the benchmark times: rows gathered by the gate/up kernel's loads, fp32 accumulate in the down
    # epilogue, one rounding.  Gate/up again on the selected experts' rows, then the layer output on sampled tokens.
    Hh_f = qg.moe_grouped_qgemm_gather(qg.MODE_GATE_UP_SILU, qbits, d["X"], r["row_pair"], k, r["offsets"], d["W1q"], d["W1s"])
    acc = qg.moe_grouped_qgemm(qg.MODE_DOWN_ACCUM_F32, qbits, Hh_f, r["offsets"], d["W2q"], d["W2s"],
                               topk_w=r["topk_w"].view(-1), row_pair=r["row_pair"], k=k, M=M)
    y_f = qg.moe_combine(acc, None, k, d_kind=qg.D_F32_ACC)
    qg.poll_status()
    for e in experts:
        seg = slice(int(offsets[e]), int(offsets[e + 1]))
        if seg.stop == seg.start:
            continue
        off1 = np.array([0, seg.stop - seg.start], np.int32)
        GU = orc.grouped_gemm(qbits, orc.bf16_to_f64(Xp[seg]), off1, W1q[e:e + 1], W1s[e:e + 1])
        util.assert_close(util.host_bf16_f64(Hh_f[seg]), orc.silu_mul(GU), f"gathered gate/up expert {e}")
    yf = util.host_bf16_f64(y_f)
    assert np.all(np.isfinite(yf))
    # the accumulated layer output on 48 sampled tokens: the oracle's down projection of the GPU's own gate/up rows,
    # weighted with the GPU's routing weights and summed in fp64
    rng = np.random.default_rng(M)
    sample = np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, 46)]))
    y_ref = np.zeros((sample.size, H))
    one = np.array([0, 1], np.int32)
    for i, t in enumerate(sample):
        for s_ in range(k):
            row = int(pair_row[t * k + s_]); e = int(idx[t, s_])
            h = util.host_bf16_f64(Hh_f[row:row + 1])
            y_ref[i] += w_gpu[t * k + s_] * orc.grouped_gemm(qbits, h, one, W2q[e:e + 1], W2s[e:e + 1])[0]
    util.assert_close(yf[sample], y_ref, "layer output of the fused path on sampled tokens")


def test_config4_gate_up_projection_sampled():
    """Config 4's largest dense launch: M = 8192 tokens, N = 2 x 14336, K = 4096 (224 weight tiles, 32 token tiles), one
    sampled element in every 128 x 128 output tile plus the corners."""
    from tests.test_gpu_dense import _sampled_on_device
    qbits, M, N, K = 8, 8192, 28672, 4096
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=0)
    out = qg.qgemm_dense(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    _sampled_on_device(qbits, A, Wq, Ws, out, per_tile=1, seed=4)


# the small-batch rows of the bench's sweep: every projection of the cfg-1 (Q8) and cfg-2 (Q4) layer sets at 1, 4 and 16
# tokens, plus the largest cfg-4 matrices, through qgemm_small_m as the library dispatches it
SMALL_M = [(8, M, N, K) for M in (1, 4, 16) for N, K in ((2560, 2048), (2048, 2048), (16384, 2048), (2048, 8192))] + \
          [(4, M, N, K) for M in (1, 4, 16) for N, K in ((5120, 3072), (3072, 3072), (16384, 3072), (3072, 8192))] + \
          [(8, 4, 28672, 4096), (8, 8, 4096, 14336), (4, 2, 28672, 4096)]


@pytest.mark.parametrize("qbits,M,N,K", SMALL_M, ids=[f"q{c[0]}-{c[1]}x{c[2]}x{c[3]}" for c in SMALL_M])
def test_small_m_full_size_sampled_rows(qbits, M, N, K):
    """All tokens against a sample of weight rows: a few in every 128-row tile (the unit a CTA of the ring kernel owns),
    the first and the last rows."""
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=3)
    out = qg.qgemm_small_m(qbits, util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws))
    qg.poll_status()
    out = util.host_bf16_f64(out)
    rng = np.random.default_rng(N + K + M)
    tiles = (N + 127) // 128
    rows = np.unique(np.concatenate([np.minimum(np.arange(tiles) * 128 + rng.integers(0, 128, tiles), N - 1),
                                     np.minimum(np.arange(tiles) * 128 + rng.integers(0, 128, tiles), N - 1),
                                     np.arange(0, 8), np.arange(N - 8, N)]))
    assert np.all(np.isfinite(out))
    util.assert_close(out[:, rows], orc.qgemm_dense(qbits, A, Wq[rows], Ws[rows]), f"small-M q{qbits} {M}x{N}x{K}")
