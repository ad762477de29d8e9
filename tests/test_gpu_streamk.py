"""Stream-K scheduling of qgemm_dense: the k-blocks of all tiles are dealt out evenly over the SM pairs, tiles cut in
the middle are completed from fp32 partials in the context's scratch.  Forced on (and off) for every token tile and
for shapes whose tiles split into two, three and many parts; the result must match the oracle either way and the
scratch counters must be back at zero afterwards (a second, different call right after must be correct too)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util
from tests.test_gpu_dense import _sampled_on_device

pytestmark = pytest.mark.gpu

SHAPES = [
    (8, 2048, 2560, 2048),     # 80 / 110 / 160 tiles on 74 pairs
    (4, 1024, 2048, 2048),     # fewer tiles than pairs: every tile is cut into several parts
    (8, 300, 384, 512),        # ragged tokens, odd weight-tile count, two units per tile
    (4, 513, 136, 768),        # token tail of one row
    (8, 1024, 2048, 8192),     # long K: 32 units per tile
    (4, 2048, 3072, 3072),
    (8, 17, 200, 256),         # one unit per tile: nothing can be cut
]


@pytest.fixture(autouse=True)
def _restore_schedule():
    yield
    qg.set_schedule(0, -1)


@pytest.mark.parametrize("bt", [0, 128, 192, 256])
@pytest.mark.parametrize("qbits,M,N,K", SHAPES, ids=[f"q{c[0]}-{c[1]}x{c[2]}x{c[3]}" for c in SHAPES])
def test_streamk_forced_matches_the_oracle(qbits, M, N, K, bt):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=14)
    dA, dWq, dWs = util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws)
    qg.set_schedule(bt, 1)
    g = util.Guarded((M, N), torch.bfloat16)
    qg.qgemm_dense(qbits, dA, dWq, dWs, out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    if M * N * K <= 2 ** 31:
        util.assert_close(util.host_bf16_f64(g.t), orc.qgemm_dense(qbits, A, Wq, Ws), "stream-K")
    else:
        _sampled_on_device(qbits, A, Wq, Ws, g.t, per_tile=4, seed=bt + M)
    # the counters are back at zero: a second stream-K call (same scratch) and a data-parallel one agree with it
    again = qg.qgemm_dense(qbits, dA, dWq, dWs)
    qg.set_schedule(bt, 0)
    plain = qg.qgemm_dense(qbits, dA, dWq, dWs)
    qg.poll_status()
    ref_max = float(g.t.float().abs().max())
    assert float((again.float() - g.t.float()).abs().max()) <= 2e-2 * ref_max
    assert float((plain.float() - g.t.float()).abs().max()) <= 2e-2 * ref_max


def test_the_cost_model_follows_the_measured_best_tile():
    """The token tile the model picks for the shapes it was fitted on (the fastest measured one), and stream-K only
    where a forced run showed it at least level with the best data-parallel tile."""
    qg.set_schedule(0, -1)
    want = {(8, 2048, 2560, 2048): 192, (8, 2048, 2048, 2048): 256, (8, 1024, 2560, 2048): 192, (8, 2048, 6144, 4096): 256,
            (8, 2048, 4096, 14336): 256, (4, 2048, 5120, 3072): 192, (4, 2048, 3072, 3072): 192, (4, 2048, 3072, 8192): 192,
            (4, 1024, 3072, 8192): 192}
    for (qbits, M, N, K), bt in want.items():
        got_bt, sk = qg.plan_dense(qbits, M, N, K)
        assert got_bt == bt and not sk, (qbits, M, N, K, got_bt, sk)
    assert qg.plan_dense(8, 64, 2048, 2048)[0] == 128
