"""The bounded device-side waits: a wait that can never be satisfied must end the launch with QG_ERR_TIMEOUT in the
status word, free tensor memory and leave the context usable.  The failure is made in the allowed form: the testing
hook shortens the poll limit and tells one producer to leave out one load, so that a barrier is never completed;
nothing traps, faults or waits without a limit."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu

QG_ERR_TIMEOUT = -7


@pytest.mark.parametrize("qbits,M,N,K,skip", [(8, 300, 512, 1024, 5), (4, 700, 1024, 512, 0), (8, 2048, 4096, 2048, 9)],
                         ids=["q8-two-accumulators", "q4-first-kblock", "q8-single-accumulator-multi-tile"])
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(qbits, M, N, K, skip):
    A, Wq, Ws = synth.dense_problem(qbits, M, N, K, seed=12)
    dA, dWq, dWs = util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws)
    good = qg.qgemm_dense(qbits, dA, dWq, dWs)
    assert qg.poll_status_code() == 0
    try:
        qg.test_inject(wait_limit_polls=2048, skip_kblock=skip)      # about 10 ms per wait
        out = qg.qgemm_dense(qbits, dA, dWq, dWs)                    # returns: the launch itself is fine
        assert qg.poll_status_code() == QG_ERR_TIMEOUT
        assert qg.poll_status_code() == 0                            # the status word was cleared by the poll
    finally:
        qg.test_inject(0, -1)
    # tensor memory was freed and the barriers of the next launch start clean: the next call is correct again.  (Two
    # runs need not agree bit for bit: the even and the odd k-blocks of a tile are issued by two warps and accumulate
    # in whichever order they reach the tensor cores, so the fp32 sums may differ in the last place.)
    again = qg.qgemm_dense(qbits, dA, dWq, dWs)
    assert qg.poll_status_code() == 0
    ref = orc.qgemm_dense(qbits, A, Wq, Ws)
    util.assert_close(util.host_bf16_f64(again), ref, "after a timeout")
    util.assert_close(util.host_bf16_f64(good), ref, "before the timeout")
    assert float((again.float() - good.float()).abs().max()) <= 2e-2 * float(np.abs(ref).max())


def test_the_hook_acts_on_one_launch_only():
    A, Wq, Ws = synth.dense_problem(8, 64, 256, 256, seed=13)
    dA, dWq, dWs = util.dev_bf16(A), util.dev(Wq), util.dev_f16(Ws)
    try:
        qg.test_inject(wait_limit_polls=2048, skip_kblock=1)
        qg.qgemm_dense(8, dA, dWq, dWs)
        assert qg.poll_status_code() == QG_ERR_TIMEOUT
        out = qg.qgemm_dense(8, dA, dWq, dWs)                        # same short limit, nothing left out
        assert qg.poll_status_code() == 0
    finally:
        qg.test_inject(0, -1)
    util.assert_close(util.host_bf16_f64(out), orc.qgemm_dense(8, A, Wq, Ws), "launch after the injected one")
