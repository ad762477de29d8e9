"""moe_route_static: routing for callers that cannot provide (or allocate) scratch memory.

A server that froze its allocator after start-up, or a plug-in that only receives raw pointers, cannot give
moe_route its workspace.  moe_route_static keeps the per-block histograms in a fixed 256 KiB array inside the
library instead.  It must produce exactly what moe_route produces, on repeated calls (the array is shared and keeps
the previous call's contents), and must refuse problems that do not fit the array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu

KEYS = ("topk_idx", "topk_w", "counts", "offsets", "row_pair", "pair_row", "Xperm")


def _same(a, b):
    for key in KEYS:
        assert torch.equal(a[key], b[key]), key


def test_static_scratch_route_matches_workspace_route_on_two_calls_in_a_row():
    # first a large skewed problem, then a smaller one with other shapes: stale histogram entries must not leak
    cases = [(2048, 128, 8, 256, True, 0), (333, 16, 3, 64, False, 7)]
    for M, E, k, H, skewed, seed in cases:
        logits = util.dev(synth.router_logits(M, E, seed=seed, hot_bias=synth.SKEW_HOT_BIAS if skewed else 0.0))
        X = util.dev_bf16(synth.activations(M, H, seed=seed + 1))
        got = qg.moe_route_static(logits, k, X=X)
        ref = qg.moe_route(logits, k, X=X)
        qg.poll_status()
        _same(got, ref)
        again = qg.moe_route_static(logits, k, X=X)      # second call in a row on the same shared array
        qg.poll_status()
        _same(again, ref)
    assert int(got["offsets"][-1]) == 333 * 3


def test_static_scratch_route_rejects_what_does_not_fit_and_handles_empty_input():
    too_big = torch.zeros((32 * 65 + 1, 1024), dtype=torch.float32, device="cuda")      # 66 blocks * 1024 > 65536
    with pytest.raises(qg.QGemmError) as e:
        qg.moe_route_static(too_big, 2)
    assert e.value.code == -8 and "65536" in str(e.value)
    fits = qg.moe_route_static(too_big[:32 * 64], 2)                                      # exactly at the limit
    ref = qg.moe_route(too_big[:32 * 64], 2)
    qg.poll_status()
    assert torch.equal(fits["row_pair"], ref["row_pair"]) and torch.equal(fits["offsets"], ref["offsets"])
    z = qg.moe_route_static(torch.empty((0, 16), dtype=torch.float32, device="cuda"), 2)
    assert z["offsets"].cpu().tolist() == [0] * 17


def test_static_scratch_route_matches_the_oracle_and_allocates_nothing():
    """Checked against the CPU oracle directly (not only against moe_route), through preallocated outputs so that
    the call under test is the only thing that runs; the device's free memory, as the driver reports it, must be the
    same before and after.  The first call on a device does the one-time set-up (address look-up, lazy loading of the
    kernels), so the measurement brackets a later call."""
    M, E, k, H = 1500, 64, 6, 128
    logits_h = synth.router_logits(M, E, seed=21, hot_bias=synth.SKEW_HOT_BIAS)
    X_h = synth.activations(M, H, seed=22)
    logits, X = util.dev(logits_h), util.dev_bf16(X_h)
    i32 = dict(dtype=torch.int32, device="cuda")
    out = dict(topk_idx=torch.empty((M, k), **i32), topk_w=torch.empty((M, k), dtype=torch.float32, device="cuda"),
               counts=torch.empty(E, **i32), offsets=torch.empty(E + 1, **i32), row_pair=torch.empty(M * k, **i32),
               pair_row=torch.empty(M * k, **i32), Xperm=torch.empty((M * k, H), dtype=torch.bfloat16, device="cuda"))
    qg.moe_route_static(logits, k, X=X, out=out)          # set-up call
    qg.poll_status()
    for t in out.values():
        t.zero_()
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    qg.moe_route_static(logits, k, X=X, out=out)
    qg.poll_status()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "device memory was allocated or freed inside moe_route_static"
    idx, w, _ = orc.route(logits_h, k)
    counts, offsets = orc.counts_offsets(idx, E)
    row_pair, pair_row = orc.permutation(idx, offsets)
    assert np.array_equal(out["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["counts"].cpu().numpy(), counts)
    assert np.array_equal(out["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(out["row_pair"].cpu().numpy(), row_pair)
    assert np.array_equal(out["pair_row"].cpu().numpy(), pair_row)
    assert np.max(np.abs(out["topk_w"].cpu().numpy().astype(np.float64) - w)) <= util.TOPK_W_ATOL
    assert np.array_equal(util.host_bf16_bits(out["Xperm"]), orc.permute(X_h, row_pair, k))
