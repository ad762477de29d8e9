"""GPU parity of prefill_attention against the fp64 oracle (plain softmax(scale Q K^T) V): causal and full, grouped-
query heads, ragged sequence lengths, inputs as strided column blocks of one fused-QKV buffer."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_19438_b200 import binding as qg, synth
from tests import util

pytestmark = pytest.mark.gpu


def _qkv(S, Hq, Hkv, d, seed, q_gain=1.0):
    """One [S, (Hq + 2 Hkv) d] bf16 buffer of N(0,1) values (queries optionally scaled to sharpen the softmax)."""
    W = (Hq + 2 * Hkv) * d
    x = synth.bf16_bits_to_f32(synth.activations(S, W, seed, 61))
    x[:, :Hq * d] *= q_gain
    return synth.f32_to_bf16_bits(x)


def _views(bits, Hq, Hkv, d):
    return bits[:, :Hq * d], bits[:, Hq * d:(Hq + Hkv) * d], bits[:, (Hq + Hkv) * d:]


CASES = [
    ("one-tile", 128, 2, 1, 128, True), ("two-tiles", 256, 2, 2, 128, True), ("ragged", 300, 4, 2, 128, True),
    ("tiny", 5, 2, 1, 128, True), ("single-token", 1, 1, 1, 128, True), ("full", 333, 2, 1, 128, False),
    ("d64", 200, 4, 2, 64, True), ("d64-full", 129, 2, 2, 64, False), ("gqa-3to1", 513, 6, 2, 128, True),
    ("sharp", 384, 2, 1, 128, True),
]


@pytest.mark.parametrize("name,S,Hq,Hkv,d,causal", CASES, ids=[c[0] for c in CASES])
def test_attention_parity(name, S, Hq, Hkv, d, causal):
    bits = _qkv(S, Hq, Hkv, d, seed=S + d, q_gain=4.0 if name == "sharp" else 1.0)
    Qh, Kh, Vh = _views(bits, Hq, Hkv, d)
    dev = util.dev_bf16(bits)
    Q, K, V = _views(dev, Hq, Hkv, d)
    g = util.Guarded((S, Hq * d), torch.bfloat16)
    qg.prefill_attention(Q, K, V, Hq, Hkv, d, causal=causal, out=g.t)
    qg.poll_status()
    assert g.intact() and not bool(g.untouched_inside().any().item())
    ref = orc.attention(Qh, Kh, Vh, Hq, Hkv, d, causal=causal)
    util.assert_close(util.host_bf16_f64(g.t), ref, f"attention {name}")


def test_attention_first_row_and_uniform_rows_are_exact_enough():
    """Row 0 of a causal problem is V[0] bit for bit (one key, weight 1); zero queries give the running mean of V."""
    S, Hq, Hkv, d = 260, 2, 1, 128
    bits = _qkv(S, Hq, Hkv, d, seed=3)
    bits[:, :Hq * d] = 0                                   # all queries zero
    Qh, Kh, Vh = _views(bits, Hq, Hkv, d)
    dev = util.dev_bf16(bits)
    Q, K, V = _views(dev, Hq, Hkv, d)
    out = qg.prefill_attention(Q, K, V, Hq, Hkv, d, causal=True)
    qg.poll_status()
    got = util.host_bf16_bits(out)
    assert np.array_equal(got[0, :d], Vh[0]) and np.array_equal(got[0, d:], Vh[0])
    Vf = orc.bf16_to_f64(np.ascontiguousarray(Vh))
    mean = np.cumsum(Vf, axis=0) / np.arange(1, S + 1)[:, None]
    util.assert_close(util.host_bf16_f64(out)[:, :d], mean, "running mean")


@pytest.mark.parametrize("S,Hq,Hkv,d", [(2048, 24, 8, 128), (4096, 32, 8, 128)], ids=["cfg2-heads-2048", "cfg4-heads-4096"])
def test_attention_full_size_sampled_rows(S, Hq, Hkv, d):
    """The head shapes of configs 2 and 4 at prompt lengths of the sweep; the oracle checks a sample of query rows
    (first, last, tile edges and random ones), all heads."""
    bits = _qkv(S, Hq, Hkv, d, seed=S)
    Qh, Kh, Vh = _views(bits, Hq, Hkv, d)
    dev = util.dev_bf16(bits)
    Q, K, V = _views(dev, Hq, Hkv, d)
    out = qg.prefill_attention(Q, K, V, Hq, Hkv, d, causal=True)
    qg.poll_status()
    assert bool(torch.isfinite(out.float()).all().item())
    rng = np.random.default_rng(S)
    qpos = np.unique(np.concatenate([[0, 1, 127, 128, 129, S // 2 - 1, S // 2, S - 129, S - 128, S - 1], rng.integers(0, S, 14)]))
    ref = orc.attention(Qh, Kh, Vh, Hq, Hkv, d, causal=True, qpos=qpos)
    got = util.host_bf16_f64(out[torch.from_numpy(qpos).cuda()])
    util.assert_close(got, ref, "attention full size")


def test_attention_argument_checks():
    x = torch.zeros((16, 3 * 128), dtype=torch.bfloat16, device="cuda")
    Q, K, V = x[:, :128], x[:, 128:256], x[:, 256:]
    with pytest.raises(qg.QGemmError) as e:
        qg.prefill_attention(Q, K, V, 1, 1, 96)
    assert e.value.code == -2
    with pytest.raises(qg.QGemmError) as e:
        qg.prefill_attention(Q, K, V, 3, 2, 128)
    assert e.value.code == -2
    assert qg.prefill_attention(Q[:0], K[:0], V[:0], 1, 1, 128).shape == (0, 128)
