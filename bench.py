#!/usr/bin/env python
"""Benchmark of the quantised prefill GEMM path on B200: one JSON line on stdout.

A step is one pass of the whole hot path over one batch of synthetic input at M = 2048 tokens:
  * the 2B-class dense Q8 layer set (QKV 2048->2560, O 2048->2048, gate/up 2048->16384, down 8192->2048):
    four qgemm_dense calls;
  * the 30B-A3B-shaped MoE Q4 layer (H=2048, E=128, top-8, F=768): moe_route (+ row gather),
    moe_grouped_qgemm gate/up+SiLU, moe_grouped_qgemm down with routing weights, moe_combine.
`value` is algorithmic TFLOP/s (2*M*N*K per dense GEMM, 2*R*3*F*H for the MoE layer, R = M*k) over the
device-timed region of K steps with inputs resident in HBM (one event pair around the whole region); a second
timed region of up to 100 steps with an event pair around every call gives the per-kernel figures and `roofline`;
`e2e` repeats the step through the same C-ABI calls with the activations and logits in pinned host memory (copied
in every step) and every output copied back, consecutive steps overlapped on three streams.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

--impl reference times the CPU oracle (fp64, naive) on a bounded sample of the same workload.
Under torchrun every rank runs its own replica of the step (the path shards by tokens with no exchange).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "Q4/Q8 prefill GEMM TFLOP/s & tok/s (dense+MoE), % of B200 bf16 tensor peak"
M_TOKENS = 2048
DENSE_SET = [("qkv", 2560, 2048), ("o", 2048, 2048), ("gate_up", 16384, 2048), ("down", 2048, 8192)]  # (name, N, K)
MOE = dict(H=2048, E=128, k=8, F=768)
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "qgemm_kernel_bench_step_traffic.json")


def ncu_traffic():
    """DRAM bytes (read + written) per launch of the GEMM kernel, quoted from the ncu capture of this step that the
    tracked data file records (with the commit it was taken at); None if the file is missing."""
    try:
        d = json.load(open(TRAFFIC_FILE))
        return float(d["dram_bytes_per_launch"]), d.get("captured_at_commit"), d.get("source")
    except Exception:
        return None, None, None


def dense_flops(M):
    return sum(2.0 * M * N * K for _, N, K in DENSE_SET)


def moe_flops(M):
    return 2.0 * M * MOE["k"] * 3 * MOE["F"] * MOE["H"]


def sustained_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path)).get("bf16_tflops_sustained", 1400.0))
    return 1400.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["bf16_tflops"]), float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json, cuBLAS bf16 burst)"
    return 1590.0, 6650.0, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------------------------------ synthetic inputs
def host_inputs(M, seed):
    from paper_2607_19438_b200 import synth
    dense = []
    for i, (name, N, K) in enumerate(DENSE_SET):
        A, Wq, Ws = synth.dense_problem(8, M, N, K, seed=seed, tid_base=16 * (i + 1))
        dense.append((name, A, Wq, Ws))
    moe = synth.moe_problem(4, M, MOE["H"], MOE["E"], MOE["F"], seed=seed)
    return dense, moe


# ------------------------------------------------------------------------------------------ CPU oracle arm
def oracle_sample_step(dense, moe, m_dense, m_moe):
    """Runs the oracle on the first m_dense rows of every dense GEMM and the first m_moe tokens of the MoE layer."""
    from oracle import oracle as orc
    for _, A, Wq, Ws in dense:
        orc.qgemm_dense(8, A[:m_dense], Wq, Ws)
    logits, X, W1q, W1s, W2q, W2s = moe
    orc.moe_layer(4, logits[:m_moe], X[:m_moe], W1q, W1s, W2q, W2s, MOE["k"])
    return dense_flops(m_dense) + moe_flops(m_moe)


def cpu_baseline(dense, moe, m_dense=128, m_moe=64):
    from oracle import oracle as orc
    t = time.perf_counter()
    fl = oracle_sample_step(dense, moe, m_dense, m_moe)
    dt = time.perf_counter() - t
    return {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"first {m_dense} of {M_TOKENS} rows of the 4 dense Q8 GEMMs + first {m_moe} tokens of the MoE Q4 "
                      f"layer, fp64 naive, {dt:.1f} s",
            "tok_per_s": 1.0 / (dense_flops(1) + moe_flops(1)) * fl / dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    dense, moe = host_inputs(M_TOKENS, seed=0)
    # calibrate on a tiny sample, then size a step so that the whole run stays within a few minutes
    # (the oracle parallelises over rows, so the sample has at least as many rows as threads)
    nthr = orc.num_threads()
    t = time.perf_counter(); fl = oracle_sample_step(dense, moe, nthr, nthr); rate = fl / (time.perf_counter() - t)
    budget = min(6.0, 150.0 / max(1, args.steps + args.warmup))
    per_tok = dense_flops(1) + moe_flops(1)
    m = int(max(nthr, min(128, rate * budget / per_tok)))
    for _ in range(args.warmup):
        oracle_sample_step(dense, moe, m, m)
    t0 = time.perf_counter()
    total = 0.0
    for _ in range(args.steps):
        total += oracle_sample_step(dense, moe, m, m)
    dt = time.perf_counter() - t0
    val = total / dt / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"cfg1 dense Q8 layer set + cfg3 MoE Q4 layer, M={M_TOKENS} (oracle on a sample)"},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "kind": "oracle", "cores": orc.num_threads(),
                             "sample": f"each step: first {m} rows of the 4 dense GEMMs + first {m} tokens of the MoE layer"},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ clocks
def clocks_in_window(samples, t0, t1):
    """Median SM clock and the throttle reasons seen between two host times (None if no sample fell inside)."""
    inside = [(mhz, act) for ts, mhz, act in samples if t0 <= ts <= t1]
    if not inside:
        return None
    return {"sm_mhz": float(np.median([m for m, _ in inside])), "samples": len(inside),
            "reasons": sorted({r for _, act in inside for r in act})}


class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,timestamp")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill(); out = ""
        import datetime
        sm, mx, pw, reasons = [], [], [], set()
        self.samples = []          # (epoch seconds, SM MHz, reasons active) for per-window summaries
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            act = [nm for nm, v in zip(names, f[3:7]) if v.lower().startswith("active")]
            reasons.update(act)
            if len(f) >= 8:
                try:
                    ts = datetime.datetime.strptime(f[7], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    self.samples.append((ts, float(f[0]), act))
                except ValueError:
                    pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(pw)),
                "samples": len(sm), "reasons": sorted(reasons)}



# ------------------------------------------------------------------------------------------ config sweep
LAYER_SETS = {   # (label, N, K) of the four projections of one transformer layer
    "cfg1_q8": (8, [("qkv", 2560, 2048), ("o", 2048, 2048), ("gate_up", 16384, 2048), ("down", 2048, 8192)]),
    "cfg2_q4": (4, [("qkv", 5120, 3072), ("o", 3072, 3072), ("gate_up", 16384, 3072), ("down", 3072, 8192)]),
    "cfg4_q8": (8, [("qkv", 6144, 4096), ("o", 4096, 4096), ("gate_up", 28672, 4096), ("down", 4096, 14336)]),
}
# the M sweep of the layer sets; below M = 1024 the weight stream (HBM) rather than the tensor pipe bounds a GEMM, the
# rows are there for the shape of the curve
SWEEP_DENSE = [("cfg1_q8", 128), ("cfg1_q8", 256), ("cfg1_q8", 512), ("cfg1_q8", 1024), ("cfg1_q8", 2048),
               ("cfg2_q4", 128), ("cfg2_q4", 256), ("cfg2_q4", 512), ("cfg2_q4", 1024), ("cfg2_q4", 2048),
               ("cfg4_q8", 2048), ("cfg4_q8", 4096), ("cfg4_q8", 8192)]
SWEEP_MOE = [(1024, False), (2048, False), (2048, True), (8192, False), (8192, True)]
L2_BYTES = 126e6


def run_sweep(torch, qg, lib, ctx, dev, stream, peak_tf, peak_hbm, iters=20):
    """Every configuration of the config list beside the headline one, each call timed with its own CUDA-event pair on
    the launching stream.  Inputs are seeded and drawn on the device (torch generator, seed 0) with the value
    distributions of the host generator: int8 uniform -127..127 / nibbles uniform 0..15, fp16 scales |N(0,0.02)|/qmax,
    bf16 N(0,1) activations, fp32 N(0,1) logits (+0.80 on every fourth expert when skewed).  Dense weights rotate
    through enough copies that the working set exceeds twice the L2; the MoE layer streams 340 MB per pass."""
    import ctypes as C
    P = lambda t: C.c_void_p(t.data_ptr())
    S = C.c_void_p(stream.cuda_stream)
    g = torch.Generator(device=dev); g.manual_seed(0)

    def chk(rc, what):
        if rc != 0:
            raise qg.QGemmError(rc, what)

    def weights(qbits, N, K):
        if qbits == 8:
            q = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev, generator=g)
        else:
            q = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device=dev, generator=g)
        sc = (torch.randn((N, K // 32), device=dev, generator=g).abs() * (0.02 / (127 if qbits == 8 else 7))).to(torch.float16)
        return q, sc

    def timed_calls(calls, n_iter):
        """calls: list of (label, flops, bytes, fn(it)).  Times (a) every call in a loop of its own, n_iter repetitions
        back to back between one pair of events (rotating through the weight copies via `it`), and (b) the whole
        sequence of calls, n_iter passes between one pair of events.  Returns {label: [total_ms, flops, bytes]} plus
        {"_all": [total_ms, 0, 0]}.  No event is recorded between two launches, so consecutive kernels overlap their
        start-up and tail as they do in a model's forward pass."""
        # burst regime, like the headline region: a pause lets the board's power average settle, then at least 15 ms
        # of warm-up passes bring the SM clock back up before the short timed regions
        torch.cuda.synchronize()
        time.sleep(0.3)
        t_w = time.perf_counter()
        it = 0
        while it < 3 or time.perf_counter() - t_w < 0.015:
            for _, _, _, fn in calls:
                fn(it)
            it += 1
            if it % 8 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        windows.append([time.time(), None])
        regions = []
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for it in range(n_iter):
            for _, _, _, fn in calls:
                fn(it)
        e1.record(stream)
        regions.append(("_all", 0.0, 0.0, e0, e1))
        if len(calls) > 1:
            for lab, fl, nb, fn in calls:
                torch.cuda.synchronize()
                time.sleep(0.05)                      # keep every region a short burst
                for it in range(2):
                    fn(it)
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for it in range(n_iter):
                    fn(it)
                e1.record(stream)
                regions.append((lab, fl, nb, e0, e1))
        else:
            lab, fl, nb, fn = calls[0]
            regions.append((lab, fl, nb, e0, e1))
        torch.cuda.synchronize()
        windows[-1][1] = time.time()
        return {lab: [e0.elapsed_time(e1), fl, nb] for lab, fl, nb, e0, e1 in regions}

    windows = []
    out = {"method": "one CUDA-event pair per call on the launching stream, at least 60 ms of warm-up passes then %d timed passes per configuration, "
                     "dense weights rotated through copies exceeding 2x L2, inputs drawn on the device (seed 0)" % iters,
           "peak_tflops": peak_tf, "dense": [], "moe": []}
    for name, M in SWEEP_DENSE:
        qbits, layers = LAYER_SETS[name]
        wbytes = sum(N * K * (1.0625 if qbits == 8 else 0.5625) for _, N, K in layers)
        ncopy = max(2, int(2 * L2_BYTES // wbytes) + 1)
        W = [[weights(qbits, N, K) for _, N, K in layers] for _ in range(ncopy)]
        A = {K: torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16) for K in {K for _, _, K in layers}}
        Cs = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _, N, _ in layers]
        calls = []
        for i, (lab, N, K) in enumerate(layers):
            def fn(it, i=i, N=N, K=K):
                q, sc = W[it % ncopy][i]
                chk(lib.qgemm_dense(ctx, qbits, M, N, K, P(A[K]), P(q), P(sc), P(Cs[i]), S), "qgemm_dense")
            calls.append((lab, 2.0 * M * N * K, 0.0, fn))
        n_it = iters if M * sum(N * K for _, N, K in layers) < 2e12 else max(5, iters // 2)
        agg = timed_calls(calls, n_it)
        tot_ms = agg.pop("_all")[0]; tot_fl = sum(v[1] for v in agg.values()) * n_it
        row = {"set": name, "M": M, "weight_copies": ncopy,
               "gemm_tflops": {lab: v[1] * n_it / (v[0] * 1e-3) / 1e12 for lab, v in agg.items()},
               "gemm_us": {lab: v[0] / n_it * 1e3 for lab, v in agg.items()},
               "set_tflops": tot_fl / (tot_ms * 1e-3) / 1e12, "tok_per_s": M * n_it / (tot_ms * 1e-3)}
        row["frac_of_measured_peak"] = row["set_tflops"] / peak_tf
        out["dense"].append(row)
        del W, A, Cs
        torch.cuda.empty_cache()

    # small batches (decode side): weight streaming, against the measured HBM copy bandwidth
    out["small_m"] = []
    for name in ("cfg1_q8", "cfg2_q4", "cfg4_q8"):
        qbits, layers = LAYER_SETS[name]
        wbytes = sum(N * K * (1.0625 if qbits == 8 else 0.5625) for _, N, K in layers)
        ncopy = max(2, int(2 * L2_BYTES // wbytes) + 1)
        W = [[weights(qbits, N, K) for _, N, K in layers] for _ in range(ncopy)]
        for M in (1, 4, 16):
            A = {K: torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16) for K in {K for _, _, K in layers}}
            Cs = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _, N, _ in layers]
            for api, label in ((lib.qgemm_small_m, "qgemm_small_m"), (lib.qgemm_dense, "qgemm_dense")):
                calls = []
                for i, (lab, N, K) in enumerate(layers):
                    def fn(it, i=i, N=N, K=K, api=api):
                        q, sc = W[it % ncopy][i]
                        chk(api(ctx, qbits, M, N, K, P(A[K]), P(q), P(sc), P(Cs[i]), S), label)
                    calls.append((lab, 2.0 * M * N * K, N * K * (1.0625 if qbits == 8 else 0.5625) + 2.0 * M * (N + K), fn))
                agg = timed_calls(calls, iters)
                tot_ms = agg.pop("_all")[0]; tot_b = sum(v[2] for v in agg.values()) * iters
                out["small_m"].append({"set": name, "M": M, "call": label,
                                       "gemm_us": {lab: v[0] / iters * 1e3 for lab, v in agg.items()},
                                       "gemm_gbs": {lab: v[2] * iters / (v[0] * 1e-3) / 1e9 for lab, v in agg.items()},
                                       "set_gbs": tot_b / (tot_ms * 1e-3) / 1e9,
                                       "frac_of_measured_hbm": tot_b / (tot_ms * 1e-3) / 1e9 / peak_hbm,
                                       "tok_per_s": M * iters / (tot_ms * 1e-3)})
        del W
        torch.cuda.empty_cache()

    # block-scaled FP8 path: weights re-encoded once (not timed), activations re-encoded inside the timed sequence (the
    # hidden state once for QKV and gate/up, the attention output for O, the FFN intermediate for down)
    out["mx_fp8"] = []
    peak_fp8 = 2.0 * peak_tf
    for name, M in (("cfg1_q8", 2048), ("cfg2_q4", 2048), ("cfg4_q8", 2048), ("cfg4_q8", 8192)):
        qbits, layers = LAYER_SETS[name]
        Wmx = []
        for _, N, K in layers:
            q, sc = weights(qbits, N, K)
            wc = torch.empty((N, K), dtype=torch.uint8, device=dev)
            wsf = torch.empty(int(lib.qg_mx_scale_bytes(N, K)), dtype=torch.uint8, device=dev)
            chk(lib.qg_mx_pack_weights(ctx, qbits, N, K, P(q), P(sc), P(wc), P(wsf), S), "qg_mx_pack_weights")
            Wmx.append((wc, wsf))
            del q, sc
        Ks = sorted({K for _, _, K in layers})
        X = {K: torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16) for K in Ks}
        Xattn = torch.randn((M, Ks[0]), device=dev, generator=g).to(torch.bfloat16)
        enc = {key: (torch.empty((M, K), dtype=torch.uint8, device=dev),
                     torch.empty(int(lib.qg_mx_scale_bytes(M, K)), dtype=torch.uint8, device=dev))
               for key, K in (("hidden", Ks[0]), ("attn", Ks[0]), ("inter", Ks[1]))}
        Cs = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _, N, _ in layers]

        def quant(key, src, K):
            return lambda it: chk(lib.qg_mx_quantize(ctx, M, K, P(src), P(enc[key][0]), P(enc[key][1]), S), "qg_mx_quantize")

        def gemm(i, key):
            _, N, K = layers[i]
            return lambda it: chk(lib.qgemm_mx_dense(ctx, M, N, K, P(enc[key][0]), P(enc[key][1]), P(Wmx[i][0]), P(Wmx[i][1]),
                                                     P(Cs[i]), S), "qgemm_mx_dense")
        fl = [2.0 * M * N * K for _, N, K in layers]
        calls = [("quantize_hidden", 0.0, 3.0 * M * Ks[0], quant("hidden", X[Ks[0]], Ks[0])), ("qkv", fl[0], 0.0, gemm(0, "hidden")),
                 ("quantize_attn", 0.0, 3.0 * M * Ks[0], quant("attn", Xattn, Ks[0])), ("o", fl[1], 0.0, gemm(1, "attn")),
                 ("gate_up", fl[2], 0.0, gemm(2, "hidden")),
                 ("quantize_inter", 0.0, 3.0 * M * Ks[1], quant("inter", X[Ks[1]], Ks[1])), ("down", fl[3], 0.0, gemm(3, "inter"))]
        n_it = iters if M <= 2048 else max(5, iters // 2)
        agg = timed_calls(calls, n_it)
        tot_ms = agg.pop("_all")[0]
        row = {"set": name + " re-encoded to block-scaled FP8 (E4M3, power-of-two scale per 32)", "M": M,
               "gemm_tflops": {lab: v[1] * n_it / (v[0] * 1e-3) / 1e12 for lab, v in agg.items() if v[1]},
               "call_us": {lab: v[0] / n_it * 1e3 for lab, v in agg.items()},
               "set_tflops_incl_quantize": sum(fl) * n_it / (tot_ms * 1e-3) / 1e12, "tok_per_s": M * n_it / (tot_ms * 1e-3),
               "peak_tflops": peak_fp8, "peak_source": "2 x the measured bf16 burst peak (nominal fp8 : bf16 ratio)"}
        row["frac_of_fp8_peak"] = row["set_tflops_incl_quantize"] / peak_fp8
        out["mx_fp8"].append(row)
        del Wmx, X, Xattn, enc, Cs
        torch.cuda.empty_cache()

    # prefill attention (causal, grouped-query heads), reading Q, K, V as column blocks of one fused-QKV buffer
    out["attention"] = []
    for name, Hq, Hkv, d, Sq in (("cfg2 heads", 24, 8, 128, 2048), ("cfg4 heads", 32, 8, 128, 2048), ("cfg4 heads", 32, 8, 128, 8192)):
        qkv = torch.randn((Sq, (Hq + 2 * Hkv) * d), device=dev, generator=g).to(torch.bfloat16)
        Q, K, V = qkv[:, :Hq * d], qkv[:, Hq * d:(Hq + Hkv) * d], qkv[:, (Hq + Hkv) * d:]
        O = torch.empty((Sq, Hq * d), dtype=torch.bfloat16, device=dev)
        fl = 4.0 * Sq * Sq * Hq * d / 2 + 2.0 * Sq * 128 * Hq * d     # causal: the lower triangle in 128-wide tiles incl. the diagonal
        calls = [("attention", fl, 0.0, lambda it: chk(lib.prefill_attention(
            ctx, Sq, Hq, Hkv, d, P(Q), qkv.stride(0), P(K), qkv.stride(0), P(V), qkv.stride(0), P(O), O.stride(0), 1,
            C.c_float(0.0), S), "prefill_attention"))]
        n_it = iters if Sq <= 2048 else max(5, iters // 2)
        agg = timed_calls(calls, n_it)
        ms = agg["attention"][0] / n_it
        out["attention"].append({"shape": name, "S": Sq, "Hq": Hq, "Hkv": Hkv, "d": d, "causal": True, "us": ms * 1e3,
                                 "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_measured_peak": fl / (ms * 1e-3) / 1e12 / peak_tf,
                                 "flops": "4 S^2 Hq d / 2 plus the diagonal tiles' upper halves that are computed and masked",
                                 "tok_per_s": Sq / (ms * 1e-3)})

    H, E, k, F = MOE["H"], MOE["E"], MOE["k"], MOE["F"]
    W1q, W1s = weights(4, E * 2 * F, H); W2q, W2s = weights(4, E * H, F)
    i32 = dict(dtype=torch.int32, device=dev)
    # the expert weights re-encoded once to block-scaled FP8 (twice the bytes of the 4-bit codes)
    Wmx = []
    for q, sc, rows, K in ((W1q, W1s, E * 2 * F, H), (W2q, W2s, E * H, F)):
        wc = torch.empty((rows, K), dtype=torch.uint8, device=dev)
        wsf = torch.empty(int(lib.qg_mx_scale_bytes(rows, K)), dtype=torch.uint8, device=dev)
        chk(lib.qg_mx_pack_weights(ctx, 4, rows, K, P(q), P(sc), P(wc), P(wsf), S), "qg_mx_pack_weights")
        Wmx.append((wc, wsf))
    for M, skewed in SWEEP_MOE:
        R = M * k
        L = torch.randn((M, E), device=dev, generator=g)
        if skewed:
            L[:, ::4] += 0.80
        X = torch.randn((M, H), device=dev, generator=g).to(torch.bfloat16)
        ws = torch.empty(max(16, qg.route_workspace_bytes(M, E, k)), dtype=torch.uint8, device=dev)
        o = dict(idx=torch.empty((M, k), **i32), w=torch.empty((M, k), dtype=torch.float32, device=dev),
                 counts=torch.empty(E, **i32), offsets=torch.empty(E + 1, **i32), row_pair=torch.empty(R, **i32),
                 pair_row=torch.empty(R, **i32), Xp=torch.empty((R, H), dtype=torch.bfloat16, device=dev),
                 Hh=torch.empty((R, F), dtype=torch.bfloat16, device=dev),
                 Dw=torch.empty((R, H), dtype=torch.bfloat16, device=dev), y=torch.empty((M, H), dtype=torch.bfloat16, device=dev),
                 acc=torch.zeros((M, H), dtype=torch.float32, device=dev))

        def down_acc(it):
            o["acc"].zero_()
            chk(lib.moe_grouped_qgemm(ctx, qg.MODE_DOWN_ACCUM_F32, 4, R, E, H, F, P(o["Hh"]), P(o["offsets"]), P(W2q),
                                      P(W2s), P(o["w"]), P(o["row_pair"]), k, P(o["acc"]), S), "down acc")
        calls_fused = [
            ("route", 0.0, 4.0 * M * E + 16.0 * R, lambda it: chk(lib.moe_route(
                ctx, M, E, k, P(L), P(o["idx"]), P(o["w"]), P(o["counts"]), P(o["offsets"]), P(o["row_pair"]),
                P(o["pair_row"]), None, None, H, P(ws), ws.numel(), S), "moe_route")),
            ("gate_up", 2.0 * R * 2 * F * H, 0.0, lambda it: chk(lib.moe_grouped_qgemm_gather(
                ctx, qg.MODE_GATE_UP_SILU, 4, M, R, E, 2 * F, H, P(X), P(o["row_pair"]), k, P(o["offsets"]), P(W1q),
                P(W1s), None, P(o["Hh"]), S), "gate/up gather")),
            ("down", 2.0 * R * F * H, 0.0, down_acc),
            ("combine", 0.0, 6.0 * M * H, lambda it: chk(lib.moe_combine(
                ctx, M, k, H, P(o["acc"]), qg.D_F32_ACC, None, None, P(o["y"]), S), "round")),
        ]
        calls = [
            ("route_permute", 0.0, 4.0 * M * E + 16.0 * R + 2.0 * M * H + 2.0 * R * H, lambda it: chk(lib.moe_route(
                ctx, M, E, k, P(L), P(o["idx"]), P(o["w"]), P(o["counts"]), P(o["offsets"]), P(o["row_pair"]),
                P(o["pair_row"]), P(X), P(o["Xp"]), H, P(ws), ws.numel(), S), "moe_route")),
            ("gate_up", 2.0 * R * 2 * F * H, 0.0, lambda it: chk(lib.moe_grouped_qgemm(
                ctx, qg.MODE_GATE_UP_SILU, 4, R, E, 2 * F, H, P(o["Xp"]), P(o["offsets"]), P(W1q), P(W1s), None, None, k,
                P(o["Hh"]), S), "gate/up")),
            ("down", 2.0 * R * F * H, 0.0, lambda it: chk(lib.moe_grouped_qgemm(
                ctx, qg.MODE_DOWN_WEIGHTED, 4, R, E, H, F, P(o["Hh"]), P(o["offsets"]), P(W2q), P(W2s), P(o["w"]),
                P(o["row_pair"]), k, P(o["Dw"]), S), "down")),
            ("combine", 0.0, 2.0 * R * H + 2.0 * M * H, lambda it: chk(lib.moe_combine(
                ctx, M, k, H, P(o["Dw"]), qg.D_BF16, P(o["pair_row"]), None, P(o["y"]), S), "combine")),
        ]
        n_it = iters if M <= 2048 else max(5, iters // 2)
        agg = timed_calls(calls, n_it)
        tot_ms = agg.pop("_all")[0]
        gemm_ms = agg["gate_up"][0] + agg["down"][0]
        gemm_fl = (agg["gate_up"][1] + agg["down"][1]) * n_it
        # composite bound of the two grouped GEMMs: the tensor time at the measured peak or the time to stream the
        # 340 MB of expert weights once from HBM, whichever is longer
        t_tensor = gemm_fl / n_it / (peak_tf * 1e12)
        t_hbm = (E * 3 * F * H * 0.5625) / (peak_hbm * 1e9)
        row = {"M": M, "routing": "skewed" if skewed else "uniform", "rows_per_expert": R / E,
               "gemm_tflops": {lab: agg[lab][1] * n_it / (agg[lab][0] * 1e-3) / 1e12 for lab in ("gate_up", "down")},
               "call_us": {lab: v[0] / n_it * 1e3 for lab, v in agg.items()},
               "gemms_tflops": gemm_fl / (gemm_ms * 1e-3) / 1e12, "layer_tok_per_s": M * n_it / (tot_ms * 1e-3),
               "hbm_gbs": {lab: agg[lab][2] * n_it / (agg[lab][0] * 1e-3) / 1e9 for lab in ("route_permute", "combine")},
               "hbm_gbs_note": "algorithmic bytes over the time of the call repeated back to back; up to M = 2048 the rows it "
                               "reads (64 MB) stay in the 126 MB L2 between repetitions, so the figure can exceed the HBM "
                               "peak; inside a layer pass the same calls take the times of the headline's `kernels` block",
               "composite_bound_us": max(t_tensor, t_hbm) * 1e6,
               "bound": "hbm (expert weights)" if t_hbm > t_tensor else "tensor"}
        row["frac_of_measured_peak"] = row["gemms_tflops"] / peak_tf
        row["frac_of_composite_bound"] = max(t_tensor, t_hbm) / (gemm_ms / n_it * 1e-3)
        windows.pop()                       # one clock window per row: the one of the fused pass below
        aggf = timed_calls(calls_fused, n_it)
        tot_ms_f = aggf.pop("_all")[0]
        gemm_ms_f = aggf["gate_up"][0] + aggf["down"][0]
        row["fused"] = {"what": "route without row gather, gate/up with gathered loads, down with fp32 accumulate "
                                "(its time includes the accumulator's zero fill), rounding",
                        "call_us": {lab: v[0] / n_it * 1e3 for lab, v in aggf.items()},
                        "gemms_tflops": gemm_fl / (gemm_ms_f * 1e-3) / 1e12,
                        "layer_tok_per_s": M * n_it / (tot_ms_f * 1e-3)}
        if not skewed:
            # the two pieces around the routed experts: router projection (hidden -> experts, bf16) and the combine that
            # adds a shared expert's row; each repeated back to back (a few microseconds each: launch-bound figures)
            Wr = (torch.randn((E, H), device=dev, generator=g) * 0.05).to(torch.bfloat16)
            shared = torch.randn((M, H), device=dev, generator=g).to(torch.bfloat16)
            windows.pop()
            ex = timed_calls([("router_logits", 2.0 * M * H * E, 2.0 * M * H + 2.0 * E * H + 4.0 * M * E,
                               lambda it: chk(lib.moe_router_logits(ctx, M, H, E, P(X), P(Wr), P(L), S), "router"))], n_it)
            windows.pop()
            ex2 = timed_calls([("combine_shared", 0.0, 2.0 * R * H + 4.0 * M * H, lambda it: chk(lib.moe_combine_shared(
                ctx, M, k, H, P(o["Dw"]), qg.D_BF16, P(o["pair_row"]), None, P(shared), P(o["y"]), S), "combine shared"))], n_it)
            row["router_and_shared_expert"] = {"router_logits_us": ex["router_logits"][0] / n_it * 1e3,
                                               "combine_shared_us": ex2["combine_shared"][0] / n_it * 1e3}
            # the two expert GEMMs on the block-scaled FP8 path (sorted rows re-encoded per call, per-segment scale tiles)
            xc = torch.empty((R, H), dtype=torch.uint8, device=dev)
            xs = torch.empty(int(lib.qg_mx_grouped_scale_bytes(R, E, H)), dtype=torch.uint8, device=dev)
            hc = torch.empty((R, F), dtype=torch.uint8, device=dev)
            hs = torch.empty(int(lib.qg_mx_grouped_scale_bytes(R, E, F)), dtype=torch.uint8, device=dev)
            mxc = [
                ("quantize_rows", 0.0, 3.0 * R * H, lambda it: chk(lib.qg_mx_quantize_grouped(
                    ctx, R, E, H, P(o["Xp"]), P(o["offsets"]), P(xc), P(xs), S), "quantize grouped")),
                ("gate_up", 2.0 * R * 2 * F * H, 0.0, lambda it: chk(lib.moe_grouped_qgemm_mx(
                    ctx, qg.MODE_GATE_UP_SILU, R, E, 2 * F, H, P(xc), P(xs), P(o["offsets"]), P(Wmx[0][0]), P(Wmx[0][1]), None,
                    None, P(o["Hh"]), S), "gate/up mx")),
                ("quantize_hidden", 0.0, 3.0 * R * F, lambda it: chk(lib.qg_mx_quantize_grouped(
                    ctx, R, E, F, P(o["Hh"]), P(o["offsets"]), P(hc), P(hs), S), "quantize grouped")),
                ("down", 2.0 * R * F * H, 0.0, lambda it: chk(lib.moe_grouped_qgemm_mx(
                    ctx, qg.MODE_DOWN_WEIGHTED, R, E, H, F, P(hc), P(hs), P(o["offsets"]), P(Wmx[1][0]), P(Wmx[1][1]), P(o["w"]),
                    P(o["row_pair"]), P(o["Dw"]), S), "down mx")),
            ]
            windows.pop()
            am = timed_calls(mxc, n_it)
            am.pop("_all")
            row["block_scaled_fp8"] = {
                "call_us": {lab: v[0] / n_it * 1e3 for lab, v in am.items()},
                "gemms_tflops": gemm_fl / ((am["gate_up"][0] + am["down"][0]) * 1e-3) / 1e12,
                "note": "604 MB of FP8 expert weights against 340 MB of 4-bit codes and scales: bound by the weight bytes "
                        "(HBM up to 2048 tokens, L2 -> SM at 8192), so no faster than the 4-bit path here"}
            del xc, xs, hc, hs
        out["moe"].append(row)
    out["_windows"] = windows
    return out

# ------------------------------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_19438_b200 import binding as qg

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    M = M_TOKENS
    dense_h, moe_h = host_inputs(M, seed=rank)

    def bf16(a): return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    def f16(a): return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.float16)
    def raw(a): return torch.from_numpy(np.ascontiguousarray(a))

    # weights live in HBM (model state); activations and logits have a pinned host copy for the e2e leg
    dW = [(name, raw(Wq).to(dev), f16(Ws).to(dev)) for name, _, Wq, Ws in dense_h]
    hA = [bf16(A).pin_memory() for _, A, _, _ in dense_h]
    logits_h, X_h, W1q, W1s, W2q, W2s = moe_h
    hL, hX = raw(logits_h).pin_memory(), bf16(X_h).pin_memory()
    dW1q, dW1s, dW2q, dW2s = raw(W1q).to(dev), f16(W1s).to(dev), raw(W2q).to(dev), f16(W2s).to(dev)
    dA = [a.to(dev) for a in hA]
    dL, dX = hL.to(dev), hX.to(dev)
    k, E, H, F = MOE["k"], MOE["E"], MOE["H"], MOE["F"]
    R = M * k
    i32 = dict(dtype=torch.int32, device=dev)
    # all outputs and scratch preallocated: nothing is allocated inside a step
    oC = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _, N, _ in DENSE_SET]
    ws = torch.empty(max(16, qg.route_workspace_bytes(M, E, k)), dtype=torch.uint8, device=dev)
    o = dict(idx=torch.empty((M, k), **i32), w=torch.empty((M, k), dtype=torch.float32, device=dev),
             counts=torch.empty(E, **i32), offsets=torch.empty(E + 1, **i32), row_pair=torch.empty(R, **i32),
             pair_row=torch.empty(R, **i32), Xp=torch.empty((R, H), dtype=torch.bfloat16, device=dev),
             Hh=torch.empty((R, F), dtype=torch.bfloat16, device=dev),
             Dw=torch.empty((R, H), dtype=torch.bfloat16, device=dev), y=torch.empty((M, H), dtype=torch.bfloat16, device=dev),
             acc=torch.zeros((M, H), dtype=torch.float32, device=dev))
    fused = (args.moe_path == "fused")
    hC = [torch.empty((M, N), dtype=torch.bfloat16).pin_memory() for _, N, _ in DENSE_SET]
    hY = torch.empty((M, H), dtype=torch.bfloat16).pin_memory()

    lib, ctx = qg.load(), qg.context(local)
    import ctypes as C
    P = lambda t: C.c_void_p(t.data_ptr())
    stream = torch.cuda.current_stream()
    S = C.c_void_p(stream.cuda_stream)
    gemm_events = []   # (label, flops, start, end) recorded inside the timed region

    def chk(rc, what):
        if rc != 0:
            raise qg.QGemmError(rc, what)

    def step(A_list, L, X, record=False, outC=None, outY=None):
        outC = oC if outC is None else outC
        outY = o["y"] if outY is None else outY
        for i, (name, N, K) in enumerate(DENSE_SET):
            if record:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True); e0.record(stream)
            chk(lib.qgemm_dense(ctx, 8, M, N, K, P(A_list[i]), P(dW[i][1]), P(dW[i][2]), P(outC[i]), S), "qgemm_dense")
            if record:
                e1.record(stream); gemm_events.append(("dense_q8_" + name, 2.0 * M * N * K, e0, e1))
        def ev():
            e = torch.cuda.Event(enable_timing=True); e.record(stream); return e
        if fused:
            # routing tables only; the token rows are gathered by the gate/up kernel's loads, the routing-weighted
            # sum over a token's experts is accumulated in fp32 by the down kernel's epilogue and rounded once
            a = ev() if record else None
            chk(lib.moe_route(ctx, M, E, k, P(L), P(o["idx"]), P(o["w"]), P(o["counts"]), P(o["offsets"]), P(o["row_pair"]),
                              P(o["pair_row"]), None, None, H, P(ws), ws.numel(), S), "moe_route")
            b = ev() if record else None
            chk(lib.moe_grouped_qgemm_gather(ctx, qg.MODE_GATE_UP_SILU, 4, M, R, E, 2 * F, H, P(X), P(o["row_pair"]), k,
                                             P(o["offsets"]), P(dW1q), P(dW1s), None, P(o["Hh"]), S), "gate/up (gather)")
            c = ev() if record else None
            o["acc"].zero_()
            chk(lib.moe_grouped_qgemm(ctx, qg.MODE_DOWN_ACCUM_F32, 4, R, E, H, F, P(o["Hh"]), P(o["offsets"]), P(dW2q),
                                      P(dW2s), P(o["w"]), P(o["row_pair"]), k, P(o["acc"]), S), "down (accumulate)")
            d = ev() if record else None
            chk(lib.moe_combine(ctx, M, k, H, P(o["acc"]), qg.D_F32_ACC, None, None, P(outY), S), "moe_combine (round)")
            e = ev() if record else None
            if record:
                gemm_events.extend([("route", 0.0, a, b), ("moe_gate_up_q4", 2.0 * R * 2 * F * H, b, c),
                                    ("moe_down_q4", 2.0 * R * F * H, c, d), ("combine", 0.0, d, e)])
            return
        a = ev() if record else None
        chk(lib.moe_route(ctx, M, E, k, P(L), P(o["idx"]), P(o["w"]), P(o["counts"]), P(o["offsets"]), P(o["row_pair"]),
                          P(o["pair_row"]), P(X), P(o["Xp"]), H, P(ws), ws.numel(), S), "moe_route")
        b = ev() if record else None
        chk(lib.moe_grouped_qgemm(ctx, qg.MODE_GATE_UP_SILU, 4, R, E, 2 * F, H, P(o["Xp"]), P(o["offsets"]), P(dW1q),
                                  P(dW1s), None, None, k, P(o["Hh"]), S), "moe_grouped_qgemm gate/up")
        c = ev() if record else None
        chk(lib.moe_grouped_qgemm(ctx, qg.MODE_DOWN_WEIGHTED, 4, R, E, H, F, P(o["Hh"]), P(o["offsets"]), P(dW2q),
                                  P(dW2s), P(o["w"]), P(o["row_pair"]), k, P(o["Dw"]), S), "moe_grouped_qgemm down")
        d = ev() if record else None
        chk(lib.moe_combine(ctx, M, k, H, P(o["Dw"]), qg.D_BF16, P(o["pair_row"]), None, P(outY), S), "moe_combine")
        e = ev() if record else None
        if record:
            gemm_events.extend([("route", 0.0, a, b), ("moe_gate_up_q4", 2.0 * R * 2 * F * H, b, c),
                                ("moe_down_q4", 2.0 * R * F * H, c, d), ("combine", 0.0, d, e)])

    # dense x4, route (topk, scan, scatter), [permute,] grouped x2, combine or rounding (the fused path's zero fill of
    # the fp32 accumulator is a memset, not counted)
    LAUNCHES_PER_STEP = 4 + 3 + (0 if fused else 1) + 2 + 1

    def gemm_step():
        """The six GEMM launches of the step alone, on the buffers the full step left behind (routing tables, permuted
        rows, gate/up output): the timed region that gives the GEMM kernel's average launch duration without an event
        pair round every call."""
        for i, (name, N, K) in enumerate(DENSE_SET):
            chk(lib.qgemm_dense(ctx, 8, M, N, K, P(dA[i]), P(dW[i][1]), P(dW[i][2]), P(oC[i]), S), "qgemm_dense")
        if fused:
            chk(lib.moe_grouped_qgemm_gather(ctx, qg.MODE_GATE_UP_SILU, 4, M, R, E, 2 * F, H, P(dX), P(o["row_pair"]), k,
                                             P(o["offsets"]), P(dW1q), P(dW1s), None, P(o["Hh"]), S), "gate/up (gather)")
            chk(lib.moe_grouped_qgemm(ctx, qg.MODE_DOWN_ACCUM_F32, 4, R, E, H, F, P(o["Hh"]), P(o["offsets"]), P(dW2q),
                                      P(dW2s), P(o["w"]), P(o["row_pair"]), k, P(o["acc"]), S), "down (accumulate)")
        else:
            chk(lib.moe_grouped_qgemm(ctx, qg.MODE_GATE_UP_SILU, 4, R, E, 2 * F, H, P(o["Xp"]), P(o["offsets"]), P(dW1q),
                                      P(dW1s), None, None, k, P(o["Hh"]), S), "moe_grouped_qgemm gate/up")
            chk(lib.moe_grouped_qgemm(ctx, qg.MODE_DOWN_WEIGHTED, 4, R, E, H, F, P(o["Hh"]), P(o["offsets"]), P(dW2q),
                                      P(dW2s), P(o["w"]), P(o["row_pair"]), k, P(o["Dw"]), S), "moe_grouped_qgemm down")

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps):
        sync_all()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
            dist.barrier()
        return ms

    # ---- device-resident leg
    for _ in range(max(3, args.warmup)):
        step(dA, dL, dX)
    qg.poll_status()
    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.05)
    # Two timed regions of `steps` steps each.  The first is bracketed by one pair of events and gives `value`; the
    # second repeats it with an event pair around every call for the per-kernel figures and the roofline (sixteen
    # extra stream operations per step cost a few per cent, so they stay out of the headline).
    ms = timed(lambda: step(dA, dL, dX), args.steps)
    if args.profile_run:
        qg.poll_status()
        if rank == 0:
            print(json.dumps({"profile_run": True, "steps": args.steps, "ms_per_step": ms / args.steps,
                              "launches_per_step": LAUNCHES_PER_STEP, "moe_path": args.moe_path}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return
    ev_steps = max(1, min(args.steps, 100))
    torch.cuda.synchronize()
    time.sleep(1.0)     # let the board's power average settle: a sustained run is clocked down under the power cap
    for _ in range(3):
        step(dA, dL, dX)
    ms_events = timed(lambda: step(dA, dL, dX, record=True), ev_steps)
    for _ in range(3):
        gemm_step()
    ms_gemm = timed(gemm_step, ev_steps)          # GEMM launches only, one event pair round the whole region
    clocks = sampler.stop() if sampler else None
    qg.poll_status()
    flops_step = dense_flops(M) + moe_flops(M)
    # sustained: the same step back to back for at least two seconds, with its own clock record (the board's power
    # cap pulls the SM clock down after a few hundred milliseconds of this load)
    sus_steps = int(min(20000, max(200, 2200.0 / (ms / args.steps))))
    sampler2 = ClockSampler(local) if rank == 0 else None
    ms_sus = timed(lambda: step(dA, dL, dX), sus_steps)
    clocks_sus = sampler2.stop() if sampler2 else None
    qg.poll_status()
    time.sleep(1.0)
    value = world * flops_step * args.steps / (ms * 1e-3) / 1e12

    # per-kernel figures from the events recorded inside the timed region
    agg = {}
    for label, fl, a, b in gemm_events:
        d = agg.setdefault(label, [0.0, 0.0, 0])
        d[0] += fl; d[1] += a.elapsed_time(b); d[2] += 1
    detail = {lab: {"launches": v[2], "avg_us": v[1] / v[2] * 1e3, "tflops": (v[0] / (v[1] * 1e-3) / 1e12) if v[0] else None}
              for lab, v in agg.items()}
    peak_tf, peak_hbm, peak_src = measured_peaks()
    # the HBM-bound calls: algorithmic bytes (route: logits in, indices/weights/permutation out; permute: X in, permuted
    # rows out; combine: weighted rows in, y out) against the measured copy bandwidth
    if fused:   # route: logits in, tables out; "combine": zero fill and rounding of the fp32 accumulator
        hbm_bytes = {"route": 4.0 * M * E + 16.0 * R, "combine": 4.0 * M * H + 2.0 * M * H}
    else:
        hbm_bytes = {"route": 4.0 * M * E + 16.0 * R + 2.0 * M * H + 2.0 * R * H, "combine": 2.0 * R * H + 2.0 * M * H}
    for lab, nbytes in hbm_bytes.items():
        gbs = nbytes / (detail[lab]["avg_us"] * 1e-6) / 1e9
        detail[lab].update({"bound": "hbm", "algorithmic_bytes": nbytes, "gbs": gbs, "frac_of_measured_hbm": gbs / peak_hbm})
    dq = [0.0, 0.0, 0]
    for lab, v in agg.items():
        if lab.startswith("dense_q8_"):
            dq[0] += v[0]; dq[1] += v[1]; dq[2] += v[2]
    # the dominant kernel is the GEMM template (all its launches of the step: 4 dense + 2 grouped)
    gk = [0.0, 0.0, 0]
    for lab, v in agg.items():
        if v[0]:
            gk[0] += v[0]; gk[1] += v[1]; gk[2] += v[2]
    # The dominant kernel's average launch duration comes from the region that holds nothing but its launches (six per
    # step, back to back as in the step itself): an event pair round every single call, as in the per-call region above,
    # costs about 2.6 us per call and keeps consecutive kernels from overlapping their start-up and tail.
    gemm_flops_step = sum(2.0 * M * N * K for _, N, K in DENSE_SET) + moe_flops(M)
    avg_launch_ms = ms_gemm / (ev_steps * 6)
    achieved = gemm_flops_step / 6 / (avg_launch_ms * 1e-3) / 1e12
    achieved_per_call_events = gk[0] / (gk[1] * 1e-3) / 1e12
    # algorithmic bytes of the six GEMM launches (weights + scales + activations in + output), averaged per launch
    alg = [N * K * 1.0625 + 2.0 * M * K + 2.0 * M * N for _, N, K in DENSE_SET]
    alg.append(E * 2 * F * H * 0.5625 + 2.0 * R * H + 2.0 * R * F)
    alg.append(E * H * F * 0.5625 + 2.0 * R * F + 2.0 * R * H)
    alg_bytes_per_launch = sum(alg) / len(alg)
    roofline = {"kernel": "qgemm_kernel (all instantiations: 4 qgemm_dense + 2 moe_grouped_qgemm launches per step)",
                "bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved / peak_tf,
                "peak_source": peak_src, "traffic": ncu_traffic()[0],
                "traffic_source": {"kind": "quoted from an ncu capture, not measured by this run", "file": os.path.relpath(TRAFFIC_FILE, ROOT),
                                   "captured_at_commit": ncu_traffic()[1]},
                "algorithmic_bytes_per_launch": alg_bytes_per_launch,
                "avg_launch_us": avg_launch_ms * 1e3, "flops_per_launch": gemm_flops_step / 6,
                "timed_region": "%d steps of the six GEMM launches alone, one CUDA-event pair round the region" % ev_steps,
                "with_an_event_pair_round_every_call": {"achieved": achieved_per_call_events,
                                                        "frac": achieved_per_call_events / peak_tf,
                                                        "avg_launch_us": gk[1] / gk[2] * 1e3},
                "dense_q8_only": {"achieved": dq[0] / (dq[1] * 1e-3) / 1e12, "frac": dq[0] / (dq[1] * 1e-3) / 1e12 / peak_tf}}
    gemm_ms = sum(v[1] for lab, v in agg.items() if v[0])
    gemm_fl = sum(v[0] for lab, v in agg.items() if v[0])
    dense_ms = dq[1] / ev_steps
    moe_ms = sum(agg[lab][1] for lab in ("route", "moe_gate_up_q4", "moe_down_q4", "combine")) / ev_steps

    # ---- end-to-end leg: host inputs in pinned memory, copies inside the timed region.  Steps are pipelined the way a
    # server would run them: step i's inputs are copied in on one stream while step i-1 computes and step i-2's
    # results are copied out on a third; two sets of device input and output buffers.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    inA = [dA, [torch.empty_like(a) for a in dA]]
    inL, inX = [dL, torch.empty_like(dL)], [dX, torch.empty_like(dX)]
    outC2, outY2 = [oC, [torch.empty_like(c) for c in oC]], [o["y"], torch.empty_like(o["y"])]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]      # compute of the step that used buffer set b has finished
    ev_out = [torch.cuda.Event() for _ in range(2)]       # its results have reached the host
    e2e_count = [0]

    def step_e2e():
        b = e2e_count[0] & 1
        e2e_count[0] += 1
        s_in.wait_event(ev_done[b])                       # inputs of set b are no longer being read
        with torch.cuda.stream(s_in):
            for d, h in zip(inA[b], hA):
                d.copy_(h, non_blocking=True)
            inL[b].copy_(hL, non_blocking=True); inX[b].copy_(hX, non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        stream.wait_event(ev_out[b])                      # outputs of set b have been copied out
        step(inA[b], inL[b], inX[b], outC=outC2[b], outY=outY2[b])
        ev_done[b].record(stream)
        s_out.wait_event(ev_done[b])
        with torch.cuda.stream(s_out):
            for h, d in zip(hC, outC2[b]):
                h.copy_(d, non_blocking=True)
            hY.copy_(outY2[b], non_blocking=True)
            ev_out[b].record(s_out)

    def timed_e2e(steps):
        sync_all()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        s_in.wait_stream(stream); s_out.wait_stream(stream)
        for _ in range(steps):
            step_e2e()
        stream.wait_stream(s_in); stream.wait_stream(s_out)   # the last results are on the host before the clock stops
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    e2e_steps = max(3, min(args.steps, 50))
    for _ in range(3):
        step_e2e()
    ms_e2e = timed_e2e(e2e_steps)
    h2d = sum(a.numel() * 2 for a in hA) + hL.numel() * 4 + hX.numel() * 2
    d2h = sum(c.numel() * 2 for c in hC) + hY.numel() * 2
    e2e_val = world * flops_step * e2e_steps / (ms_e2e * 1e-3) / 1e12

    sweep = None
    if world == 1 and not args.no_sweep:
        del inA, inL, inX, outC2, outY2
        torch.cuda.empty_cache()
        sampler3 = ClockSampler(local)
        sweep = run_sweep(torch, qg, lib, ctx, dev, stream, peak_tf, peak_hbm)
        qg.poll_status()
        sweep["clocks"] = sampler3.stop()
        wins = sweep.pop("_windows")
        for row, (t0, t1) in zip(sweep["dense"] + sweep["small_m"] + sweep["mx_fp8"] + sweep["attention"] + sweep["moe"], wins):
            row["clocks"] = clocks_in_window(getattr(sampler3, "samples", []), t0 - 0.02, t1 + 0.02)
    if rank == 0:
        dense_h0, moe_h0 = dense_h, moe_h
        cpu = cpu_baseline(dense_h0, moe_h0) if world == 1 else None
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms / args.steps, "ms_per_step_with_per_call_events": ms_events / ev_steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"cfg1 dense Q8 layer set (QKV/O/gate-up/down, K=2048/8192) + cfg3 MoE Q4 layer "
                                   f"(H=2048,E=128,top-8,F=768), M={M} tokens per GPU",
                       "l2": "inputs exceed L2: 403 MB of weights stream per step", "parallelism": f"replicas x{world}",
                       "moe_path": args.moe_path},
            "tok_per_s": {"dense_q8_layer_set": world * M / (dense_ms * 1e-3), "moe_q4_layer": world * M / (moe_ms * 1e-3),
                          "definition": "tokens / time of that layer's calls; not a whole-model figure"},
            "gemm_only": {"tflops": gemm_fl / (gemm_ms * 1e-3) / 1e12, "frac_of_peak": gemm_fl / (gemm_ms * 1e-3) / 1e12 / peak_tf},
            "frac_of_measured_bf16_peak": value / world / peak_tf, "frac_of_nominal_2250": value / world / 2250.0,
            "roofline": roofline, "kernels": detail, "clocks": clocks,
            "per_kernel_region": "a separate region of %d steps with an event pair around every call (about 2.6 us of overhead "
                                 "per call, and no overlap of one kernel's start-up with the previous one's tail), started "
                                 "after a 1 s pause so that it runs at burst clocks like the headline region" % ev_steps,
            "sustained": {"steps": sus_steps, "seconds": ms_sus * 1e-3, "ms_per_step": ms_sus / sus_steps,
                          "tflops": world * flops_step * sus_steps / (ms_sus * 1e-3) / 1e12,
                          "frac_of_sustained_peak": flops_step * sus_steps / (ms_sus * 1e-3) / 1e12 / sustained_peak(),
                          "sustained_peak_tflops": sustained_peak(), "clocks": clocks_sus},
            "e2e": {"value": e2e_val, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / e2e_steps, "steps": e2e_steps,
                    "overlap": "steps pipelined on three streams (copy in / compute / copy out), two buffer sets"},
            "gpu_launches": LAUNCHES_PER_STEP * args.steps,
        }
        if cpu is not None:
            line["cpu_baseline"] = cpu
        if sweep is not None:
            line["sweep"] = sweep
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_case(args):
    """One small case, a few passes, no timing: a target for profiler captures (one kernel, few launches)."""
    import ctypes as C
    import torch
    from paper_2607_19438_b200 import binding as qg
    if args.case == "roles":
        from paper_2607_19438_b200 import build as qg_build
        qg.LIB_PATH = qg_build.build_profile()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    lib, ctx = qg.load(), qg.context(0)
    g = torch.Generator(device=dev); g.manual_seed(0)
    if args.case == "roles":
        return run_roles(lib, ctx, qg, dev, g)
    if args.case == "attention":
        S, Hq, Hkv, d = 2048, 32, 8, 128
        qkv = torch.randn((S, (Hq + 2 * Hkv) * d), device=dev, generator=g).to(torch.bfloat16)
        for _ in range(3):
            qg.prefill_attention(qkv[:, :Hq * d], qkv[:, Hq * d:(Hq + Hkv) * d], qkv[:, (Hq + Hkv) * d:], Hq, Hkv, d)
        qg.poll_status()
        print(json.dumps({"case": args.case, "S": S, "Hq": Hq, "Hkv": Hkv, "d": d, "passes": 3}))
        return
    if args.case == "mx":
        M, N, K = 2048, 16384, 2048
        Wq = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev, generator=g)
        Ws = (torch.randn((N, K // 32), device=dev, generator=g).abs() * (0.02 / 127)).to(torch.float16)
        X = torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16)
        wc, wsf = qg.mx_pack_weights(8, Wq, Ws)
        for _ in range(3):
            ac, asf = qg.mx_quantize(X)
            qg.qgemm_mx_dense(ac, asf, wc, wsf)
        qg.poll_status()
        print(json.dumps({"case": args.case, "M": M, "N": N, "K": K, "passes": 3}))
        return
    if args.case == "small_m":
        M, N, K = 4, 28672, 4096
        Wq = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev, generator=g)
        Ws = (torch.randn((N, K // 32), device=dev, generator=g).abs() * (0.02 / 127)).to(torch.float16)
        A = torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        for _ in range(3):
            flush.zero_()
            qg.qgemm_small_m(8, A, Wq, Ws)
        qg.poll_status()
        print(json.dumps({"case": args.case, "M": M, "N": N, "K": K, "passes": 3}))
        return
    H, F, k = MOE["H"], MOE["F"], MOE["k"]
    E, M = 16, 256
    R = M * k
    W1q = torch.randint(0, 256, (E, 2 * F, H // 2), dtype=torch.uint8, device=dev, generator=g)
    W2q = torch.randint(0, 256, (E, H, F // 2), dtype=torch.uint8, device=dev, generator=g)
    W1s = (torch.randn((E, 2 * F, H // 32), device=dev, generator=g).abs() * (0.02 / 7)).to(torch.float16)
    W2s = (torch.randn((E, H, F // 32), device=dev, generator=g).abs() * (0.02 / 7)).to(torch.float16)
    L = torch.randn((M, E), device=dev, generator=g)
    X = torch.randn((M, H), device=dev, generator=g).to(torch.bfloat16)
    for _ in range(3):
        r = qg.moe_route(L, k, X=X)
        Hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, 4, r["Xperm"], r["offsets"], W1q, W1s)
        Dw = qg.moe_grouped_qgemm(qg.MODE_DOWN_WEIGHTED, 4, Hh, r["offsets"], W2q, W2s, topk_w=r["topk_w"].view(-1),
                                  row_pair=r["row_pair"], k=k)
        qg.moe_combine(Dw, r["pair_row"], k)
    qg.poll_status()
    print(json.dumps({"case": args.case, "E": E, "M": M, "rows_per_expert": R / E, "passes": 3}))


def run_roles(lib, ctx, qg, dev, g):
    """Cycle accounting of the GEMM kernel's roles (profiling build of the library): for one launch each of two dense
    and the two grouped GEMMs of the bench step, the cycles the first CTA's producer, MMA-issuing, conversion and
    epilogue warps spent in each of their waits, next to the cycles from the CTA's start to its last commit."""
    import ctypes as C
    import torch
    lib.qg_debug_set_stats.argtypes = [C.c_void_p, C.c_void_p]
    lib.qg_debug_set_stats.restype = None
    stats = torch.zeros(148 * 12 + 16 + 2 * 148 + 8, dtype=torch.int64, device=dev)
    names = ["x_producer_wait", "w_producer_wait", "mma_wait_accumulator", "mma_wait_stage_full", None,
             "convert_wait_packed", "convert_wait_stage_free", "convert_arithmetic_and_store", "epilogue_wait",
             "epilogue_drain", "mma_issue", None]
    rows = []

    def measure(label, call, kblocks_per_tile):
        lib.qg_debug_set_stats(ctx, None)
        for _ in range(3):
            call()
        stats.zero_()
        torch.cuda.synchronize()
        lib.qg_debug_set_stats(ctx, C.c_void_p(stats.data_ptr()))
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); call(); e1.record()
        torch.cuda.synchronize()
        lib.qg_debug_set_stats(ctx, None)
        st = stats.cpu().numpy()
        marks = st[148 * 12:148 * 12 + 16]
        row = {"call": label, "event_us_profiling_build": round(e0.elapsed_time(e1) * 1e3, 1),
               "cta0_cycles_start_to_last_commit": int(marks[3] - marks[0]),
               "cta0_cycles_start_to_first_stage_full": int(marks[2] - marks[0]),
               "k_blocks_per_tile": kblocks_per_tile,
               "cta0_cycles_in": {n: int(st[i]) for i, n in enumerate(names) if n}}
        rows.append(row)

    for (M, N, K) in [(2048, 2048, 2048), (2048, 2048, 8192)]:
        Wq = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev, generator=g)
        Ws = (torch.randn((N, K // 32), device=dev, generator=g).abs() * (0.02 / 127)).to(torch.float16)
        A = torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16)
        out = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        measure(f"dense Q8 {M}x{N}x{K}", lambda: qg.qgemm_dense(8, A, Wq, Ws, out=out), K // 64)
    H, F, k, E, M = MOE["H"], MOE["F"], MOE["k"], MOE["E"], 2048
    W1q = torch.randint(0, 256, (E, 2 * F, H // 2), dtype=torch.uint8, device=dev, generator=g)
    W2q = torch.randint(0, 256, (E, H, F // 2), dtype=torch.uint8, device=dev, generator=g)
    W1s = (torch.randn((E, 2 * F, H // 32), device=dev, generator=g).abs() * (0.02 / 7)).to(torch.float16)
    W2s = (torch.randn((E, H, F // 32), device=dev, generator=g).abs() * (0.02 / 7)).to(torch.float16)
    L = torch.randn((M, E), device=dev, generator=g)
    X = torch.randn((M, H), device=dev, generator=g).to(torch.bfloat16)
    r = qg.moe_route(L, k, X=X)
    Hh = qg.moe_grouped_qgemm(qg.MODE_GATE_UP_SILU, 4, r["Xperm"], r["offsets"], W1q, W1s)
    measure(f"MoE Q4 gate/up, {M} tokens, {E} experts", lambda: qg.moe_grouped_qgemm(
        qg.MODE_GATE_UP_SILU, 4, r["Xperm"], r["offsets"], W1q, W1s, out=Hh), H // 64)
    Dw = torch.empty((M * k, H), dtype=torch.bfloat16, device=dev)
    measure(f"MoE Q4 down, {M} tokens, {E} experts", lambda: qg.moe_grouped_qgemm(
        qg.MODE_DOWN_WEIGHTED, 4, Hh, r["offsets"], W2q, W2s, topk_w=r["topk_w"].view(-1), row_pair=r["row_pair"], k=k,
        out=Dw), F // 64)
    qg.poll_status()
    print(json.dumps({"case": "roles", "rows": rows}, indent=1))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-configuration sweep block")
    ap.add_argument("--profile-run", action="store_true",
                    help="warm-up and the timed steps only (no per-call region, sustained run, end-to-end leg, sweep or CPU "
                         "baseline): a short target for profiler launch lists; prints a reduced JSON line")
    ap.add_argument("--moe-path", default="staged", choices=["fused", "staged"],
                    help="staged: permute, routing-weighted bf16 rows, slot-ordered combine (deterministic, faster on "
                         "B200); fused: token gather in the gate/up loads + fp32 accumulate in the down epilogue")
    ap.add_argument("--case", default=None, choices=["moe_small", "attention", "small_m", "mx", "roles"],
                    help="run one small case a few times and exit (for profiler captures): moe_small = the cfg-3 MoE "
                         "layer shape with 16 experts and 256 tokens (128 rows per expert); attention = cfg-4 heads "
                         "(32 / 8, d = 128) at 2048 positions; small_m = the cfg-4 gate/up weights (28672 x 4096, Q8) "
                         "times 4 tokens; mx = the block-scaled FP8 GEMM 2048 x 16384 x 2048; roles = per-role wait cycles of the "
                         "GEMM kernel from a -DQG_PROFILE build of the library (not a profiler target)")
    args = ap.parse_args()
    if args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
