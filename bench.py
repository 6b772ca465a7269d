#!/usr/bin/env python
"""Benchmark of the FAEDKV / IWDFT hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--decode-iters D]

One "step" is one pass of the whole hot path over one synthetic, Llama-3-8B-shaped cache (32 layers,
8 kv heads / 32 query heads, head_dim 128, batch 1, T = P = 32768 bf16 tokens, per-layer mixed bin
masks keeping 1/8 of the bins):

    A. faedkv_compress_prefill of all 32 layers                      -> prefill tokens/s (the `value`)
    B. D decode iterations of (faedkv_append + faedkv_decode_attn) on all 32 layers, then D more through
       the fused faedkv_append_decode_attn                           -> decode us / layer / step
    C. faedkv_reconstruct of all 32 layers (L = P)

Beside the timed step the line carries: `prefill_fft` (the same prefill through prefill_mode = FFT, the
paper's own O(N log N) route, for comparison with the tensor-core contraction that `value` measures) and
`decode.configs` (decode us / layer / step at the configs[2] and configs[3] shapes, whose state comes
from a real prefill).

Inputs are resident in HBM before the timed region; every layer's tensors are distinct and the layers
are cycled (4 GiB of K/V, 2 GiB of coefficients), so nothing survives in the 126 MB L2 between uses.
`e2e` repeats phase A through the same C-ABI calls with the K/V in pinned HOST memory and the
coefficients copied back to the host, copies inside the timed region.

With N > 1 (torchrun) every rank runs the same workload on its own GPU: the path needs no
inter-GPU exchange ("replicas only"), `value` is the sum over ranks, time the max over ranks.

`--impl reference` times the float64 CPU oracle, as it stands, on the host cores on a bounded
sample of the same workload and prints the same JSON line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "iwdft_prefill_tokens_per_s"
UNIT = "tokens/s"

WORKLOAD = dict(name="configs[1]: Llama-3-8B-shaped full cache, prefill 32768 tokens at 1/8 bin retention",
                config=1, n_layers=32, n_kv_heads=8, n_q_heads=32, head_dim=128, batch=1, T=32768,
                M=4096, mask="mixed")


def workload_config(W, prefill_path, twiddle_terms):
    """The `config` object of a bench line (both arms print the same one for the same workload)."""
    return {"workload": W["name"], "n_layers": W["n_layers"], "n_kv_heads": W["n_kv_heads"], "n_q_heads": W["n_q_heads"],
            "head_dim": W["head_dim"], "batch": W["batch"], "T": W["T"], "n_dft": W["T"], "n_bins": W["M"],
            "mask": "mixed (seeded, per layer)", "prefill_path": prefill_path, "twiddle_terms": twiddle_terms,
            "l2": "inputs larger than L2: 32 layers cycled, 128 MiB K/V + 64 MiB planes per layer",
            "multi_gpu": "replicas only"}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# --------------------------------------------------------------------------------------- ranks
def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (every rank gets the result).  The path
    needs no inter-GPU exchange; this one reduction only puts the slowest replica's time on the line."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_value(units_per_rank: float, world: int, ms: float) -> float:
    """Weak scaling over independent replicas: every rank processes `units_per_rank` in `ms` (the maximum over
    ranks), so the job's throughput is world * units_per_rank / time."""
    return world * units_per_rank / (ms * 1e-3)


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # the busiest half of the samples is "under load"
        sm_sorted = sorted(sm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_mhz_min": sm_sorted[0] if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------- reference arm
def _oracle_units_seconds(orc, torch, synth, n_units, T, P, bins, seed):
    """Time the oracle's pruned DFT of `n_units` units (kv heads of layer 0, K) over the bins given."""
    K, _ = synth.make_kv(seed, 1, n_units, T, 128, dtype=torch.bfloat16)
    x = K[0].double().numpy()
    t0 = time.perf_counter()
    orc.compress(x, P, bins)
    return time.perf_counter() - t0


def _cpu_config0(orc, torch, synth):
    """configs[0] in full on the oracle: prefill of the 16 units, 64 appends, reconstruction (seconds each)."""
    import numpy as np
    P = T = 2048
    M, H, steps = 256, 8, 64
    seed = synth.config_seed(0, 0)
    bins = orc.plan(P, orc.mask_lowpass(P, M))
    K, V = synth.make_kv(seed, 1, H, T, 128, dtype=torch.float32)
    xs = [K[0].double().numpy(), V[0].double().numpy()]
    t0 = time.perf_counter()
    planes = [orc.compress(x, P, bins) for x in xs]
    t1 = time.perf_counter()
    toks = [synth.make_token(seed, s_, 1, H, 128, pos=T + s_, dtype=torch.float32) for s_ in range(steps)]
    toks = [(k[0].double().numpy(), v[0].double().numpy()) for k, v in toks]
    planes = [(np.ascontiguousarray(re), np.ascontiguousarray(im)) for re, im in planes]
    t2 = time.perf_counter()
    for s_ in range(steps):
        for kv in range(2):
            for h in range(H):
                orc.append(planes[kv][0][h], planes[kv][1][h], P, bins, T + s_, toks[s_][kv][h])
    t3 = time.perf_counter()
    for kv in range(2):
        for h in range(H):
            orc.reconstruct(planes[kv][0][h], planes[kv][1][h], P, bins, P)
    t4 = time.perf_counter()
    return {"what": "configs[0] in full: prefill of 2 x 8 units (2048 tokens, 256 bins), 64 appends, reconstruct L = 2048",
            "prefill_s": t1 - t0, "appends_s": t3 - t2, "reconstruct_s": t4 - t3, "total_s": (t1 - t0) + (t3 - t2) + (t4 - t3),
            "prefill_tokens_per_s": T / (t1 - t0), "append_us_per_step": (t3 - t2) / steps * 1e6}


def _cpu_decode_slice(orc, torch, synth, DW, rows_cap=2048):
    """One unit slice of the decode calls at a decode workload's shape: 8 appends of one (sequence, kv head)'s K
    planes, the reconstruction of `rows_cap` of its rows and decode attention of the kv head's query heads over
    `rows_cap` positions; each scaled linearly to a layer-step of the workload (units and rows are independent)."""
    import numpy as np
    P = T = DW["T"]
    M, H, HQ, B = DW["M"], DW["n_kv_heads"], DW["n_q_heads"], DW["batch"]
    seed = synth.config_seed(DW["config"])
    bins = orc.plan(P, orc.mask_mixed(P, M, 0, seed))
    rng = np.random.default_rng(seed)
    re, im = rng.standard_normal((M, 128)) * np.sqrt(T), rng.standard_normal((M, 128)) * np.sqrt(T)
    vre, vim = rng.standard_normal((M, 128)) * np.sqrt(T), rng.standard_normal((M, 128)) * np.sqrt(T)
    x = rng.standard_normal(128)
    t0 = time.perf_counter()
    for s_ in range(8):
        orc.append(re, im, P, bins, T + s_, x)
    t_app = (time.perf_counter() - t0) / 8
    rows = min(rows_cap, P)
    t0 = time.perf_counter()
    orc.reconstruct(re, im, P, bins, rows)
    t_rec = time.perf_counter() - t0
    G = HQ // H
    q = rng.standard_normal((G, 128))
    t0 = time.perf_counter()
    orc.decode_attn(q, re / T, im / T, vre, vim, P, bins, rows)
    t_att = time.perf_counter() - t0
    units = B * H
    return {"workload": DW["name"], "extrapolated": True,
            "slice": f"1 of {units} (sequence, kv head) units; {rows} of {P} positions for reconstruct / attention",
            "slice_seconds": {"append_one_tensor": t_app, "reconstruct_one_tensor": t_rec, "decode_attn": t_att},
            "append_us_per_layer_step": t_app * 2 * units * 1e6,
            "reconstruct_ms_per_layer": t_rec * (P / rows) * 2 * units * 1e3,
            "decode_attn_us_per_layer_step": t_att * (P / rows) * units * 1e6}


def cpu_baseline(target_s: float = 10.0, extras: bool = True) -> dict:
    """Oracle prefill throughput on the host cores, from a bounded sample extrapolated over the independent
    (layer, head, tensor) units of the workload; with `extras` also the same on one thread, configs[0] in full and
    a unit slice of the decode calls at the streaming-decode shape."""
    import torch
    import oracle as orc
    from paper_2507_20030_b200 import synth
    orc.build()
    W = WORKLOAD
    P = T = W["T"]
    cores = len(os.sched_getaffinity(0))
    orc.set_threads(cores)
    bins = orc.plan(P, orc.mask_mixed(P, W["M"], 0, synth.config_seed(W["config"])))
    seed = synth.config_seed(W["config"], 0)
    t1 = _oracle_units_seconds(orc, torch, synth, 1, T, P, bins, seed)
    n_units = int(max(1, min(W["n_kv_heads"], round(target_s / t1))))
    t_sample = t1 if n_units == 1 else _oracle_units_seconds(orc, torch, synth, n_units, T, P, bins, seed)
    units = W["n_layers"] * W["batch"] * W["n_kv_heads"] * 2            # (layer, head, K|V)
    full_s = t_sample * units / n_units
    res = {"value": W["batch"] * T / full_s, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": (f"pruned DFT of {n_units} of {units} units (layer 0, kv heads 0..{n_units - 1}, K): all {T} tokens "
                      f"x 128 channels x {W['M']} bins in {t_sample:.2f} s; extrapolated linearly over units"),
           "sample_seconds": t_sample}
    if extras:
        # one thread: every 8th retained bin of one unit (bins are independent loops of equal cost)
        orc.set_threads(1)
        sub = bins[::8]
        t_one = _oracle_units_seconds(orc, torch, synth, 1, T, P, sub, seed)
        full_one = t_one * (len(bins) / len(sub)) * units
        res["one_thread"] = {"value": W["batch"] * T / full_one, "unit": UNIT, "cores": 1,
                             "sample": f"{len(sub)} of {len(bins)} bins of 1 unit in {t_one:.2f} s; extrapolated linearly over bins and units",
                             "sample_seconds": t_one}
        orc.set_threads(cores)
        res["config0_full"] = _cpu_config0(orc, torch, synth)
        res["decode_slices"] = [_cpu_decode_slice(orc, torch, synth, DECODE_WORKLOADS[0])]
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    W = WORKLOAD
    vals = []
    base = None
    for i in range(args.warmup + args.steps):
        base = cpu_baseline(target_s=max(2.0, min(12.0, 90.0 / max(1, args.warmup + args.steps))), extras=False)
        if i >= args.warmup:
            vals.append(base)
    v = statistics.mean(b["value"] for b in vals)
    ms = statistics.mean(W["batch"] * W["T"] / b["value"] for b in vals) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(W, "tcgen05-bf16", 1),     # the same workload description as our arm's line
            "extrapolated": True,
            "cpu_baseline": {**base, "value": v},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))



# --------------------------------------------------------------------------------------- profiler figures
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the prefill contraction at the bench
# size, from a profiler capture, together with the hash of the kernel source the capture was taken from.  The
# figure is reported only while the kernel source still hashes to that value; after any change to the kernel it
# reads null until the capture is repeated.
PREFILL_TRAFFIC = {"bytes": 183.5e6, "kernel_sha256_16": "524bb33b3ed2290c", "captured": "2026-11-28"}


def _kernel_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("k_prefill_umma.cuh", "umma_common.cuh"):
        with open(os.path.join(ROOT, "paper_2507_20030_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def prefill_kernel_traffic():
    cur = _kernel_hash()
    if PREFILL_TRAFFIC["bytes"] is not None and PREFILL_TRAFFIC["kernel_sha256_16"] == cur:
        return PREFILL_TRAFFIC["bytes"], (f"ncu capture of {PREFILL_TRAFFIC['captured']}, one launch at this size; "
                                          f"kernel source sha256 {cur}")
    return None, f"kernel source (sha256 {cur}) has changed since the last profiler capture"


# --------------------------------------------------------------------------------------- decode sections
DECODE_WORKLOADS = [
    dict(name="configs[2]: streaming decode, batch 16, prefill 16384 tokens at 1/8 retention", config=2,
         n_layers=32, n_kv_heads=8, n_q_heads=32, batch=16, T=16384, M=2048),
    dict(name="configs[3]: long context, batch 1, 131072 tokens at 1/16 retention", config=3,
         n_layers=32, n_kv_heads=8, n_q_heads=32, batch=1, T=131072, M=8192),
    dict(name="configs[4] cell: 32 kv = 32 query heads, batch 32, 4096 tokens at 1/8 retention", config=4,
         n_layers=32, n_kv_heads=32, n_q_heads=32, batch=32, T=4096, M=512),
]


def recon_alu_roofline(P, n_cols, seconds):
    """The reconstruction as float32 arithmetic: a real inverse FFT of length P per channel is a complex FFT of
    N = P/2 points, 5 N log2 N flop, against the float32 FMA peak 148 SMs x 128 lanes x 2 x 1.965 GHz.  At the
    bench sizes this floor is level with the HBM floor, so both fractions are reported."""
    N = P // 2
    flop = 5.0 * N * (N.bit_length() - 1) * n_cols
    peak = 148 * 128 * 2 * 1.965e9 / 1e12
    tf = flop / seconds / 1e12
    return {"bound": "alu", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
            "flop_model": "5 N log2 N per channel, N = P/2"}


def decode_section(torch, binding, synth, dev, W, peaks, iters, graphs=True):
    """Decode us / layer / step at one workload shape: the state comes from a real prefill (one layer of
    K/V resident at a time), then the three decode calls are timed over all layers, each loop replayed
    as one CUDA graph (launch gaps excluded) and, for the fused call, also launched eagerly."""
    NL, H, HQ, B, T, M = (W[k] for k in ("n_layers", "n_kv_heads", "n_q_heads", "batch", "T", "M"))
    P, D = T, 128
    ctx = binding.Context(n_layers=NL, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=binding.BF16,
                          n_sink=10, n_recent=50)       # the paper's window sizes; only step_windowed looks at them
    seed = synth.config_seed(W["config"])
    cKs, cVs, tls = [], [], []
    for l in range(NL):
        ctx.plan(l, binding.mask_mixed(P, M, l, seed))
    prefill_ms = []
    for l in range(NL):
        K, V = synth.make_kv(synth.config_seed(W["config"], l), B, H, T, D, dtype=torch.bfloat16, device=dev)
        cK, cV = ctx.alloc_coef(l, B, device=dev), ctx.alloc_coef(l, B, device=dev)
        tl = torch.zeros(B, dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.compress_prefill(l, K, V, cK, cV, tl)
        b.record()
        cKs.append(cK); cVs.append(cV); tls.append(tl)
        torch.cuda.synchronize()
        prefill_ms.append(a.elapsed_time(b))
        del K, V
    # the state's own prefill (tensor-core contraction), one launch per layer; the first layers warm the kernel up
    pf = sorted(prefill_ms[min(2, NL - 1):])
    pf_ms = pf[len(pf) // 2]
    pf_flop = 2.0 * (2 * M) * T * (B * H * D) * 2
    prefill = {"ms_per_layer": pf_ms, "tokens_per_s": B * T / (pf_ms * 1e-3 * NL), "flop_per_layer": pf_flop,
               "bound": "tensor", "achieved": pf_flop / (pf_ms * 1e-3) / 1e12, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
               "frac": pf_flop / (pf_ms * 1e-3) / 1e12 / peaks["bf16_sustained"],
               "frac_of_burst": pf_flop / (pf_ms * 1e-3) / 1e12 / peaks["bf16"],
               "what": "median over layers of the event-timed faedkv_compress_prefill that builds this section's state"}
    k_new, v_new = synth.make_token(seed, 0, B, H, D, pos=T, dtype=torch.bfloat16, device=dev)
    q = synth.make_q(seed, 0, B, HQ, D, dtype=torch.bfloat16, device=dev)
    out = torch.empty((B, HQ, D), dtype=torch.bfloat16, device=dev)
    # windows of the paper's workflow (sink 10 + recent 50), filled with tokens of the same distributions
    wK, wV = synth.make_kv(seed + 7, B, H, 60, D, pos0=T - 60, dtype=torch.bfloat16, device=dev)
    loops = {
        "append": lambda: [ctx.append(l, k_new, v_new, cKs[l], cVs[l], tls[l]) for l in range(NL)],
        "decode_attn": lambda: [ctx.decode_attn(l, q, cKs[l], cVs[l], tls[l], out) for l in range(NL)],
        "append_decode_attn": lambda: [ctx.append_decode_attn(l, k_new, v_new, q, cKs[l], cVs[l], tls[l], out)
                                       for l in range(NL)],
        "step_windowed": lambda: [ctx.step_windowed(l, k_new, v_new, q, cKs[l], cVs[l], wK, wV, tls[l], out) for l in range(NL)],
    }
    coef_bytes = 2 * B * H * 2 * M * D * 4                      # K and V planes of one layer
    alg_bytes = {"append": 2 * coef_bytes, "decode_attn": coef_bytes, "append_decode_attn": 2 * coef_bytes,
                 "step_windowed": 2 * coef_bytes}
    if not W.get("no_reconstruct"):
        Ko = torch.empty((B, H, P, D), dtype=torch.bfloat16, device=dev)
        Vo = torch.empty_like(Ko)
        loops["reconstruct"] = lambda: [ctx.reconstruct(l, cKs[l], cVs[l], tls[l], P, Ko, Vo) for l in range(NL)]
        alg_bytes["reconstruct"] = coef_bytes + 2 * B * H * P * D * 2          # planes in + bf16 rows out
    res = {"workload": W["name"], "iters": iters, "planes_bytes_per_layer": coef_bytes, "prefill": prefill,
           "l2": "32 layers cycled: %.0f MiB of planes per layer" % (coef_bytes / 2 ** 20)}
    side = torch.cuda.Stream()
    for name, fn in loops.items():
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        eager_us = a.elapsed_time(b) / iters / NL * 1e3
        if not graphs:
            res[name] = {"us_eager_launches": eager_us}
            continue
        graph = torch.cuda.CUDAGraph()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.synchronize()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(iters):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / iters / NL * 1e3
        gbs = alg_bytes[name] / (us * 1e-6) / 1e9
        res[name] = {"us": us, "us_eager_launches": eager_us, "bytes": alg_bytes[name], "bound": "hbm", "achieved": gbs,
                     "peak": peaks["hbm"], "unit": "GB/s", "frac": gbs / peaks["hbm"], "frac_of_nominal_8000": gbs / 8000.0}
        if name == "reconstruct":
            res[name]["alu"] = recon_alu_roofline(P, 2 * B * H * D, us * 1e-6)
    if graphs:
        res["decode_us_per_layer_step"] = res["append_decode_attn"]["us"]
        res["decode_us_per_layer_step_two_calls"] = res["append"]["us"] + res["decode_attn"]["us"]
    # the same windowed workflow with the block-deferred fold: 50 tokens folded at once every 50th step, the
    # other steps only read the planes.  All layers' steps (one CUDA graph, or eager launches) are run 50
    # times, each run timed; the counters are first set so that the first of the 50 is the one that folds.
    DEFER, S_, R_ = 50, 10, 50
    ctx2 = binding.Context(n_layers=NL, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=binding.BF16,
                           n_sink=S_, n_recent=R_, n_defer=DEFER)
    for l in range(NL):
        ctx2.plan(l, binding.mask_mixed(P, M, l, seed))
    w2K, w2V = synth.make_kv(seed + 9, B, H, S_ + R_ + DEFER, D, pos0=T - 60 - DEFER, dtype=torch.bfloat16, device=dev)
    fn = lambda: [ctx2.step_windowed(l, k_new, v_new, q, cKs[l], cVs[l], w2K, w2V, tls[l], out) for l in range(NL)]
    t_now = int(tls[0][0].item())
    t_fold = S_ + R_ + ((t_now - S_ - R_) // DEFER + 2) * DEFER - 1      # a step from this count folds
    run = fn
    if graphs:
        for tl in tls:
            tl.fill_(t_fold - 3)
        graph = torch.cuda.CUDAGraph()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.synchronize()
        run = graph.replay
        for _ in range(2):
            run()
    else:
        for tl in tls:
            tl.fill_(t_fold)
    torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(DEFER + 1)]
    evs[0].record()
    for i in range(DEFER):
        run()
        evs[i + 1].record()
    torch.cuda.synchronize()
    per = [evs[i].elapsed_time(evs[i + 1]) / NL * 1e3 for i in range(DEFER)]
    us = evs[0].elapsed_time(evs[DEFER]) / DEFER / NL * 1e3
    nbytes = coef_bytes + 2 * coef_bytes / DEFER
    gbs = nbytes / (us * 1e-6) / 1e9
    res["step_windowed_deferred"] = {
        "us": us, "us_step_without_fold": sorted(per)[len(per) // 2], "us_step_with_fold": per[0], "defer": DEFER,
        "launch": "one CUDA graph per step of all layers" if graphs else "eager launches",
        "bytes": nbytes, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s", "frac": gbs / peaks["hbm"],
        "frac_of_nominal_8000": gbs / 8000.0,
        "what": "mean over 50 consecutive steps, the first of which folds 50 tokens into every layer's planes; "
                "bytes = planes read once per step + read and written once per 50 steps"}
    if ctx2.device_status() != 0:
        raise RuntimeError("a kernel reported a device-side timeout; the numbers are invalid")
    ctx2.close()
    if ctx.device_status() != 0:
        raise RuntimeError("a kernel reported a device-side timeout; the numbers are invalid")
    ctx.close()
    del cKs, cVs
    torch.cuda.empty_cache()
    return res


# --------------------------------------------------------------------------------------- configs[0]
def config0_section(torch, binding, synth, dev):
    """configs[0] on the GPU as it is stated: 1 layer, 8 kv heads, 2048 float32 tokens, 256 low-pass bins; prefill, 64
    appends, reconstruct (L = 2048).  Its planes (8 MiB) sit in L2, so only times are reported, no bandwidth
    fraction; the oracle's times for the same work are under cpu_baseline.config0_full."""
    P = T = 2048
    M, H, HQ, steps = 256, 8, 32, 64
    seed = synth.config_seed(0, 0)
    ctx = binding.Context(n_layers=1, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=1, kv_dtype=binding.F32)
    ctx.plan(0, binding.mask_lowpass(P, M))
    K, V = synth.make_kv(seed, 1, H, T, 128, dtype=torch.float32, device=dev)
    toks = [synth.make_token(seed, s_, 1, H, 128, pos=T + s_, dtype=torch.float32, device=dev) for s_ in range(steps)]
    cK, cV = ctx.alloc_coef(0, 1, device=dev), ctx.alloc_coef(0, 1, device=dev)
    tl = torch.zeros(1, dtype=torch.int32, device=dev)
    Ko = torch.empty((1, H, P, 128), dtype=torch.float32, device=dev)
    Vo = torch.empty_like(Ko)

    def run():
        ctx.compress_prefill(0, K, V, cK, cV, tl)
        for k, v in toks:
            ctx.append(0, k, v, cK, cV, tl)
        ctx.reconstruct(0, cK, cV, tl, P, Ko, Vo)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    reps = 10
    tp = ta = tr = 0.0
    for _ in range(reps):
        ev[0].record()
        ctx.compress_prefill(0, K, V, cK, cV, tl)
        ev[1].record()
        for k, v in toks:
            ctx.append(0, k, v, cK, cV, tl)
        ev[2].record()
        ctx.reconstruct(0, cK, cV, tl, P, Ko, Vo)
        ev[3].record()
        torch.cuda.synchronize()
        tp += ev[0].elapsed_time(ev[1]); ta += ev[1].elapsed_time(ev[2]); tr += ev[2].elapsed_time(ev[3])
    if ctx.device_status() != 0:
        raise RuntimeError("a kernel reported a device-side timeout; the numbers are invalid")
    ctx.close()
    return {"workload": "configs[0]: 1 layer, batch 1, 8 kv heads, 2048 float32 tokens, 256 low-pass bins, 64 appends, reconstruct",
            "prefill_us": tp / reps * 1e3, "prefill_tokens_per_s": T / (tp / reps * 1e-3), "prefill_path": "FFT-shaped float32 (default for float32 K/V)",
            "append_us_per_step": ta / reps / steps * 1e3, "reconstruct_us": tr / reps * 1e3, "total_us": (tp + ta + tr) / reps * 1e3,
            "launch": "eager, CUDA events around each phase; planes are L2-resident (8 MiB)"}


# --------------------------------------------------------------------------------------- configs[4] sweep
def sweep_cells():
    """The 48 cells of the retention / batch sweep on the MHA cache (32 kv = 32 query heads)."""
    cells = []
    for T in (4096, 16384):
        for B in (1, 8, 32):
            for r_den in (4, 8, 16, 32):
                for mask in ("lowpass", "mixed"):
                    cells.append(dict(T=T, batch=B, r_den=r_den, M=T // r_den, mask=mask))
    return cells


def sweep_section(torch, binding, synth, dev, peaks, cells, iters=5):
    """Per cell: the prefill through both routes (tensor-core contraction, FFT-shaped) and the fused decode step
    (CUDA graph over the cell's layers).  A cell uses as many layers as make its planes exceed twice the L2
    (at least 4, at most 32), so that no layer's planes survive in L2 between steps."""
    H = HQ = 32
    D = 128
    out_cells = []
    seed = synth.config_seed(4)
    side = torch.cuda.Stream()
    for c in cells:
        T, B, M = c["T"], c["batch"], c["M"]
        P = T
        coef_bytes = 2 * B * H * 2 * M * D * 4                  # K and V planes of one layer
        NL = int(min(32, max(4, -(-2 * 126 * 2 ** 20 // coef_bytes))))
        ctxs = {}
        for route, mode in (("gemm", binding.PREFILL_UMMA), ("fft", binding.PREFILL_FFT)):
            ctxs[route] = binding.Context(n_layers=NL, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B,
                                          kv_dtype=binding.BF16, prefill_mode=mode)
            for l in range(NL):
                m = binding.mask_lowpass(P, M) if c["mask"] == "lowpass" else binding.mask_mixed(P, M, l, seed)
                ctxs[route].plan(l, m)
        kv_bytes = 2 * B * H * T * D * 2
        n_kv = NL if kv_bytes * NL <= (2 << 30) else 1          # small caches: one per layer, so that none is L2-resident
        KV = [synth.make_kv(seed + 31 * l + T + B, B, H, T, D, dtype=torch.bfloat16, device=dev) for l in range(n_kv)]
        cKs = [ctxs["gemm"].alloc_coef(l, B, device=dev) for l in range(NL)]
        cVs = [ctxs["gemm"].alloc_coef(l, B, device=dev) for l in range(NL)]
        tls = [torch.zeros(B, dtype=torch.int32, device=dev) for _ in range(NL)]
        ms = {}
        for route in ("fft", "gemm"):                             # the contraction last: its planes are the decode state
            ctx = ctxs[route]
            run = lambda: [ctx.compress_prefill(l, KV[l % n_kv][0], KV[l % n_kv][1], cKs[l], cVs[l], tls[l]) for l in range(NL)]
            run()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            run()
            b.record()
            torch.cuda.synchronize()
            ms[route] = a.elapsed_time(b) / NL
        ctx = ctxs["gemm"]
        k_new, v_new = synth.make_token(seed, 0, B, H, D, pos=T, dtype=torch.bfloat16, device=dev)
        q = synth.make_q(seed, 0, B, HQ, D, dtype=torch.bfloat16, device=dev)
        out = torch.empty((B, HQ, D), dtype=torch.bfloat16, device=dev)
        fn = lambda: [ctx.append_decode_attn(l, k_new, v_new, q, cKs[l], cVs[l], tls[l], out) for l in range(NL)]
        graph = torch.cuda.CUDAGraph()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.synchronize()
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / iters / NL * 1e3
        gbs = 2 * coef_bytes / (us * 1e-6) / 1e9
        flop = 2.0 * (2 * M) * T * (B * H * D) * 2
        for cx in ctxs.values():
            if cx.device_status() != 0:
                raise RuntimeError("a kernel reported a device-side timeout; the numbers are invalid")
            cx.close()
        out_cells.append({"T": T, "B": B, "r": f"1/{c['r_den']}", "M": M, "mask": c["mask"], "layers": NL,
                          "fused_us": round(us, 2), "fused_frac": round(gbs / peaks["hbm"], 4),
                          "gemm_ms": round(ms["gemm"], 4), "gemm_tflops": round(flop / (ms["gemm"] * 1e-3) / 1e12, 1),
                          "fft_ms": round(ms["fft"], 4), "fft_tok_s": round(B * T / (ms["fft"] * 1e-3)),
                          "gemm_tok_s": round(B * T / (ms["gemm"] * 1e-3)),
                          "faster_prefill": "gemm" if ms["gemm"] < ms["fft"] else "fft"})
        del KV, cKs, cVs
        torch.cuda.empty_cache()
    return {"what": "configs[4]: MHA cache (32 kv = 32 query heads, 32-layer model; per cell the layers that are cycled are listed), "
                    "fused step = faedkv_append_decode_attn us per layer (CUDA graph), frac = planes read + written / measured HBM peak; "
                    "prefill ms per layer through the tensor-core contraction and through the FFT-shaped route",
            "cells": out_cells}

# --------------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2507_20030_b200 import binding, build, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    peaks = _peaks()
    if args.only_decode_config:
        # small profiling case: one decode section alone, eager launches, optionally fewer layers
        DW = dict(DECODE_WORKLOADS[args.only_decode_config - 2])
        if args.layers:
            DW["n_layers"] = args.layers
            DW["name"] += f" [first {args.layers} layers only: profiling case, not a bench value]"
        res = decode_section(torch, binding, synth, torch.device("cuda", local), DW, peaks, args.decode_config_iters,
                             graphs=False)
        if rank == 0:
            print(json.dumps({"profiling_case": res}))
        return
    W = dict(WORKLOAD)
    if args.layers:
        W["n_layers"] = args.layers
        W["name"] += f" [first {args.layers} layers only: profiling case, not a bench value]"
    NL, H, HQ, D, B, T, M = (W[k] for k in ("n_layers", "n_kv_heads", "n_q_heads", "head_dim", "batch", "T", "M"))
    P = T
    dev = torch.device("cuda", local)
    ctx = binding.Context(n_layers=NL, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B,
                          kv_dtype=binding.BF16, prefill_mode=args.prefill_mode,
                          twiddle_terms=args.twiddle_terms)
    base_seed = synth.config_seed(W["config"])
    for l in range(NL):
        ctx.plan(l, binding.mask_mixed(P, M, l, base_seed))

    # ---- resident inputs and state
    Ks, Vs, cKs, cVs, tls = [], [], [], [], []
    for l in range(NL):
        K, V = synth.make_kv(synth.config_seed(W["config"], l), B, H, T, D, dtype=torch.bfloat16, device=dev)
        Ks.append(K); Vs.append(V)
        cKs.append(ctx.alloc_coef(l, B, device=dev)); cVs.append(ctx.alloc_coef(l, B, device=dev))
        tls.append(torch.zeros(B, dtype=torch.int32, device=dev))
    n_dec = args.decode_iters
    k_new = [synth.make_token(base_seed, s, B, H, D, pos=T + s, dtype=torch.bfloat16, device=dev) for s in range(2 * n_dec)]
    q_new = [synth.make_q(base_seed, s, B, HQ, D, dtype=torch.bfloat16, device=dev) for s in range(2 * n_dec)]
    attn_out = torch.empty((B, HQ, D), dtype=torch.bfloat16, device=dev)
    Ko = torch.empty((B, H, P, D), dtype=torch.bfloat16, device=dev)
    Vo = torch.empty_like(Ko)
    stream = torch.cuda.current_stream()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(record):
        """One pass of the hot path. `record`: dict of lists of (start, stop) event pairs, or None."""
        def timed(key, fn):
            if record is None:
                fn()
                return
            a, b = ev(), ev()
            a.record(stream); fn(); b.record(stream)
            record.setdefault(key, []).append((a, b))
        for l in range(NL):
            timed("prefill", lambda: ctx.compress_prefill(l, Ks[l], Vs[l], cKs[l], cVs[l], tls[l]))
        for s in range(n_dec):
            for l in range(NL):
                timed("append", lambda: ctx.append(l, k_new[s][0], k_new[s][1], cKs[l], cVs[l], tls[l]))
                timed("attn", lambda: ctx.decode_attn(l, q_new[s], cKs[l], cVs[l], tls[l], attn_out))
        for s in range(n_dec, 2 * n_dec):
            for l in range(NL):
                timed("append_attn", lambda: ctx.append_decode_attn(l, k_new[s][0], k_new[s][1], q_new[s], cKs[l], cVs[l],
                                                                    tls[l], attn_out))
        for l in range(NL):
            timed("reconstruct", lambda: ctx.reconstruct(l, cKs[l], cVs[l], tls[l], P, Ko, Vo))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local)
    for i in range(args.warmup):
        if i == args.warmup - 1 and rank == 0:
            sampler.start()          # nvidia-smi needs a moment to come up: start it one warm-up step early
        step(None)
    barrier()
    launches0 = ctx.launch_count()
    rec = {}
    t_start, t_stop = ev(), ev()
    barrier()
    t_start.record(stream)
    for _ in range(args.steps):
        step(rec)
    t_stop.record(stream)
    barrier()
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if ctx.device_status() != 0:
        raise RuntimeError("a kernel reported a device-side timeout; the numbers are invalid")

    def total_ms(key):
        return sum(a.elapsed_time(b) for a, b in rec[key])

    phase_ms = {k: total_ms(k) / args.steps for k in rec}
    step_ms = t_start.elapsed_time(t_stop) / args.steps
    prefill_ms = phase_ms["prefill"]

    prefill_ms, step_ms = max_over_ranks([prefill_ms, step_ms], dev)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        hK = [torch.empty(Ks[0].shape, dtype=torch.bfloat16).pin_memory() for _ in range(NL)]
        hV = [torch.empty(Vs[0].shape, dtype=torch.bfloat16).pin_memory() for _ in range(NL)]
        hcK = [torch.empty(cKs[l].shape, dtype=torch.float32).pin_memory() for l in range(NL)]
        hcV = [torch.empty(cVs[l].shape, dtype=torch.float32).pin_memory() for l in range(NL)]
        for l in range(NL):
            hK[l].copy_(Ks[l]); hV[l].copy_(Vs[l])
        torch.cuda.synchronize()
        copy_in, copy_out = torch.cuda.Stream(), torch.cuda.Stream()
        sK = [torch.empty_like(Ks[0]) for _ in range(2)]
        sV = [torch.empty_like(Vs[0]) for _ in range(2)]

        def e2e_step():
            in_done = [None, None]
            slot_free = [None, None]
            for l in range(NL):
                s = l & 1
                with torch.cuda.stream(copy_in):
                    if slot_free[s] is not None:
                        copy_in.wait_event(slot_free[s])
                    sK[s].copy_(hK[l], non_blocking=True)
                    sV[s].copy_(hV[l], non_blocking=True)
                    in_done[s] = copy_in.record_event()
                stream.wait_event(in_done[s])
                ctx.compress_prefill(l, sK[s], sV[s], cKs[l], cVs[l], tls[l])
                done = stream.record_event()
                slot_free[s] = done
                with torch.cuda.stream(copy_out):
                    copy_out.wait_event(done)
                    hcK[l].copy_(cKs[l], non_blocking=True)
                    hcV[l].copy_(cVs[l], non_blocking=True)
            stream.wait_stream(copy_out)

        h2d = sum(t.numel() * 2 for t in hK) + sum(t.numel() * 2 for t in hV)
        d2h = sum(t.numel() * 4 for t in hcK) + sum(t.numel() * 4 for t in hcV)
        e2e_step()
        barrier()
        k_e2e = max(1, min(args.steps, 3))
        t0 = time.perf_counter()
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(k_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        wall_ms = (time.perf_counter() - t0) * 1e3 / k_e2e
        e2e_ms = max(a.elapsed_time(b) / k_e2e, wall_ms if world == 1 else 0.0)
        e2e_ms = max_over_ranks([e2e_ms], dev)[0]
        e2e = {"value": whole_job_value(B * T, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
               "what": "phase A through the C ABI with pinned host K/V in and host coefficient planes out"}
        del hK, hV, hcK, hcV

    # ---- the same prefill through the FFT-shaped path (comparison; not part of `value`)
    prefill_fft = None
    if not args.no_prefill_fft:
        fctx = binding.Context(n_layers=NL, n_kv_heads=H, n_q_heads=HQ, n_dft=P, max_batch=B, kv_dtype=binding.BF16,
                               prefill_mode=binding.PREFILL_FFT)
        for l in range(NL):
            fctx.plan(l, binding.mask_mixed(P, M, l, base_seed))

        def fft_prefill():
            for l in range(NL):
                fctx.compress_prefill(l, Ks[l], Vs[l], cKs[l], cVs[l], tls[l])
        fft_prefill()
        barrier()
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(args.steps):
            fft_prefill()
        b.record(stream)
        barrier()
        f_ms = a.elapsed_time(b) / args.steps
        f_ms = max_over_ranks([f_ms], dev)[0]
        n_cols = 2 * B * H * D                                           # channels of K and V
        lgN = (P // 2).bit_length() - 1
        flop = 5.0 * (P // 2) * lgN * n_cols                             # 5 N log2 N per complex length-N FFT
        f_bytes = 2 * B * H * T * D * 2 + 2 * B * H * 2 * M * D * 4      # K/V in (bf16) + planes out (float32)
        peak_alu = 148 * 128 * 2 * 1.965e9 / 1e12                        # float32 FMA lanes x 2 x max SM clock
        prefill_fft = {"value": whole_job_value(B * T, world, f_ms), "unit": UNIT, "ms_per_layer": f_ms / NL,
                       "speedup_vs_value_path": prefill_ms / f_ms, "precision": "float32 (rel. error ~1e-6)",
                       "roofline": {"bound": "alu", "achieved": flop / (f_ms / NL * 1e-3) / 1e12, "peak": peak_alu,
                                    "unit": "TFLOP/s", "frac": flop / (f_ms / NL * 1e-3) / 1e12 / peak_alu,
                                    "flop_per_layer": flop, "flop_model": "5 N log2 N per channel, N = P/2",
                                    "hbm_gbs": f_bytes / (f_ms / NL * 1e-3) / 1e9, "hbm_frac": f_bytes / (f_ms / NL * 1e-3) / 1e9 / peaks["hbm"],
                                    "bytes_per_layer": f_bytes}}
        if fctx.device_status() != 0:
            raise RuntimeError("a kernel reported a device-side timeout; the numbers are invalid")
        fctx.close()

    # ---- decode at the workloads that define it (streaming decode, long context)
    decode_sections = []
    if not args.no_decode_configs and not args.layers:
        del Ks, Vs, cKs, cVs, Ko, Vo
        ctx.close()
        torch.cuda.empty_cache()
        for DW in DECODE_WORKLOADS:
            decode_sections.append(decode_section(torch, binding, synth, dev, DW, peaks, args.decode_config_iters))
    config0 = None
    if not args.no_decode_configs and not args.layers:
        config0 = config0_section(torch, binding, synth, dev)
    sweep = None
    if not args.no_sweep and not args.no_decode_configs and not args.layers:
        cells = sweep_cells()
        if args.sweep_cells:
            cells = cells[:args.sweep_cells]
        sweep = sweep_section(torch, binding, synth, dev, peaks, cells)
    barrier()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (prefill contraction), per launch (= one layer, K and V)
    n_c = B * H * D
    flop_per_launch = 2.0 * (2 * M) * T * n_c * 2            # 2*(2M)*T*N_c per tensor, K and V
    prefill_launch_ms = total_ms("prefill") / len(rec["prefill"])
    achieved_tf = flop_per_launch / (prefill_launch_ms * 1e-3) / 1e12
    mode = "simt-f32" if args.prefill_mode == binding.PREFILL_SIMT else "tcgen05-bf16"
    traffic, traffic_source = None, "no profiler capture for this mode"
    if mode == "tcgen05-bf16" and (args.twiddle_terms or 1) == 1:
        traffic, traffic_source = prefill_kernel_traffic()
    if mode == "tcgen05-bf16":
        peak_tf, bound = peaks["bf16_sustained"], "tensor"
    else:
        # float32 FMA pipe: 148 SMs x 128 lanes x 2 FLOP x 1.965 GHz
        peak_tf, bound = 148 * 128 * 2 * 1.965e9 / 1e12, "alu"
    roofline = {"kernel": "prefill transform (" + mode + ")", "bound": bound, "achieved": achieved_tf,
                "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved_tf / peak_tf, "frac_of_nominal_2250": (achieved_tf / 2250.0) if bound == "tensor" else None,
                "traffic": traffic, "traffic_source": traffic_source,
                "peak_source": peaks["source"] + (" bf16 sustained" if bound == "tensor" else " (derived f32 FMA peak)"),
                "flop_per_launch": flop_per_launch, "launch_ms": prefill_launch_ms,
                "mma_passes": (args.twiddle_terms if args.twiddle_terms else 1) if bound == "tensor" else None}

    coef_bytes = 2 * B * H * 2 * M * D * 4                     # K and V planes of one layer
    append_ms = total_ms("append") / len(rec["append"])
    attn_ms = total_ms("attn") / len(rec["attn"])
    recon_ms = total_ms("reconstruct") / len(rec["reconstruct"])
    fused_ms = total_ms("append_attn") / len(rec["append_attn"])
    decode = {
        "decode_us_per_layer_step": fused_ms * 1e3,
        "decode_us_per_layer_step_two_calls": (append_ms + attn_ms) * 1e3,
        "append_decode_attn": {"us": fused_ms * 1e3, "bytes": 2 * coef_bytes, "bound": "hbm",
                               "achieved": 2 * coef_bytes / (fused_ms * 1e-3) / 1e9, "peak": peaks["hbm"], "unit": "GB/s",
                               "frac": 2 * coef_bytes / (fused_ms * 1e-3) / 1e9 / peaks["hbm"],
                               "what": "fused call: planes read once and written once per step"},
        "append": {"us": append_ms * 1e3, "bytes": 2 * coef_bytes, "bound": "hbm",
                   "achieved": 2 * coef_bytes / (append_ms * 1e-3) / 1e9, "peak": peaks["hbm"], "unit": "GB/s",
                   "frac": 2 * coef_bytes / (append_ms * 1e-3) / 1e9 / peaks["hbm"]},
        "decode_attn": {"us": attn_ms * 1e3, "bytes": coef_bytes, "bound": "hbm",
                        "achieved": coef_bytes / (attn_ms * 1e-3) / 1e9, "peak": peaks["hbm"], "unit": "GB/s",
                        "frac": coef_bytes / (attn_ms * 1e-3) / 1e9 / peaks["hbm"]},
        "reconstruct": {"us": recon_ms * 1e3, "bytes": coef_bytes + 2 * B * H * P * D * 2, "bound": "hbm",
                        "achieved": (coef_bytes + 2 * B * H * P * D * 2) / (recon_ms * 1e-3) / 1e9, "peak": peaks["hbm"],
                        "unit": "GB/s", "frac": (coef_bytes + 2 * B * H * P * D * 2) / (recon_ms * 1e-3) / 1e9 / peaks["hbm"],
                        "alu": recon_alu_roofline(P, 2 * B * H * D, recon_ms * 1e-3),
                        "what": "FFT-shaped (float32 FFT per channel); bytes = planes in + bf16 rows out",
                        "dense_equivalent_tflops": 2.0 * P * (2 * M) * n_c * 2 / (recon_ms * 1e-3) / 1e12},
        "decode_iters": n_dec,
    }

    decode["what"] = "configs[1] shape (batch 1), calls launched eagerly with events around each"
    if decode_sections:
        decode["configs"] = decode_sections
        # the headline decode number is the streaming-decode workload's
        decode["decode_us_per_layer_step_configs1_shape"] = decode["decode_us_per_layer_step"]
        decode["decode_us_per_layer_step"] = decode_sections[0]["decode_us_per_layer_step"]
    line = {"metric": METRIC, "value": whole_job_value(B * T, world, prefill_ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(W, mode, args.twiddle_terms or 1),
            "phase_ms": phase_ms, "prefill_ms": prefill_ms,
            "roofline": roofline, "prefill_fft": prefill_fft, "decode": decode, "e2e": e2e, "gpu_launches": launches, "clocks": clocks}
    line["config0"] = config0
    line["sweep"] = sweep
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline()
    # compact last key, so that a truncated record of the line still carries every headline figure:
    # [us per layer-step, fraction of the measured HBM peak] per call and workload; prefill [TFLOP/s, fraction of
    # the measured sustained bf16 peak]
    def pair(d):
        return [round(d["us"], 1), round(d["frac"], 3)]
    summary = {"unit": "[us/layer/step, frac of measured HBM peak]; prefill: [TFLOP/s, frac of measured sustained bf16 peak]",
               "cfg1": {"prefill": [round(achieved_tf, 1), round(achieved_tf / peak_tf, 3)], "append": pair(decode["append"]),
                        "attn": pair(decode["decode_attn"]), "fused": pair(decode["append_decode_attn"]),
                        "recon": pair(decode["reconstruct"])}}
    for key, sec in zip(("cfg2", "cfg3", "cfg4cell"), decode_sections):
        summary[key] = {"prefill": [round(sec["prefill"]["achieved"], 1), round(sec["prefill"]["frac"], 3)],
                        "append": pair(sec["append"]), "attn": pair(sec["decode_attn"]), "fused": pair(sec["append_decode_attn"]),
                        "win": pair(sec["step_windowed"]), "defer": pair(sec["step_windowed_deferred"])}
        if "reconstruct" in sec:
            summary[key]["recon"] = pair(sec["reconstruct"])
    if config0 is not None:
        summary["cfg0"] = {"prefill_us": round(config0["prefill_us"], 1), "append_us": round(config0["append_us_per_step"], 2),
                           "recon_us": round(config0["reconstruct_us"], 1)}
    line["decode_summary"] = summary
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--decode-iters", type=int, default=2)
    ap.add_argument("--prefill-mode", type=int, default=0, help="0 auto, 1 float32 SIMT, 2 tcgen05")
    ap.add_argument("--twiddle-terms", type=int, default=0, help="tcgen05 prefill: 1 or 2 bf16 terms per twiddle")
    ap.add_argument("--layers", type=int, default=0,
                    help="run only the first N layers of the workload (small case for profiler captures; "
                         "a bench value must use the default = all layers)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-prefill-fft", action="store_true", help="skip the FFT-shaped prefill comparison")
    ap.add_argument("--no-decode-configs", action="store_true",
                    help="skip the decode sections at the configs[2] and configs[3] shapes")
    ap.add_argument("--decode-config-iters", type=int, default=10)
    ap.add_argument("--only-decode-config", type=int, default=0, choices=[0, 2, 3, 4],
                    help="profiling case: run only the decode section of configs[2] or configs[3] (eager launches; "
                         "combine with --layers and --decode-config-iters 1)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the configs[4] retention / batch sweep")
    ap.add_argument("--sweep-cells", type=int, default=0, help="run only the first N cells of the sweep")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
