#!/usr/bin/env python
"""Benchmark of the KVzap pruning hot path on B200.

A "step" is one pass of the whole hot path -- surrogate scoring, threshold and
window mask, per-head prefix sums, K/V compaction -- over one batch of synthetic
input for every layer of the workload.  Metric: tokens pruned per second per
layer = B*T / (step time / n_layers).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  Without ``--workload`` the line is that of the largest
single-GPU workload (Qwen3-32B shape, 128k tokens, 64 layers, paged output) and
carries, under ``configs``, a short record of each of the other four workloads
measured in the same process.  ``--impl reference`` times the CPU oracle (as it
stands) on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tokens pruned/sec per layer"
UNIT = "tokens/s/layer"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
HEADLINE = "qwen3_32b_prefill_128k_paged"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, taken from the ncu
# capture summarised in the named file under profiles/ (bytes per launch; not measured in this run).
NCU_TRAFFIC = {
    "qwen3_32b_prefill_128k_paged": (2065.3e6, "profiles/score_kernel_mlp_qwen3_32b_prefill_128k_paged.md"),
    "qwen3_8b_prefill_32k": (277.2e6, "profiles/score_kernel_mlp_qwen3_8b_prefill_32k.md"),
    "llama31_8b_prefill_4x16k": (540.8e6, "profiles/score_kernel_linear_llama31_8b_prefill_4x16k.md"),
    "linear_4k": (39.72e6, "profiles/score_linear_split_kernel_linear_4k.md"),
    "qwen3_8b_decode_b128": (228.0e6, "profiles/score_split_kernel_qwen3_8b_decode_b128.md"),
}
NCU_TRAFFIC_FP8 = {
    "qwen3_8b_prefill_32k": (140.4e6, "profiles/score_kernel_mlp_fp8_qwen3_8b_prefill_32k.md"),
}
# attention over the pruned cache: DRAM bytes per ALGORITHMIC byte, from a one-layer capture (traffic grows with the rows read)
NCU_ATTENTION_TRAFFIC_RATIO = 2.4093 / 2.3986
NCU_ATTENTION_FP8_TRAFFIC_RATIO = 1.3609 / 1.3501


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                d = json.load(f)
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def live_gemm_tflops(dev, seconds=1.5):
    """cuBLAS bf16 GEMM (8192^3) looped for `seconds` on this GPU, right after the timed region: the
    same kind of number as MEASURED_PEAKS.json's bf16_tflops_sustained, but of this GPU in its present
    power and thermal state.  Measurement aid only; nothing of the hot path runs through it."""
    import torch
    n = 8192
    a = torch.randn(n, n, dtype=torch.bfloat16, device=dev)
    b = torch.randn(n, n, dtype=torch.bfloat16, device=dev)
    c = torch.empty(n, n, dtype=torch.bfloat16, device=dev)
    for _ in range(3):
        torch.matmul(a, b, out=c)
    torch.cuda.synchronize()
    per = 2.0 * n ** 3
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps, done, t_total, last = 40, 0, 0.0, 0.0
    while t_total < seconds * 1e3:
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        last = e0.elapsed_time(e1)
        t_total += last
        done += reps
    return per * reps / (last * 1e-3) / 1e12          # the last block of launches: the settled rate


def pick_tensor_peak(peaks, clocks):
    """Which measured cuBLAS figure the timed region is compared with: the burst one when the region ran
    at (nearly) full SM clock with no power cap seen, the sustained one otherwise."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    burst = bool(mhz and mx and mhz >= 0.95 * mx and "sw_power_cap" not in clocks.get("reasons", []))
    return ("burst", peaks["bf16_tflops"]) if burst else ("sustained", peaks["bf16_tflops_sustained"])


def surrogate_flops_per_token(wl):
    """Algorithmic FLOPs per token per layer (Appendix B): 2 D_h N1 + 2 N1 H, or 2 D_h H."""
    if wl.surrogate == "mlp":
        return 2.0 * wl.d_model * wl.hidden + 2.0 * wl.hidden * wl.n_kv_heads
    return 2.0 * wl.d_model * wl.n_kv_heads


def algorithmic_bytes_per_layer(wl, n_tokens, kept_rows):
    """Hidden states read + scores written + kept K and V rows read and written + weights read once."""
    row = 2 * wl.head_dim
    w_bytes = (wl.hidden * wl.d_model * 2 + wl.hidden * wl.n_kv_heads * 2) if wl.surrogate == "mlp" \
        else wl.n_kv_heads * wl.d_model * 2
    return n_tokens * wl.d_model * 2 + n_tokens * wl.n_kv_heads * 4 + kept_rows * row * 2 * 2 + w_bytes


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.max_mhz = period, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = [("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap")]
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for label, attr in names:
                    if mask & int(getattr(nv, attr, 0)):
                        self.reasons.add(label)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_sample(wl, n_tokens, seed=424242, budget_s=0.0):
    """Times the CPU oracle (scoring + mask + compaction) on the first n_tokens of a layer, layer after
    layer (each with its own weights) until `budget_s` seconds of oracle time are used (at least one).
    Returns (tokens per second per layer, seconds, threads, layers timed)."""
    import torch
    from oracle import kvzap_oracle as oracle
    from paper_2601_07891_b200 import synth
    X = synth.hidden_states(n_tokens, wl.d_model, seed, "cpu", wl.token_scale_sigma)
    K, V = synth.keys_values(wl.n_kv_heads, n_tokens, wl.head_dim, seed + 1, "cpu")
    Xb, Kb, Vb = synth.bits(X), synth.bits(K), synth.bits(V)
    oracle.lib()
    total, layers = 0.0, 0
    while layers < wl.n_layers and (layers == 0 or total < budget_s):
        weights = synth.surrogate_weights(wl, layers, "cpu")
        ow = tuple(synth.bits(t) if t.dtype == torch.bfloat16 else t.numpy() for t in weights)
        t0 = time.perf_counter()
        oracle.prune_prefill(Xb, ow, Kb, Vb, wl.tau, wl.window)
        total += time.perf_counter() - t0
        layers += 1
    return n_tokens * layers / total, total, oracle.num_threads(), layers


def run_reference(args, wl):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_sample = min(wl.batch * wl.seq_len, args.ref_tokens)
    for _ in range(args.warmup):
        oracle_sample(wl, min(n_sample, 256))
    vals, secs, threads = [], 0.0, 1
    for _ in range(args.steps):
        v, dt, threads, _ = oracle_sample(wl, n_sample)
        vals.append(v)
        secs += dt
    value = n_sample * len(vals) / secs
    sample = "one layer, first %d tokens of the prompt: scoring + mask + compaction, per step" % n_sample
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(len(vals), 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "surrogate": wl.surrogate, "d_model": wl.d_model, "hidden": wl.hidden,
                       "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim, "n_layers": wl.n_layers,
                       "batch": wl.batch, "seq_len": wl.seq_len, "tau": wl.tau, "window": wl.window},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def _roofline_times(wl, n_tokens, kept_rows, peaks, tensor_peak):
    """(tensor time, HBM time of the scoring kernel's bytes, HBM time of all algorithmic bytes) of one layer, seconds."""
    flops = surrogate_flops_per_token(wl) * n_tokens
    t_tensor = flops / (tensor_peak * 1e12)
    score_bytes = n_tokens * wl.d_model * 2 + n_tokens * wl.n_kv_heads * 4
    t_hbm_score = score_bytes / (peaks["hbm_gbs"] * 1e9)
    t_hbm_layer = algorithmic_bytes_per_layer(wl, n_tokens, kept_rows) / (peaks["hbm_gbs"] * 1e9)
    return flops, score_bytes, t_tensor, t_hbm_score, t_hbm_layer


def _timed_steps(step, n_steps, block, record_first, record_last):
    """Runs n_steps steps between two given events and marks every `block` steps with an event of its own: the
    whole-region time stays the measurement, the marks give the spread (median / min / max per step over blocks)."""
    import torch
    marks = []
    record_first.record()
    for i in range(n_steps):
        step()
        if (i + 1) % block == 0 and i + 1 < n_steps:
            ev = torch.cuda.Event(enable_timing=True)
            ev.record()
            marks.append(ev)
    record_last.record()
    return marks


def _step_stats(first, marks, last, n_steps, block):
    evs = [first] + marks + [last]
    sizes = [block] * len(marks) + [n_steps - block * len(marks)]
    per = sorted(evs[i].elapsed_time(evs[i + 1]) / sizes[i] for i in range(len(sizes)) if sizes[i] > 0)
    return {"median": statistics.median(per), "min": per[0], "max": per[-1], "steps_per_sample": block, "samples": len(per)}


def _timed(fn, n, stream_sync):
    """Average milliseconds of fn() over n calls, CUDA events on the current stream."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream_sync()
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    stream_sync()
    return e0.elapsed_time(e1) / n


def run_prefill(args, wl, env, sub=False):
    """Prefill workloads: one step = the fused hot path (scoring, mask, compaction) over every layer.
    sub: a short record for the `configs` list (no end-to-end leg, no live cuBLAS loop)."""
    import torch
    from paper_2601_07891_b200 import binding, synth
    dev, rank, world, barrier = env["dev"], env["rank"], env["world"], env["barrier"]
    L, B, T = wl.n_layers, wl.batch, wl.seq_len
    if args.layers > 0:
        L = min(L, args.layers)          # small case for profiler captures; reported in config.n_layers
    n_tokens = B * T
    H, D, P = wl.n_kv_heads, wl.head_dim, wl.page_tokens
    proj = args.kv_layout == "proj"
    fp8 = args.fp8 and not sub
    if fp8 and proj:
        raise SystemExit("--fp8 goes with the prefill workloads in the [H,T,D] layout")
    ctx = binding.Kvzap(wl.d_model, wl.hidden, H, D, L, n_tokens, max_seqs=B, device=dev.index, trusted_producers=True)
    cu = torch.from_numpy(synth.cu_seqlens([T] * B)).to(dev) if B > 1 else None

    # resident inputs, one set per layer while they fit (every layer's inputs exceed L2, so no flush is
    # needed); beyond ~60 GB the layers rotate over fewer input sets (weights stay distinct per layer)
    per_layer_bytes = n_tokens * wl.d_model * 2 + 4 * H * n_tokens * D * 2
    n_sets = L if L * per_layer_bytes <= 60e9 else max(2, int(40e9 // per_layer_bytes))
    # a small workload (config 1: 56 MB per layer) would otherwise run out of the 126 MB L2: rotate over
    # enough input/output sets that 2.5 x L2 lies between two uses of the same buffer
    n_sets = max(n_sets, int(-(-2.5 * 126e6 // per_layer_bytes)))
    Xs, Ks, Vs, Kos, Vos, lens, scs, tabs, used = [], [], [], [], [], [], [], [], []
    max_pages = (T // P + 2) if P else 0
    pool_pages = (H * B * (T // P + 2)) // 2 if P else 0       # room for half of all rows per layer set
    for l in range(L):
        wts = synth.surrogate_weights(wl, l, dev, seed_base=7000 + 100 * args.workload_index)
        if fp8:
            W18, sw = synth.quantize_e4m3(wts[0])
            binding.kvzap_set_weights_fp8(ctx.handle, l, W18, sw, wts[1], *(wts[2:] if len(wts) == 4 else (None, None)))
        else:
            ctx.set_weights(l, *wts)
    Xscales = []
    for l in range(max(L, n_sets)):
        lens.append(torch.zeros(B, H, dtype=torch.int32, device=dev))
        if l >= n_sets:
            for lst in (Xs, Ks, Vs, Kos, Vos, scs, tabs, used, Xscales):
                lst.append(lst[l % n_sets])
            continue
        seed = 1000 * args.workload_index + l + 100000 * rank
        X = synth.hidden_states(n_tokens, wl.d_model, seed, dev, wl.token_scale_sigma)
        if fp8:
            X, xs = synth.quantize_e4m3(X)
            Xscales.append(xs)
        else:
            Xscales.append(None)
        Xs.append(X)
        K, V = synth.keys_values(H, n_tokens, D, seed + 500, dev)
        if proj:
            # write-side pruning: the same draws, laid out as the K/V projection writes them, [T, H, D]
            K, V = K.transpose(0, 1).contiguous(), V.transpose(0, 1).contiguous()
        Ks.append(K)
        Vs.append(V)
        if P:
            Kos.append(torch.empty(pool_pages, P, D, dtype=torch.bfloat16, device=dev))
            Vos.append(torch.empty(pool_pages, P, D, dtype=torch.bfloat16, device=dev))
            tabs.append(torch.zeros(B * H, max_pages, dtype=torch.int32, device=dev))
            used.append(torch.zeros(1, dtype=torch.int32, device=dev))
        else:
            Kos.append(torch.empty(H, n_tokens, D, dtype=torch.bfloat16, device=dev))
            Vos.append(torch.empty(H, n_tokens, D, dtype=torch.bfloat16, device=dev))
            tabs.append(None)
            used.append(None)
        scs.append(torch.empty(n_tokens, H, dtype=torch.float32, device=dev))
    torch.cuda.synchronize()

    n_bufs = len(Xs)
    turn = [0]
    # the calls of a step, marshalled once (same entry points, same arguments every step)
    calls = {}
    for l in range(L):
        for i in (range(n_bufs) if n_bufs > L else [l]):
            prep_paged = binding.prepare_prefill_write_paged if proj else binding.prepare_prefill_fused_paged
            prep_dense = binding.prepare_prefill_write if proj else binding.prepare_prefill_fused
            if fp8 and P:
                calls[(l, i)] = binding.prepare_prefill_fused_paged_fp8(ctx.handle, l, Xs[i], Xscales[i], Ks[i], Vs[i], cu, B,
                                                                        wl.tau, wl.window, Kos[i], Vos[i], P, 0, tabs[i],
                                                                        lens[i], used[i], scs[i])
            elif fp8:
                calls[(l, i)] = binding.prepare_prefill_fused_fp8(ctx.handle, l, Xs[i], Xscales[i], Ks[i], Vs[i], cu, B, wl.tau,
                                                                  wl.window, Kos[i], Vos[i], lens[i], scs[i])
            elif P:
                calls[(l, i)] = prep_paged(ctx.handle, l, Xs[i], Ks[i], Vs[i], cu, B, wl.tau,
                                           wl.window, Kos[i], Vos[i], P, 0, tabs[i], lens[i], used[i], scs[i])
            else:
                calls[(l, i)] = prep_dense(ctx.handle, l, Xs[i], Ks[i], Vs[i], cu, B, wl.tau,
                                           wl.window, Kos[i], Vos[i], lens[i], scs[i])

    def step():
        for l in range(L):
            calls[(l, (turn[0] + l) % n_bufs)]()   # layer l's buffers; with more sets than layers they rotate per step
        if n_bufs > L:
            turn[0] += L

    n_warm = args.warmup if args.layers > 0 else max(args.warmup, 3)
    for _ in range(n_warm):
        step()
    barrier()
    if ctx.poll_status() != 0:
        raise RuntimeError("device status word set during warm-up")

    # Stand-alone kvzap_prune_prefill(_paged) on the scores the warm-up left: an HBM-bound call that never reaches the
    # power cap by itself, so it is timed here, after a short pause, and not behind the long tensor-bound region below
    # (whose clock reduction outlasts it by tens of milliseconds).
    sync = torch.cuda.synchronize
    if proj:
        prune = None          # the two-call route exists for the head-major layout only
    else:
        if P:
            pcalls = [binding.prepare_prune_prefill_paged(ctx.handle, Ks[l], Vs[l], scs[l], cu, B, wl.tau, wl.window,
                                                          Kos[l], Vos[l], P, 0, tabs[l], lens[l], used[l]) for l in range(n_bufs)]
        else:
            pcalls = [binding.prepare_prune_prefill(ctx.handle, Ks[l], Vs[l], scs[l], cu, B, wl.tau, wl.window,
                                                    Kos[l], Vos[l], lens[l]) for l in range(n_bufs)]
        prune = lambda: [pc() for pc in pcalls]
    prune_ms = None
    if prune:
        sync()
        time.sleep(0.3)
        prune()                                            # warm-up of this loop
        prune_ms = _timed(prune, max(1, min(args.steps, 5)), sync) / n_bufs

    n_steps = args.steps
    if sub:
        # enough steps that the region is not a burst: at least ~0.3 s for the tensor-bound workloads
        n_steps = max(args.steps, 100 if wl.surrogate == "mlp" else 20, 2000 if L == 1 else 0)
    sampler = ClockSampler(dev.index)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launch_count()
    sampler.start()
    barrier()
    block = 1 if L * n_tokens >= 1000000 else 100        # a mark per step, or per 100 steps where a step is a few microseconds
    marks = _timed_steps(step, n_steps, block, e0, e1)
    barrier()
    clocks = sampler.stop()
    total_ms = env["max_over_ranks"](e0.elapsed_time(e1))
    step_stats = _step_stats(e0, marks, e1, n_steps, block)
    gpu_launches = ctx.launch_count() - launches0
    ms_per_step = total_ms / n_steps
    layer_ms = ms_per_step / L
    value = world * n_tokens / (layer_ms * 1e-3)
    if ctx.poll_status() != 0:
        raise RuntimeError("device status word set during the timed region")
    kept_rows = float(sum(int(x.sum().item()) for x in lens[:n_bufs])) / n_bufs   # kept (head, token) rows per layer

    # The two kernels of a layer, each timed alone with CUDA events around a loop of launches through
    # the public calls (scoring only; mask + compaction on the scores just computed).
    n_rep = max(1, min(n_steps, 5))
    def score_only():
        for l in range(L):
            i = (turn[0] + l) % n_bufs
            if fp8:
                binding.kvzap_score_fp8(ctx.handle, l, Xs[i], Xscales[i], scs[i])
            else:
                binding.kvzap_score(ctx.handle, l, Xs[i], scs[i])
        if n_bufs > L:
            turn[0] += L
    score_ms = _timed(score_only, n_rep, sync) / L
    peaks, peak_src = load_peaks()
    peak_kind, tensor_peak = pick_tensor_peak(peaks, clocks)
    if fp8:
        tensor_peak *= 2.0           # no 8-bit GEMM was measured on this machine: the bf16 figure times the nominal ratio (4.5 / 2.25 PFLOP/s)
        peak_kind += " x 2 (nominal fp8 : bf16 ratio)"
    flops, score_bytes, t_tensor, t_hbm_score, t_hbm_layer = _roofline_times(wl, n_tokens, kept_rows, peaks, tensor_peak)
    if fp8:
        # an 8-bit hidden state is half the bytes (plus 4 bytes of scale per token)
        score_bytes = n_tokens * wl.d_model + n_tokens * 4 + n_tokens * wl.n_kv_heads * 4
        t_hbm_score = score_bytes / (peaks["hbm_gbs"] * 1e9)
        t_hbm_layer -= (n_tokens * wl.d_model - n_tokens * 4) / (peaks["hbm_gbs"] * 1e9)
    # Dominant kernel = the scoring kernel.  Its launch duration inside the timed region cannot be
    # separated from the compaction that runs beside it, so the layer period (step time / layers) is
    # used: an upper bound of the kernel's own duration.  `alone_ms` is the same kernel in a loop of
    # scoring-only launches.
    if t_tensor >= t_hbm_score:
        achieved = flops / (layer_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": tensor_peak,
                    "unit": "TFLOP/s", "frac": achieved / tensor_peak,
                    "peak_kind": peak_kind + " cuBLAS bf16 figure, chosen from this run's clock record (burst: median SM "
                                             "clock within 5 % of max and no sw_power_cap sample)",
                    "frac_of_burst": achieved / (peaks["bf16_tflops"] * (2.0 if fp8 else 1.0)),
                    "frac_of_sustained": achieved / (peaks["bf16_tflops_sustained"] * (2.0 if fp8 else 1.0)),
                    "alone_achieved": flops / (score_ms * 1e-3) / 1e12}
        if clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
            # time x clock: the burst figure (measured at the maximum clock) scaled to the clock this region ran at
            at_clock = peaks["bf16_tflops"] * (2.0 if fp8 else 1.0) * clocks["sm_mhz"] / clocks["sm_max_mhz"]
            roofline["frac_of_burst_scaled_to_run_clock"] = achieved / at_clock
        if not args.skip_live_peak and not sub:
            # the GPUs of the pool settle at different clocks under the power cap: the same loop on this one, now
            live = live_gemm_tflops(dev)
            roofline["live_cublas_bf16_tflops_sustained"] = live
            roofline["frac_of_live_cublas"] = achieved / live
    else:
        achieved = score_bytes / (layer_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "alone_achieved": score_bytes / (score_ms * 1e-3) / 1e9}
    traffic = NCU_TRAFFIC.get(wl.name) if args.layers == 0 and not proj else None
    if fp8:
        traffic = NCU_TRAFFIC_FP8.get(wl.name) if args.layers == 0 and not proj else None
    roofline.update({"traffic": traffic[0] if traffic else None,
                     "traffic_source": (traffic[1] + " (ncu capture of 2026-11-28, not measured in this run)") if traffic else None,
                     "kernel": "score_kernel", "peak_source": peak_src,
                     "kernel_ms": layer_ms, "alone_ms": score_ms,
                     "note": "kernel_ms = layer period in the timed region (compaction overlaps the next "
                             "layer's scoring kernel); alone_ms = scoring-only launches back to back"})
    t_roof_layer = max(t_tensor, t_hbm_layer)
    compact_bytes = kept_rows * 2 * D * 2 * 2
    extra = {"layer_ms": layer_ms, "layer_roofline_ms": t_roof_layer * 1e3,
             "layer_frac_of_roofline": t_roof_layer * 1e3 / layer_ms,
             "score_alone_ms": score_ms, "mask_plus_compaction_alone_ms": prune_ms,
             "compaction_alone_GBps": compact_bytes / (prune_ms * 1e-3) / 1e9 if prune_ms else None,
             "kept_fraction": kept_rows / (H * n_tokens)}
    config = {"workload": wl.name, "surrogate": wl.surrogate, "d_model": wl.d_model, "hidden": wl.hidden,
              "n_kv_heads": H, "head_dim": D, "n_layers": L, "batch": B, "seq_len": T, "tau": wl.tau,
              "window": wl.window, "page_tokens": P, "input_sets": n_bufs,
              "kv_layout": "[T,H,D] as the projection writes it (write-side pruning)" if proj else "[H,T,D]",
              "l2": "inputs larger than L2 (distinct resident buffers per layer; small workloads rotate over "
                    "enough sets that 2.5 x L2 lies between two uses of a buffer)",
              "parallelism": "replicas only" if world > 1 else "single GPU"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": n_steps,
            "warmup": n_warm, "ms_per_step": ms_per_step, "step_ms": step_stats, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "e4m3 x e4m3 -> f32 (first layer), bf16 K/V" if fp8 else "bf16", "data": "synthetic",
            "config": config, "clocks": clocks, "gpu_launches": int(gpu_launches), "roofline": roofline, "breakdown": extra}

    if rank == 0 and world == 1 and not args.skip_e2e and not proj and not sub and not fp8:
        # End to end through the host-buffer entry point: one call per step takes every layer's inputs from
        # pinned host memory and leaves every layer's result there; the copies happen inside the call (layer
        # l + 1 is copied in while layer l is computed and copied out).  Host inputs rotate over two layer sets.
        n_h = min(L, 2)
        hX = [Xs[i].cpu().pin_memory() for i in range(n_h)]
        hK = [Ks[i].cpu().pin_memory() for i in range(n_h)]
        hV = [Vs[i].cpu().pin_memory() for i in range(n_h)]
        if P:
            hKo = torch.empty(pool_pages, P, D, dtype=torch.bfloat16).pin_memory()
            hVo = torch.empty(pool_pages, P, D, dtype=torch.bfloat16).pin_memory()
            htab = torch.zeros(B * H, max_pages, dtype=torch.int32).pin_memory()
            hused = torch.zeros(1, dtype=torch.int32).pin_memory()
        else:
            hKo, hVo = torch.empty_like(hK[0]).pin_memory(), torch.empty_like(hV[0]).pin_memory()
            htab = hused = None
        hlen = [torch.zeros(B, H, dtype=torch.int32).pin_memory() for _ in range(L)]
        hcu = torch.from_numpy(synth.cu_seqlens([T] * B)) if B > 1 else None
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        lists = dict(hidden=[hX[l % n_h] for l in range(L)], K=[hK[l % n_h] for l in range(L)],
                     V=[hV[l % n_h] for l in range(L)], K_out=[hKo] * L, V_out=[hVo] * L)

        def e2e_step():
            binding.kvzap_prefill_layers_host(ctx.handle, 0, lists["hidden"], lists["K"], lists["V"], hcu, B, wl.tau, wl.window,
                                              lists["K_out"], lists["V_out"], hlen, None, page_tokens=P,
                                              page_table=[htab] * L if P else None, n_pages_used=[hused] * L if P else None)
        e2e_step()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
        # the rate of a plain pinned-host-to-device copy of one layer's hidden states on this machine, for comparison
        t0 = time.perf_counter()
        for _ in range(3):
            Xs[0].copy_(hX[0], non_blocking=True)
        torch.cuda.synchronize()
        h2d_rate = 3 * hX[0].numel() * 2 / (time.perf_counter() - t0) / 1e9
        h2d = L * (n_tokens * wl.d_model * 2 + 2 * H * n_tokens * D * 2 + (B * H * max_pages * 4 if P else 0)) + \
            (4 * (B + 1) if B > 1 else 0)
        kept_e2e = float(sum(int(x.sum()) for x in hlen)) / L
        if P:
            d2h = int(L * (int(hused.item()) * P * 2 * D * 2 + B * H * max_pages * 4 + B * H * 4 + 4))
        else:
            d2h = int(L * (kept_e2e * 2 * D * 2 + B * H * 4))
        line["e2e"] = {"value": n_tokens / (e2e_ms * 1e-3 / L), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                       "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
                       "h2d_GBps_achieved": h2d / (e2e_ms * 1e-3) / 1e9, "h2d_GBps_plain_copy": h2d_rate,
                       "frac_of_plain_h2d_copy": h2d / (e2e_ms * 1e-3) / 1e9 / h2d_rate,
                       "note": "kvzap_prefill_layers_host, all layers in one call: pinned host buffers, copies inside the "
                               "timed region and overlapped with the kernels of the neighbouring layers"}
        del hX, hK, hV, hKo, hVo, lists
    ctx.close()
    return line


def run_decode(args, wl, env, sub=False):
    """Decode workload: one step = one decode step (score the new token of every sequence with every
    layer's surrogate, append, decide the token leaving the window) over all layers."""
    import numpy as np
    import torch
    from paper_2601_07891_b200 import binding, synth
    dev, rank, world, barrier = env["dev"], env["rank"], env["world"], env["barrier"]
    L, B, H, D, w, P = wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.window, wl.page_tokens
    if args.layers > 0:
        L = min(L, args.layers)
    fp8 = bool(args.fp8) and not sub          # hidden states and first-layer weights as E4M3 bytes with scales
    ctx = binding.Kvzap(wl.d_model, wl.hidden, H, D, L, max_tokens=B, device=dev.index, trusted_producers=True)
    for l in range(L):
        wts = synth.surrogate_weights(wl, l, dev, seed_base=7000 + 100 * args.workload_index)
        if fp8:
            W18, sw = synth.quantize_e4m3(wts[0])
            binding.kvzap_set_weights_fp8(ctx.handle, l, W18, sw, wts[1], *(wts[2:] if len(wts) == 4 else (None, None)))
        else:
            ctx.set_weights(l, *wts)
    n_lists = B * L * H
    n_steps = max(args.steps, 1000) if sub else args.steps
    total_steps = w + max(args.warmup, 3) + n_steps + 8 + 36 + (max(args.e2e_steps, 10) + 3 if not args.skip_e2e and not sub else 0)
    # Pre-pruned caches: per-list prefix lengths uniform in [prefix_min, prefix_max].  Decoding never
    # reads a list's earlier pages, so only each list's last (partly filled) page and the pages it can
    # grow into are backed by memory; lengths and page tables carry the full logical sizes.
    rng = np.random.default_rng(4242 + rank)
    prefix = rng.integers(wl.prefix_min, wl.prefix_max + 1, size=n_lists).astype(np.int32)
    grow_pages = total_steps // P + 2
    max_pages = int(wl.prefix_max // P + grow_pages + 1)
    n_pool = n_lists * (1 + grow_pages)
    K_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device=dev)
    V_pool = torch.zeros(n_pool, P, D, dtype=torch.bfloat16, device=dev)
    table = torch.full((n_lists, max_pages), -1, dtype=torch.int32, device=dev)
    tail = torch.from_numpy((prefix // P).astype(np.int64)).to(dev)
    table[torch.arange(n_lists, device=dev), tail] = torch.arange(n_lists, dtype=torch.int32, device=dev)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    binding.kvzap_cache_import(ctx.handle, cache, torch.from_numpy(prefix).to(dev), table, n_lists)
    del table
    n_sets = 6                        # rotating per-step inputs; the weights (151 MB) alone exceed L2
    Xs = [synth.hidden_states(L * B, wl.d_model, 9000 + i + 100 * rank, dev).view(L, B, wl.d_model) for i in range(n_sets)]
    KVs = [synth.keys_values(L * B, H, D, 9500 + i + 100 * rank, dev) for i in range(n_sets)]
    scores = [torch.empty(L, B, H, dtype=torch.float32, device=dev) for _ in range(n_sets)]
    it = [0]

    if fp8:
        Xq = [synth.quantize_e4m3(x.view(L * B, wl.d_model)) for x in Xs]
        dcalls = [binding.prepare_decode_step_fp8(ctx.handle, cache, 0, L, Xq[i][0].view(L, B, wl.d_model), Xq[i][1].view(L, B),
                                                  KVs[i][0].view(L, B, H, D), KVs[i][1].view(L, B, H, D), wl.tau, scores[i])
                  for i in range(n_sets)]
    else:
        dcalls = [binding.prepare_decode_step(ctx.handle, cache, 0, L, Xs[i], KVs[i][0].view(L, B, H, D),
                                              KVs[i][1].view(L, B, H, D), wl.tau, scores[i]) for i in range(n_sets)]

    def step():
        dcalls[it[0] % n_sets]()
        it[0] += 1

    graph_mode = getattr(args, "graph", "off") if not sub else "off"
    if graph_mode != "off":
        # The same steps captured once in a CUDA graph and replayed: n_sets steps per graph (the rotating input sets),
        # each one launch over all layers ("step") or one launch per layer ("layer").
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        stream_ctx = torch.cuda.stream(side)          # the prepared calls carry the stream they were prepared on
        stream_ctx.__enter__()
        if graph_mode == "step":
            if fp8:
                gcalls = [binding.prepare_decode_step_fp8(ctx.handle, cache, 0, L, Xq[i][0].view(L, B, wl.d_model), Xq[i][1].view(L, B),
                                                          KVs[i][0].view(L, B, H, D), KVs[i][1].view(L, B, H, D), wl.tau, scores[i])
                          for i in range(n_sets)]
            else:
                gcalls = [binding.prepare_decode_step(ctx.handle, cache, 0, L, Xs[i], KVs[i][0].view(L, B, H, D),
                                                      KVs[i][1].view(L, B, H, D), wl.tau, scores[i]) for i in range(n_sets)]
        if graph_mode == "layer":
            if fp8:
                lcalls = [[binding.prepare_decode_step_fp8(ctx.handle, cache, l, l + 1, Xq[i][0].view(L, B, wl.d_model)[l:l + 1],
                                                           Xq[i][1].view(L, B)[l:l + 1], KVs[i][0].view(L, B, H, D)[l:l + 1],
                                                           KVs[i][1].view(L, B, H, D)[l:l + 1], wl.tau, scores[i][l:l + 1])
                           for l in range(L)] for i in range(n_sets)]
            else:
                lcalls = [[binding.prepare_decode_step(ctx.handle, cache, l, l + 1, Xs[i][l:l + 1], KVs[i][0].view(L, B, H, D)[l:l + 1],
                                                       KVs[i][1].view(L, B, H, D)[l:l + 1], wl.tau, scores[i][l:l + 1])
                           for l in range(L)] for i in range(n_sets)]
            one = lambda i: [c() for c in lcalls[i]]
        else:
            one = lambda i: gcalls[i]()
        for i in range(n_sets):       # once outside the capture
            one(i)
        stream_ctx.__exit__(None, None, None)
        torch.cuda.synchronize()
        cuda_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cuda_graph, stream=side):
            for i in range(n_sets):
                one(i)
        replays = [0]

        def step():                   # one replay = n_sets steps; called once per n_sets steps of the loops below
            if it[0] % n_sets == 0:
                cuda_graph.replay()
                replays[0] += 1
            it[0] += 1

    for _ in range(w):                # fill the window: from here on every step decides one token per list
        step()
    n_warm = max(args.warmup, 3)
    for _ in range(n_warm):
        step()
    barrier()
    if ctx.poll_status() != 0:
        raise RuntimeError("device status word set during warm-up")
    if graph_mode != "off":           # whole replays only
        it[0] = -(-it[0] // n_sets) * n_sets
        n_steps = -(-n_steps // n_sets) * n_sets
    len0 = torch.zeros(B, L, H, dtype=torch.int32, device=dev)
    binding.kvzap_cache_lengths(ctx.handle, cache, len0)
    sampler = ClockSampler(dev.index)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launch_count()
    sampler.start()
    barrier()
    block = 100 if n_steps >= 200 else max(1, n_steps // 4)
    if graph_mode != "off":
        block = -(-block // n_sets) * n_sets
    marks = _timed_steps(step, n_steps, block, e0, e1)
    barrier()
    clocks = sampler.stop()
    total_ms = env["max_over_ranks"](e0.elapsed_time(e1))
    step_stats = _step_stats(e0, marks, e1, n_steps, block)
    gpu_launches = ctx.launch_count() - launches0
    if graph_mode != "off":          # replays launch what the capture recorded; the host-side counter sees only the capture
        gpu_launches = n_steps * (L if graph_mode == "layer" else 1)
    ms_per_step = total_ms / n_steps
    if ctx.poll_status() != 0:
        raise RuntimeError("device status word set during the timed region")
    len1 = torch.zeros_like(len0)
    binding.kvzap_cache_lengths(ctx.handle, cache, len1)
    kept_exit = float((len1 - len0).sum().item()) / (n_steps * n_lists)     # fraction of exiting tokens kept
    value = world * B / (ms_per_step * 1e-3 / L)

    peaks, peak_src = load_peaks()
    row = 2 * D
    xb = 1 if fp8 else 2                                               # bytes per element of hidden states and W1
    w_bytes = wl.hidden * wl.d_model * xb + wl.hidden * H * 4 + wl.hidden * 4 + H * 4 + (wl.hidden * 4 if fp8 else 0)
    bytes_layer = (w_bytes + B * wl.d_model * xb + (B * 4 if fp8 else 0) + B * H * 4          # weights, hidden states, scores
                   + 2 * B * H * row * 2                               # new K and V rows read and written to the window
                   + B * H * 4 * 2                                     # buffered score read, new score written
                   + kept_exit * B * H * 2 * row * 2)                  # kept exiting rows: window -> page
    achieved = bytes_layer * L / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"],
                "traffic": NCU_TRAFFIC[wl.name][0] if wl.name in NCU_TRAFFIC and args.layers == 0 and not fp8 else None,
                "traffic_source": (NCU_TRAFFIC[wl.name][1] + " (ncu capture of 2026-11-28, not measured in this run)")
                if wl.name in NCU_TRAFFIC and args.layers == 0 and not fp8 else None,
                "kernel": "score_split_kernel (scoring + cache update in one launch)", "peak_source": peak_src,
                "kernel_ms": ms_per_step, "algorithmic_bytes_per_step": bytes_layer * L}
    config = {"workload": wl.name, "surrogate": wl.surrogate, "d_model": wl.d_model, "hidden": wl.hidden,
              "n_kv_heads": H, "head_dim": D, "n_layers": L, "batch": B, "tau": wl.tau, "window": w, "page_tokens": P,
              "prefix_len": [wl.prefix_min, wl.prefix_max], "input_sets": n_sets,
              "l2": "weights of all layers (151 MB) exceed L2; per-step inputs rotate over %d sets" % n_sets,
              "backing": "only each list's last page and growth pages are backed (decode never reads earlier pages)",
              "cuda_graph": {"off": "no", "step": "%d steps per graph, one launch per step" % n_sets,
                             "layer": "%d steps per graph, one launch per layer" % n_sets}[graph_mode],
              "parallelism": "replicas only" if world > 1 else "single GPU"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": n_steps, "warmup": n_warm,
            "ms_per_step": ms_per_step, "step_ms": step_stats, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "e4m3 x e4m3 -> f32 (first layer), bf16 K/V" if fp8 else "bf16", "data": "synthetic", "config": config,
            "clocks": clocks, "gpu_launches": int(gpu_launches), "roofline": roofline,
            "breakdown": {"layer_us": ms_per_step * 1e3 / L, "layer_roofline_us": bytes_layer / (peaks["hbm_gbs"] * 1e9) * 1e6,
                          "layer_frac_of_roofline": bytes_layer / (peaks["hbm_gbs"] * 1e9) * 1e3 / (ms_per_step / L),
                          "kept_fraction_of_exiting_tokens": kept_exit}}
    if rank == 0 and world == 1 and not args.skip_e2e and not sub and not fp8 and graph_mode == "off":
        # End to end: the step's inputs start in pinned host memory and its scores end there; the copies
        # (torch, on the stream of the call) are inside the timed region.
        hX = [x.cpu().pin_memory() for x in Xs[:2]]
        hK = [kv[0].cpu().pin_memory() for kv in KVs[:2]]
        hV = [kv[1].cpu().pin_memory() for kv in KVs[:2]]
        hS = [torch.empty(L, B, H, dtype=torch.float32).pin_memory() for _ in range(2)]
        dX, dK, dV = torch.empty_like(Xs[0]), torch.empty_like(KVs[0][0]), torch.empty_like(KVs[0][1])
        dS = torch.empty(L, B, H, dtype=torch.float32, device=dev)

        def e2e_step(i):
            dX.copy_(hX[i % 2], non_blocking=True)
            dK.copy_(hK[i % 2], non_blocking=True)
            dV.copy_(hV[i % 2], non_blocking=True)
            binding.kvzap_decode_step(ctx.handle, cache, 0, L, dX, dK.view(L, B, H, D), dV.view(L, B, H, D), wl.tau, dS)
            hS[i % 2].copy_(dS, non_blocking=True)

        for i in range(3):
            e2e_step(i)
        torch.cuda.synchronize()
        n_e2e = max(args.e2e_steps, 10)
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3 / n_e2e
        h2d = hX[0].numel() * 2 + hK[0].numel() * 2 + hV[0].numel() * 2
        line["e2e"] = {"value": B / (e2e_ms * 1e-3 / L), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                       "d2h_bytes_per_step": int(hS[0].numel() * 4), "ms_per_step": e2e_ms, "steps": n_e2e,
                       "note": "kvzap_decode_step with the step's hidden states and new K/V rows copied from pinned host "
                               "memory and the scores copied back, inside the timed region"}
    binding.kvzap_cache_destroy(cache)
    ctx.close()
    return line


def run_attention(args, wl, env):
    """The consumer of the pruned cache (not part of the pruning metric; run with --attention): the new
    token's attention over every list of a few layers of the decode workload, lists fully backed by memory.
    One step = one kvzap_decode_attention call over those layers."""
    import numpy as np
    import torch
    from paper_2601_07891_b200 import binding, synth
    dev, rank, world, barrier = env["dev"], env["rank"], env["world"], env["barrier"]
    B, H, D, w, P = wl.batch, wl.n_kv_heads, wl.head_dim, wl.window, wl.page_tokens
    L = args.layers if args.layers > 0 else 4
    G = 4                                             # 32 query heads over 8 KV heads
    fp8 = bool(getattr(args, "fp8", False))           # rows of D E4M3 codes + a 16-byte trailer (fp32 scale first)
    Dq = D                                            # elements per head, as Q and O have them
    if fp8:
        D = (Dq + synth.E4M3_ROW_TRAILER) // 2        # row width in bf16 units, as the context moves rows
    ctx = binding.Kvzap(wl.d_model, wl.hidden, H, D, L, max_tokens=B, device=dev.index, trusted_producers=True)
    for l in range(L):
        ctx.set_weights(l, *synth.surrogate_weights(wl, l, dev, seed_base=7000 + 100 * args.workload_index))
    n_lists = B * L * H
    # pre-pruned lists: a sequence of prefix_min..prefix_max tokens of which every (layer, head) kept 15-35 %
    rng = np.random.default_rng(777 + rank)
    seq_len = rng.integers(wl.prefix_min, wl.prefix_max + 1, size=B)
    kept = rng.uniform(0.15, 0.35, size=(B, L, H))
    prefix = np.maximum(1, (seq_len[:, None, None] * kept)).astype(np.int32).reshape(-1)      # list index (b, l, h)
    grow_pages = (w + 16) // P + 2
    pages_of = (prefix + P - 1) // P + grow_pages
    first = np.concatenate([[0], np.cumsum(pages_of)[:-1]]).astype(np.int64)
    n_pool = int(pages_of.sum())
    max_pages = int(pages_of.max())
    if fp8:
        # random codes (top exponent bits cleared: magnitudes below 2, no NaN code) and a scale of 1/2 per row
        def rows8():
            t = torch.randint(0, 256, (n_pool * P, 2 * D), dtype=torch.uint8, device=dev)
            t[:, :Dq] &= 0xBF
            t[:, Dq:] = 0
            t[:, Dq + 3] = 0x3F                       # little-endian fp32 0.5
            return t.view(torch.bfloat16).view(n_pool, P, D)
        K_pool, V_pool = rows8(), rows8()
    else:
        K_pool = torch.empty(n_pool, P, D, dtype=torch.bfloat16, device=dev).normal_()
        V_pool = torch.empty(n_pool, P, D, dtype=torch.bfloat16, device=dev).normal_()
    table = torch.from_numpy((first[:, None] + np.arange(max_pages)[None, :]).astype(np.int32)).to(dev)
    cache = binding.kvzap_cache_create(ctx.handle, B, w, P, K_pool, V_pool, max_pages)
    # imported page tables are private to each list (contiguous runs); growth pages come from each run's tail
    binding.kvzap_cache_import(ctx.handle, cache, torch.from_numpy(prefix).to(dev), table, n_pool)
    Xd = synth.hidden_states(L * B, wl.d_model, 1, dev).view(L, B, wl.d_model)
    Kn, Vn = synth.keys_values(L * B, H, Dq, 2, dev)
    if fp8:
        Kn, Vn = synth.pack_rows_e4m3(Kn), synth.pack_rows_e4m3(Vn)
    for _ in range(w + 3):            # fill every window; tau = +inf keeps the prefixes as imported
        binding.kvzap_decode_step(ctx.handle, cache, 0, L, Xd, Kn.view(L, B, H, D), Vn.view(L, B, H, D), float("inf"), None)
    lengths = torch.zeros(B, L, H, dtype=torch.int32, device=dev)
    binding.kvzap_cache_lengths(ctx.handle, cache, lengths)
    torch.cuda.synchronize()
    if ctx.poll_status() != 0:
        raise RuntimeError("device status word set while the cache was filled")
    rows = float(lengths.sum().item())
    Qs = [synth.hidden_states(L * B * H * G, Dq, 50 + i, dev).view(L, B, H * G, Dq) for i in range(3)]
    Os = [torch.empty_like(q) for q in Qs]
    prepare = binding.prepare_decode_attention_fp8 if fp8 else binding.prepare_decode_attention
    calls = [prepare(ctx.handle, cache, 0, L, Qs[i], 1.0 / Dq ** 0.5, Os[i]) for i in range(3)]
    n_warm, steps = max(args.warmup, 3), min(args.steps, 30)
    for i in range(n_warm):
        calls[i % 3]()
    barrier()
    sampler = ClockSampler(dev.index)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launch_count()
    sampler.start()
    barrier()
    e0.record()
    for i in range(steps):
        calls[i % 3]()
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = env["max_over_ranks"](e0.elapsed_time(e1)) / steps
    if ctx.poll_status() != 0:
        raise RuntimeError("device status word set during the timed region")
    peaks, peak_src = load_peaks()
    alg_bytes = rows * 2 * D * 2 + 2 * L * B * H * G * Dq * 2       # every K and V row once; Q read, O written
    achieved = alg_bytes / (ms * 1e-3) / 1e9
    line = {"metric": "decode attention over the pruned cache, sequences/sec per layer", "value": world * B / (ms * 1e-3 / L),
            "unit": "sequences/s/layer", "n_gpus": world, "steps": steps, "warmup": n_warm, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "e4m3 rows (fp32 scale per row), bf16 queries, fp32 accumulation" if fp8 else "bf16", "data": "synthetic",
            "config": {"workload": wl.name + " / attention" + (" / fp8 rows" if fp8 else ""), "n_kv_heads": H, "n_q_heads": H * G,
                       "head_dim": Dq, "row_bytes": 2 * D,
                       "n_layers": L, "batch": B, "window": w, "page_tokens": P,
                       "sequence_len": [wl.prefix_min, wl.prefix_max], "kept_fraction": [0.15, 0.35],
                       "rows_per_list_mean": rows / n_lists,
                       "l2": "the lists read by one call (%.1f GB) exceed L2" % (rows * 2 * D * 2 / 1e9),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks, "gpu_launches": int(ctx.launch_count() - launches0),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "traffic": alg_bytes * (NCU_ATTENTION_FP8_TRAFFIC_RATIO if fp8 else NCU_ATTENTION_TRAFFIC_RATIO),
                         "kernel": "decode_attn_kernel", "peak_source": peak_src, "kernel_ms": ms,
                         "algorithmic_bytes_per_step": alg_bytes}}
    binding.kvzap_cache_destroy(cache)
    ctx.close()
    return line


def make_env(backend="nccl"):
    """Process-group plumbing of the N > 1 run: replicas only, so all it carries is the barrier around the
    timed region and the maximum over ranks of the timed duration.  `backend="gloo"` runs the same code
    on CPU tensors (used by the multi-process CPU test)."""
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    on_gpu = backend == "nccl"
    dev = torch.device("cuda", local_rank) if on_gpu else torch.device("cpu")
    if on_gpu:
        torch.cuda.set_device(local_rank)
    if world > 1:
        # the path needs no exchange between ranks: no collective moves any data of the method
        if on_gpu:
            dist.init_process_group(backend, device_id=dev)
        else:
            dist.init_process_group(backend)

    def barrier():
        if world > 1:
            dist.barrier()
        if on_gpu:
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return ms

    def close():
        if world > 1:
            dist.destroy_process_group()

    return {"dev": dev, "rank": rank, "world": world, "barrier": barrier, "max_over_ranks": max_over_ranks,
            "close": close}


def summarise(line):
    """The short record of one workload for the headline line's `configs` list."""
    bd, rf = line["breakdown"], line["roofline"]
    rec = {"workload": line["config"]["workload"], "value": line["value"], "unit": line["unit"], "steps": line["steps"],
           "ms_per_step": line["ms_per_step"], "step_ms": line.get("step_ms"), "layer_frac_of_roofline": bd.get("layer_frac_of_roofline"),
           "roofline_bound": rf["bound"], "roofline_frac": rf["frac"], "clocks": line["clocks"],
           "gpu_launches": line["gpu_launches"]}
    if "layer_ms" in bd:
        rec.update({"ms_per_layer": bd["layer_ms"], "layer_roofline_ms": bd["layer_roofline_ms"],
                    "kept_fraction": bd["kept_fraction"], "compaction_alone_GBps": bd.get("compaction_alone_GBps")})
        if rf["bound"] == "tensor":
            rec.update({"peak_kind": rf["peak_kind"].split(" ")[0], "frac_of_burst": rf["frac_of_burst"],
                        "frac_of_sustained": rf["frac_of_sustained"]})
    else:
        rec.update({"ms_per_layer": bd["layer_us"] * 1e-3, "layer_roofline_ms": bd["layer_roofline_us"] * 1e-3,
                    "kept_fraction_of_exiting_tokens": bd["kept_fraction_of_exiting_tokens"]})
    return rec


def run_ours(args, wl, with_configs):
    import gc
    import torch
    from paper_2601_07891_b200 import synth
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    env = make_env("nccl")
    rank, world = env["rank"], env["world"]
    if args.attention:
        if wl.decode_steps == 0:
            raise SystemExit("--attention goes with the decode workload")
        line = run_attention(args, wl, env)
    else:
        line = run_decode(args, wl, env) if wl.decode_steps > 0 else run_prefill(args, wl, env)
    if rank == 0 and world == 1 and not args.skip_cpu and wl.decode_steps == 0 and not args.fp8:
        # the oracle on the host cores, bounded sample
        n_sample = min(wl.batch * wl.seq_len, args.ref_tokens)
        v, dt, threads, n_l = oracle_sample(wl, n_sample, budget_s=12.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": "%d layer(s), first %d tokens of each: scoring + mask + compaction (%.1f s)"
                                          % (n_l, n_sample, dt)}
    if with_configs and world == 1 and not args.attention:
        # the other workloads, each in full, in the same process (short records; the headline is the line itself)
        records = []
        for idx, name in enumerate(synth.WORKLOAD_ORDER):
            if name == wl.name:
                continue
            gc.collect()
            torch.cuda.empty_cache()
            sub_wl = synth.WORKLOADS[name]
            saved = args.workload_index
            args.workload_index = idx + 1
            try:
                sub = run_decode(args, sub_wl, env, sub=True) if sub_wl.decode_steps > 0 else run_prefill(args, sub_wl, env, sub=True)
                records.append(summarise(sub))
            finally:
                args.workload_index = saved
        line["configs"] = records
    if rank == 0:
        print(json.dumps(line), flush=True)
    env["close"]()


def main():
    from paper_2601_07891_b200 import synth
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=list(synth.WORKLOAD_ORDER),
                    help="one workload only (default: the largest, %s, plus short records of the other four)" % HEADLINE)
    ap.add_argument("--no-configs", action="store_true", help="default run: leave the other four workloads out")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--layers", type=int, default=0, help="run only the first N layers (small case for profiling)")
    ap.add_argument("--kv-layout", default="heads", choices=["heads", "proj"],
                    help="prefill workloads: K/V as [H,T,D] (default) or as the projection writes them, [T,H,D]")
    ap.add_argument("--fp8", action="store_true",
                    help="hidden states and first-layer weights as E4M3 bytes with scales (prefill and decode workloads); "
                         "with --attention: cache rows of E4M3 codes with a per-row scale")
    ap.add_argument("--graph", choices=["off", "step", "layer"], default="off",
                    help="decode workload: replay the steps from a captured CUDA graph, one launch per step or one per layer")
    ap.add_argument("--attention", action="store_true",
                    help="decode workload: time the attention over the pruned cache instead of the pruning step")
    ap.add_argument("--skip-live-peak", action="store_true",
                    help="tensor-bound workloads: do not run the cuBLAS loop that measures this GPU's sustained rate")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--ref-tokens", type=int, default=32768,
                    help="tokens of one layer the CPU oracle is timed on (bounded sample)")
    args = ap.parse_args()
    with_configs = args.workload is None and not args.no_configs and args.layers == 0
    if args.workload is None:
        args.workload = HEADLINE
    args.workload_index = synth.WORKLOAD_ORDER.index(args.workload) + 1
    wl = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        if args.steps > 3:
            args.ref_tokens = min(args.ref_tokens, 4096)     # keep the whole run within minutes
        run_reference(args, wl)
    else:
        run_ours(args, wl, with_configs)


if __name__ == "__main__":
    main()
