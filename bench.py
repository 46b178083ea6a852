#!/usr/bin/env python
"""Decode-step benchmark of the WeightedKV CUDA library.

One *step* = one new token for every sequence of the batch through all layers: n_layers calls of
wkv_decode_step (one kernel launch each), compression and value merge included.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl wkv|reference]

N > 1 is launched by torch.distributed.run, one rank per GPU; every rank decodes its own batch (the lanes of
Algorithm 1 are independent, so there is no data-path collective) and the time is the maximum over ranks.
`--impl reference` times the CPU oracle on the host cores instead (rank 0 only).
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

import torch  # noqa: E402

from paper_2503_01330_b200.multi import aggregate_steps_per_s, max_over_ranks, rank_seed  # noqa: E402
from paper_2503_01330_b200.synth import BASE_SEED, WORKLOADS, TokenStream, sequence_lengths  # noqa: E402

METRIC = "decode steps/sec incl. merge; achieved HBM GB/s vs B200 peak (1 GPU)"
FALLBACK_HBM_GBS = 6650.0
# workload -> (dram__bytes_read.sum + dram__bytes_write.sum per layer call, hash of the kernel source when captured);
# profiles/scan_kernel_and_lane_epilogue_kernel_serving_b16.md
NCU_TRAFFIC = {"serving_b16": (1090256000 + 3704320 + 27001000 + 4352, "31d998bb0dfd8fd1")}


def kernel_source_hash() -> str:
    import hashlib
    path = os.path.join(ROOT, "paper_2503_01330_b200", "csrc", "wkv_kernels.cuh")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


# ------------------------------------------------------------------------------------------------------
def algorithmic_bytes_per_launch(wl) -> int:
    """Bytes one layer launch must move at a full cache (L = budget + 1 entries per lane):
    K and V rows read once, a read + written, pos read, plus q, the appended k and v, out and the merge rows."""
    L, d, e, G = wl.budget + 1, wl.head_dim, wl.elem_bytes, wl.group
    per_lane = L * (2 * d * e + 12) + (2 * G + 5) * d * e
    return wl.batch * wl.n_kv_heads * per_lane


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples the SM clock and the throttle reasons while the timed regions run: NVML every 20 ms from a thread
    (read-only queries), or nvidia-smi every 100 ms when NVML cannot be loaded.  Every sample carries a host time, so
    that a timed region can be given the median of its own samples."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples = []                      # (host time, sm MHz, set of active reasons)
        self.max_mhz, self.proc, self.thread, self._stop, self.source = None, None, None, threading.Event(), None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            # bits of NVML's clocks-event-reasons mask
            bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
            get_reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(pynvml, "nvmlDeviceGetCurrentClocksThrottleReasons")

            def loop():
                while not self._stop.is_set():
                    try:
                        mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                        mask = int(get_reasons(h))
                        self.samples.append((time.perf_counter(), mhz, {n for n, b in bits.items() if mask & b}))
                    except Exception:
                        pass
                    self._stop.wait(self.period)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.source = "nvml"
            return
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            self.source = "nvidia-smi"
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            r = [x.strip() for x in line.split(",")]
            try:
                self.max_mhz = max(self.max_mhz or 0.0, float(r[1]))
                self.samples.append((time.perf_counter(), float(r[0]),
                                     {n for n, v in zip(self.NAMES, r[2:6]) if v.lower().startswith("active")}))
            except Exception:
                pass

    def stop(self):
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def summary(self, t0=None, t1=None):
        """Median SM MHz and the reasons seen between host times t0 and t1 (default: all samples)."""
        if self.source is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source"], "samples": 0}
        rows = [r for r in self.samples if (t0 is None or r[0] >= t0) and (t1 is None or r[0] <= t1)]
        reasons = set()
        for r in rows:
            reasons |= r[2]
        return {"sm_mhz": statistics.median(r[1] for r in rows) if rows else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(reasons), "samples": len(rows), "source": self.source}


# ------------------------------------------------------------------------------------------------------
def oracle_lane_steps_per_s(wl, n_lanes: int, steps: int, warmup: int, seed: int, budget_s: float = 0.0):
    """Times the CPU oracle as it stands on `n_lanes` lanes of the workload's shape at a full cache.  The caches are
    set up through the oracle's import (synthetic full lanes of the workload's key / value distributions) -- filling
    them token by token would cost minutes of growth steps that the metric does not time.  With budget_s > 0 the number
    of timed steps is chosen from the warm-up steps' duration so that the timed part takes about budget_s seconds
    (at least `steps`).  Returns (lane-steps per second, threads used, timed steps)."""
    import numpy as np
    import oracle
    oracle.build()
    sub = wl.scaled(n_layers=1, batch=1, n_kv_heads=n_lanes, n_q_heads=n_lanes * wl.group)
    ref = oracle.Oracle(n_lanes, wl.head_dim, wl.budget, window=wl.window, sink=wl.sink, group=wl.group,
                        dtype=oracle.F32 if wl.dtype == "f32" else oracle.BF16, mode=oracle.MODE_PINNED)
    stream = TokenStream(sub, seed, "cpu")
    m = wl.budget
    _, Kp, Vp = stream.prompt(0, m)                               # [1, m, n_lanes, d]
    rng = np.random.default_rng(seed)
    pos = np.arange(m, dtype=np.int32)
    for lane in range(n_lanes):
        ref.import_state(lane, m, pos, rng.random(m) + 0.1, Kp[0, :, lane].float().numpy(), Vp[0, :, lane].float().numpy())

    def tok(t):
        q, k, v = stream.token(t)
        return q[0, 0].float().numpy().reshape(n_lanes, wl.group, -1), k[0, 0].float().numpy(), v[0, 0].float().numpy()

    t0 = time.perf_counter()
    for i in range(max(1, warmup)):
        ref.step(*tok(m + i))
    per_step = (time.perf_counter() - t0) / max(1, warmup)
    if budget_s > 0:
        steps = max(steps, min(256, int(budget_s / max(per_step, 1e-6))))
    toks = [tok(m + max(1, warmup) + i) for i in range(steps)]
    t0 = time.perf_counter()
    for q, k, v in toks:
        ref.step(q, k, v)
    dt = time.perf_counter() - t0
    ref.close()
    return n_lanes * steps / dt, min(n_lanes, os.cpu_count() or 1), steps


FP32_LANES_PER_SM = 128          # fp32 FMA lanes per SM (4 sub-partitions x 32); one FMA per lane and clock


def bulk_prefill_figures(wl, dev, seed, n_tokens=0, reps=3):
    """wkv_prefill_bulk on ONE layer of the workload's shape: every sequence brings a prompt of n_tokens (default:
    the budget, i.e. the whole dense phase).  The kernel is arithmetic-bound: the roofline is the fp32 FMA pipe,
    peak = SMs x 128 lanes x max SM clock; algorithmic FMAs = lanes x G x n(n+1)/2 x head_dim x 2 (logits and P.V)."""
    from paper_2503_01330_b200 import binding
    one = wl.scaled(n_layers=1)
    n = n_tokens if n_tokens else one.budget
    n = min(n, one.budget)
    ctx = binding.Context(1, one.batch, one.n_q_heads, one.n_kv_heads, one.head_dim, one.budget, one.window, one.sink,
                          binding.WKV_F32 if one.dtype == "f32" else binding.WKV_BF16, device=dev)
    Q, K, V = TokenStream(one, seed, dev).prompt(0, n)
    out = torch.empty(one.batch, n, one.n_q_heads, one.head_dim, dtype=one.torch_dtype, device=dev)
    times = []
    for _ in range(reps + 1):                      # the first run also takes the scratch from the allocator
        ctx.wkv_reset()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.wkv_prefill_bulk(0, Q, K, V, None, out)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    # the same prompt token by token (wkv_prefill: one decode launch per token), for scale
    ctx.wkv_reset()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ctx.wkv_prefill(0, Q, K, V, None, out)
    e1.record()
    torch.cuda.synchronize()
    streamed_ms = e0.elapsed_time(e1)
    assert ctx.wkv_status() == 0
    ctx.close()
    ms = min(times[1:])
    lanes = one.batch * one.n_kv_heads
    fma = lanes * one.group * n * (n + 1) // 2 * one.head_dim * 2
    props = torch.cuda.get_device_properties(dev)
    try:
        import pynvml
        pynvml.nvmlInit()
        max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(pynvml.nvmlDeviceGetHandleByIndex(dev.index or 0), pynvml.NVML_CLOCK_SM)
    except Exception:
        max_mhz = 1965
    peak = props.multi_processor_count * FP32_LANES_PER_SM * max_mhz * 1e6 / 1e12
    achieved = fma / (ms * 1e-3) / 1e12
    return {"value": one.batch * n / (ms * 1e-3), "unit": "prompt tokens/s per layer", "ms_per_layer": ms,
            "tokens_per_sequence": n, "kernel": "prefill_bulk_kernel",
            "streamed_ms_per_layer": streamed_ms,
            "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFMA/s (fp32)", "frac": achieved / peak,
                         "traffic": None, "peak_kind": f"{props.multi_processor_count} SMs x {FP32_LANES_PER_SM} lanes x {max_mhz} MHz",
                         "algorithmic_fma_per_launch": fma}}


def whole_prompt_figures(wl, dev, seed, n_tokens):
    """A prompt of n_tokens per sequence for ALL layers in one wkv_prefill_bulk_layers call, and the same prompt streamed
    layer by layer through wkv_prefill (Algorithm 1 as printed), for workloads whose prompt tensors fit beside the cache."""
    from paper_2503_01330_b200 import binding
    per_layer = wl.batch * n_tokens * (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim * wl.elem_bytes
    if per_layer * wl.n_layers > (24 << 30):
        raise SystemExit("prompt tensors of all layers would take more than 24 GB: use --mode prefill (one layer)")
    ctx = binding.Context(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.budget, wl.window, wl.sink,
                          binding.WKV_F32 if wl.dtype == "f32" else binding.WKV_BF16, device=dev)
    st = TokenStream(wl, seed, dev)
    parts = [st.prompt(layer, n_tokens) for layer in range(wl.n_layers)]
    Q, K, V = (torch.stack([p[i] for p in parts]) for i in range(3))
    parts = None
    out = torch.empty_like(Q)                       # the attention output of every prompt token is part of the work

    def timed(fn):
        ctx.wkv_reset()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def streamed():
        for layer in range(wl.n_layers):
            ctx.wkv_prefill(layer, Q[layer], K[layer], V[layer], None, out[layer])

    timed(lambda: ctx.wkv_prefill_bulk_layers(Q, K, V, None, out))            # takes the scratch, warms the path
    bulk_ms = min(timed(lambda: ctx.wkv_prefill_bulk_layers(Q, K, V, None, out)) for _ in range(2))
    streamed_ms = timed(streamed)
    assert ctx.wkv_status() == 0
    ctx.close()
    return {"metric": "whole_prompt_ms_all_layers", "value": bulk_ms, "unit": "ms", "higher_is_better": False,
            "streamed_layer_by_layer_ms": streamed_ms, "prompt_tokens_per_s": wl.batch * n_tokens / (bulk_ms * 1e-3),
            "n_gpus": 1, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "n_layers": wl.n_layers, "batch": wl.batch, "budget": wl.budget,
                       "window": wl.window, "sink": wl.sink, "prompt_tokens": n_tokens,
                       "call": "wkv_prefill_bulk_layers with outputs: dense phase for the first budget tokens, the rest in blocks "
                               "of tokens that share two sweeps of the cache (token by token where the shape does not allow blocks)"}}


def run_reference(args, wl):
    """The reference arm: the CPU oracle on the host cores; each step is a bounded sample of the workload."""
    cores = os.cpu_count() or 1
    n_lanes = min(wl.lanes, 4 * cores)
    lane_rate, used, steps = oracle_lane_steps_per_s(wl, n_lanes, args.steps, args.warmup, BASE_SEED)
    value = lane_rate / wl.lanes
    sample = (f"{n_lanes} of {wl.lanes} lanes at a full cache ({wl.budget + 1} entries attended, caches imported), "
              f"{steps} timed steps after {max(1, args.warmup)} warm-up steps; full-workload rate = lane-steps/s / lanes "
              f"(lanes are independent)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, args, None),
            "cpu_baseline": {"value": value, "unit": "steps/s", "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(wl, args, splits):
    return {"workload": wl.name, "n_layers": wl.n_layers, "batch_per_gpu": wl.batch, "n_q_heads": wl.n_q_heads,
            "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim, "budget": wl.budget, "window": wl.window,
            "sink": wl.sink, "prefill_tokens": args.prefill_tokens if args.prefill_tokens else wl.budget + 64,
            "prefill": "wkv_prefill_bulk per layer (dense for the first budget tokens, the rest streamed) until every cache is full and compressing" if args.init == "prefill"
            else "synthetic full caches through wkv_import_state (profiling only)",
            "n_splits": splits, "l2": "inputs larger than L2 (cache rows streamed once per step)",
            "parallelism": f"lanes replicated per GPU x{args.gpus}, no collective"}


OTHER_WORKLOADS = ["tiny", "llama7b_layer", "llama7b_b8", "gqa_b32"]
REPEATS = 5


def decode_figures(wl, args, dev, seed, dist, world, sampler, headline):
    """Sets a context of workload `wl` up (prompt of budget + 64 tokens per sequence, or imported full caches), runs the
    warm-up steps and then REPEATS timed regions of `steps` decode steps each (n_layers wkv_decode_step calls per step),
    every region bracketed by a stream synchronisation and CUDA events on the launching stream.  The value is the
    median region; the regions' own median SM clocks are reported beside them.  headline = True adds the all-layers
    call, the end-to-end leg from pinned host buffers and the ncu traffic figure."""
    from paper_2503_01330_b200 import binding
    steps = args.steps if headline else max(8, min(args.steps, 2000 // wl.n_layers if wl.n_layers > 1 else 200))
    warmup = max(3, args.warmup)
    dt_code = binding.WKV_F32 if wl.dtype == "f32" else binding.WKV_BF16
    ctx = binding.Context(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.budget, wl.window, wl.sink,
                          dt_code, n_splits=args.n_splits if headline else 0, device=dev,
                          schedule=args.schedule if headline else 0)
    stream = TokenStream(wl, seed, dev)
    n_prefill = args.prefill_tokens if (args.prefill_tokens and headline) else wl.budget + 64
    # ragged prompt lengths in the last 32 tokens of the (shortened) prefill: every cache ends up full
    lens = sequence_lengths(wl.scaled(prefill=n_prefill, prefill_min=max(1, n_prefill - 32)), seed).to(dev)
    if args.init == "import":
        g = torch.Generator().manual_seed(seed)
        m = wl.budget
        K1 = torch.randn(m, wl.head_dim, generator=g).to(wl.torch_dtype)
        V1 = torch.randn(m, wl.head_dim, generator=g).to(wl.torch_dtype)
        a1 = torch.rand(m, generator=g) + 0.1
        p1 = torch.arange(m, dtype=torch.int32)
        for layer in range(wl.n_layers):
            for b in range(wl.batch):
                for h in range(wl.n_kv_heads):
                    ctx.wkv_import_state(layer, b, h, m, p1, a1, K1, V1)
        n_prefill = m
    else:
        # the prompt, layer by layer: the first `budget` tokens through the dense kernel, the rest streamed behind it
        rel = lens.clamp(max=n_prefill).to(torch.int32)
        for layer in range(wl.n_layers):
            Q, K, V = stream.prompt(layer, n_prefill)
            ctx.wkv_prefill_bulk(layer, Q, K, V, rel)
            torch.cuda.synchronize()
        Q = K = V = None
    torch.cuda.synchronize()

    n_distinct = min(warmup + steps, 64)                      # tokens are cycled: the values do not matter to the timing
    toks = [stream.token(n_prefill + i) for i in range(n_distinct)]
    out = torch.empty(wl.n_layers, wl.batch, wl.n_q_heads, wl.head_dim, dtype=wl.torch_dtype, device=dev)
    ev = torch.empty(wl.n_layers, wl.batch, wl.n_kv_heads, dtype=torch.int32, device=dev)

    def step(i):
        q, k, v = toks[i % n_distinct]
        for layer in range(wl.n_layers):
            ctx.wkv_decode_step(layer, q[layer], k[layer], v[layer], out[layer], ev[layer])

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    regions, launches = [], 0
    for r in range(REPEATS):
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        launches0 = ctx.wkv_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0 = time.perf_counter()
        e0.record()
        for i in range(steps):
            step(warmup + r * steps + i)
        e1.record()
        torch.cuda.synchronize()
        h1 = time.perf_counter()
        launches = ctx.wkv_launch_count() - launches0
        ms = max_over_ranks(e0.elapsed_time(e1), dist, dev)
        if dist is not None:
            dist.barrier()
        ck = sampler.summary(h0, h1)
        regions.append({"ms": ms, "steps_per_s": aggregate_steps_per_s(world, steps, ms), "sm_mhz": ck["sm_mhz"],
                        "clock_samples": ck["samples"], "reasons": ck["reasons"]})
    assert ctx.wkv_status() == 0, "device status word reports an error"
    assert int((ev >= 0).sum()) == ev.numel(), "every lane must compress in the timed region"
    by_ms = sorted(regions, key=lambda x: x["ms"])
    med = by_ms[len(by_ms) // 2]
    elapsed_ms = med["ms"]
    value = med["steps_per_s"]
    peak, peak_kind = hbm_peak()
    bytes_launch = algorithmic_bytes_per_launch(wl)
    # one layer call = the scan kernel plus (two-kernel schedule) the lane-epilogue kernel; their bytes are the
    # algorithmic bytes of one layer, so the fraction is taken over the whole call, not over the scan alone
    launch_ms = elapsed_ms / (steps * wl.n_layers)
    achieved = bytes_launch / (launch_ms * 1e-3) / 1e9
    two_kernels = launches == 2 * steps * wl.n_layers
    # DRAM bytes per layer call from the ncu capture summarised under profiles/ (scan + lane epilogue kernels); only
    # reported while the kernel source is the one that was profiled
    traffic = None
    if headline and NCU_TRAFFIC.get(wl.name) and NCU_TRAFFIC[wl.name][1] == kernel_source_hash() and not args.layers:
        traffic = NCU_TRAFFIC[wl.name][0]
    mhz = [x["sm_mhz"] for x in regions if x["sm_mhz"] is not None]
    reasons = sorted({n for x in regions for n in x["reasons"]})
    fig = {"value": value, "unit": "steps/s", "steps": steps, "ms_per_step": elapsed_ms / steps,
           "n_splits": ctx.wkv_splits(), "gpu_launches": launches,
           "init": "prompt of budget + 64 tokens through wkv_prefill_bulk" if args.init == "prefill" else "imported full caches",
           "clocks": {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": sampler.max_mhz, "reasons": reasons,
                      "samples": sum(x["clock_samples"] for x in regions), "source": sampler.source},
           "repeats": {"n": REPEATS, "value": "median", "min_steps_per_s": by_ms[-1]["steps_per_s"],
                       "max_steps_per_s": by_ms[0]["steps_per_s"], "regions": regions},
           "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                        "traffic": traffic, "peak_kind": f"of {peak_kind}", "frac_of_8000_nominal": achieved / 8000.0,
                        "kernel": "scan_kernel (+ lane_epilogue_kernel)" if two_kernels else "decode_step_cluster_kernel",
                        "algorithmic_bytes_per_launch": bytes_launch, "launch_ms": launch_ms}}

    # ---- additionally: the same steps through wkv_decode_step_layers (all layers' inputs handed over at once, so the
    # library may overlap one layer's lane epilogues with the next layer's scan, or run all layers in one launch) ----
    if wl.n_layers > 1:
        n_all = max(1, min(steps, 100))
        for i in range(3):
            q, k, v = toks[i % n_distinct]
            ctx.wkv_decode_step_layers(q, k, v, out, ev)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for i in range(n_all):
            q, k, v = toks[(warmup + i) % n_distinct]
            ctx.wkv_decode_step_layers(q, k, v, out, ev)
        a1.record()
        torch.cuda.synchronize()
        all_ms = max_over_ranks(a0.elapsed_time(a1), dist, dev)
        fig["all_layers_call"] = {"value": aggregate_steps_per_s(world, n_all, all_ms), "unit": "steps/s", "steps": n_all,
                                  "ms_per_step": all_ms / n_all,
                                  "frac": bytes_launch * wl.n_layers / (all_ms / n_all * 1e-3) / 1e9 / peak,
                                  "note": "wkv_decode_step_layers: one call per step with every layer's q, k, v ready beforehand"}
    else:
        fig["all_layers_call"] = None

    if headline:
        # ---- end to end: host buffers through wkv_decode_step_layers_host, copies inside the timed region ----
        n_e2e = max(1, min(args.e2e_steps, steps))
        host = [tuple(x.cpu().pin_memory() for x in toks[(warmup + i) % n_distinct]) for i in range(min(n_e2e, n_distinct))]
        out_h = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        ev_h = torch.empty(ev.shape, dtype=ev.dtype).pin_memory()
        ctx.wkv_decode_step_layers_host(host[0][0], host[0][1], host[0][2], out_h, ev_h)       # warm the path once
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for i in range(n_e2e):
            q, k, v = host[i % len(host)]
            ctx.wkv_decode_step_layers_host(q, k, v, out_h, ev_h)    # copies in, all layers, copies out, stream wait
        h1.record()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(h0.elapsed_time(h1), dist, dev)
        h2d = sum(x.numel() * x.element_size() for x in host[0])
        d2h = out_h.numel() * out_h.element_size() + ev_h.numel() * ev_h.element_size()
        fig["e2e"] = {"value": aggregate_steps_per_s(world, n_e2e, e2e_ms), "unit": "steps/s", "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": n_e2e,
                      "call": "wkv_decode_step_layers_host: one call per step from pinned host buffers"}
    assert ctx.wkv_status() == 0, "device status word reports an error"
    ctx.close()
    del ctx, toks, out, ev
    torch.cuda.empty_cache()
    return fig


# ------------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="serving_b16", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="wkv", choices=["wkv", "reference"])
    ap.add_argument("--prefill-tokens", type=int, default=0, help="0 = budget + 64")
    ap.add_argument("--n-splits", type=int, default=0)
    ap.add_argument("--schedule", type=int, default=0, help="0 = library's choice, 1 = scan + epilogue kernels, 2 = clusters")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling captures)")
    ap.add_argument("--mode", default="decode", choices=["decode", "prefill", "prompt"],
                    help="prefill: time only the dense prompt phase (wkv_prefill_bulk) on one layer and print its line; "
                         "prompt: a whole prompt of --prefill-tokens (default: the workload's prefill length) for all "
                         "layers through wkv_prefill_bulk_layers, beside the same prompt streamed")
    ap.add_argument("--no-bulk-prefill", action="store_true", help="leave the bulk-prefill figure out of the decode line")
    ap.add_argument("--no-other-workloads", action="store_true", help="leave the short runs of the other workloads out of the line")
    ap.add_argument("--init", default="prefill", choices=["prefill", "import"],
                    help="import: fill every cache through wkv_import_state with one synthetic full lane instead of "
                         "streaming a prompt (profiling captures: no launches before the steps)")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    if args.layers > 0:
        wl = wl.scaled(n_layers=args.layers)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            if args.steps > 64:
                args.steps = 16          # keep the whole run within a few minutes
            run_reference(args, wl)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation of the path")
    if args.warmup < 3:
        args.warmup = 3
    from paper_2503_01330_b200 import binding
    from paper_2503_01330_b200.build import build_library
    if rank == 0:
        build_library()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)

    seed = rank_seed(BASE_SEED, rank)
    if args.mode == "prompt":
        fig = whole_prompt_figures(wl, dev, seed, args.prefill_tokens if args.prefill_tokens else wl.prefill)
        if rank == 0:
            print(json.dumps(fig), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return
    if args.mode == "prefill":
        fig = bulk_prefill_figures(wl, dev, seed, args.prefill_tokens)
        if rank == 0:
            fig.update({"metric": "bulk_prefill_prompt_tokens_per_s_per_layer", "n_gpus": 1, "higher_is_better": True,
                        "dtype": wl.dtype, "data": "synthetic",
                        "config": {"workload": wl.name, "layers_timed": 1, "batch": wl.batch, "budget": wl.budget}})
            print(json.dumps(fig), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return
    sampler = ClockSampler(local_rank)
    sampler.start()
    head = decode_figures(wl, args, dev, seed, dist, world, sampler, headline=True)
    others = {}
    if rank == 0 and world == 1 and not args.no_other_workloads and not args.layers:
        for name in OTHER_WORKLOADS:
            if name != wl.name:
                others[name] = decode_figures(WORKLOADS[name], args, dev, seed, None, 1, sampler, headline=False)
    sampler.stop()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {"metric": METRIC, "value": head["value"], "unit": "steps/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_config(wl, args, head["n_splits"]),
            "gpu_launches": head["gpu_launches"], "clocks": head["clocks"], "repeats": head["repeats"],
            "all_layers_call": head["all_layers_call"], "roofline": head["roofline"], "e2e": head["e2e"]}
    if others:
        line["other_workloads"] = others
    if not args.no_bulk_prefill:
        line["bulk_prefill"] = bulk_prefill_figures(wl, dev, seed)
        if world == 1 and not args.layers and wl.name == "serving_b16":
            # a whole prompt past the budget (dense phase + blocked tail) on two layers of the shape, beside the same
            # prompt streamed as Algorithm 1 prints it
            import dataclasses
            line["whole_prompt"] = whole_prompt_figures(dataclasses.replace(wl, n_layers=2), dev, seed, 2 * wl.budget)
    if not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        n_lanes = min(wl.lanes, 4 * cores)
        lane_rate, used, n_steps = oracle_lane_steps_per_s(wl, n_lanes, 4, 1, BASE_SEED, budget_s=12.0)
        line["cpu_baseline"] = {"value": lane_rate / wl.lanes, "unit": "steps/s", "cores": used, "kind": "oracle",
                                "sample": f"{n_lanes} of {wl.lanes} lanes at a full cache (imported), {n_steps} timed steps; "
                                          f"full-workload rate = lane-steps/s / lanes (lanes are independent)"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
