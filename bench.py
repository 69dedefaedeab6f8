#!/usr/bin/env python
"""Benchmark of the mixed decode + chunked-prefill paged-attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--repeats R] [--impl ours|reference] [--no-per-config]

One *step* = one unit of one layer of the agentic long-context mixed batch: cf_kv_append followed by
cf_mixed_attention (split-K decode with its merge, chunked prefill) over 16 decode sequences with
contexts of 8K..32K plus one 2048-token prefill chunk that sits on 24,576 + 2048*t cached tokens;
steps cycle through the four chunks t = 0..3 of the 8192-token prompt.
Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank runs an
independent replica of the batch on its own GPU: the path has no exchange step, so there is no
data-path collective; the only collective is the max-over-ranks of the device time.

The timed region of K steps is repeated R times inside the invocation (synchronised on both sides
every time); `value` and `ms_per_step` are the median repeat, `repeats` lists every repeat with the
SM clock sampled while it ran, so that a cold burst and the power-limited steady state can be told
apart.  `value` is measured in the library's default launch sequence; `serial` repeats the steps with
one kernel after the other, which is also the sequence the per-kernel times under `kernels` /
`roofline` are taken in.  `per_config` carries the same measurements for the other workload
configurations (device times only, fewer repeats).

`--impl reference` times the fp64 CPU oracle (as it stands) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import cf_synth as syn  # noqa: E402

METRIC = "mixed decode+prefill paged-attention query-tokens/s"
UNIT = "query-tokens/s"
WORKLOAD = ("configs[3] agentic long-context mixed batch: 16 decode seqs (ctx uniform in [8192, 32768]) "
            "+ 1 prefill of 8192 new tokens over 24576 cached, 2048-token chunks; Hq 32, Hkv 8, D 128, block 16, bf16; "
            "one step = kv_append + mixed attention of one chunk iteration (t cycles 0..3)")
# DRAM traffic per algorithmic byte of the split-K decode kernel, from an ncu capture on the reduced
# decode case (dram bytes read + written: 560.9 MB for 555.2 MB algorithmic); traffic grows in
# proportion to the K/V bytes, so a full launch is scaled by its algorithmic bytes.
DECODE_TRAFFIC_RATIO = 1.010
# DRAM traffic per algorithmic byte of the tcgen05 prefill kernel, from an ncu capture of the headline's own prefill
# launch in the serial sequence (first chunk iteration: 2048 new tokens over 24,576 cached; 162.5 MB moved for
# 142.6 MB algorithmic: K/V once, q, out and the fp32 partial rows of the KV-split items).  A 4096-token chunk over
# 8192 cached tokens measures 1.28.  Prefill is tensor-bound; the figure is scaled by the launch's algorithmic bytes
# and is approximate for the later chunk iterations.
PREFILL_TRAFFIC_RATIO = 1.14
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    except Exception:
        return dict(FALLBACK_PEAKS, source="fallback")


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock, power and throttle reasons through NVML (read-only) while a region runs.
    Samples carry a host timestamp, so a caller can ask for the samples of a sub-interval."""

    def __init__(self, torch_device_index: int, period_s: float = 0.002):
        self.period = period_s
        self.samples = []            # (perf_counter, sm_mhz, watts)
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0
                except Exception:
                    watts = None
                self.samples.append((time.perf_counter(), mhz, watts))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=1.0)

    def between(self, t0: float, t1: float):
        """Median SM MHz and peak watts of the samples taken in [t0, t1] (None when there are none)."""
        sel = [(m, w) for (t, m, w) in self.samples if t0 <= t <= t1]
        if not sel:
            return None, None
        watts = [w for _, w in sel if w is not None]
        return float(np.median([m for m, _ in sel])), (max(watts) if watts else None)

    def summary(self, t0: float = None, t1: float = None):
        sel = [m for (t, m, _) in self.samples if (t0 is None or t >= t0) and (t1 is None or t <= t1)]
        if not sel:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(sel)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(sel)}


# ------------------------------------------------------------------------------------------ device workload
class DeviceWorkload:
    """A scenario resident on the GPU: pools, block table, per-iteration inputs."""

    def __init__(self, sc: syn.Scenario, torch, cf, ctx, window: int = 0, sinks: bool = False, fp8: bool = False):
        """window / sinks: the sliding-window + attention-sink variant; fp8: the pools are converted to an e4m3
        cache (per-head scale 1/32: N(0,1) values use the format's upper half without saturating)."""
        self.sc, self.torch, self.cf, self.ctx = sc, torch, cf, ctx
        self.window, self.kv_elem_bytes = window, (1 if fp8 else 2)
        g = sc.geom

        def dev(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

        self.sinks = torch.linspace(-2.0, 2.0, g.num_q_heads, device="cuda") if sinks else None
        variant = dict(window_size=window, sink_logits=self.sinks)
        if fp8:
            self.k_scale = torch.full((g.num_kv_heads,), 1.0 / 32.0, device="cuda")
            self.v_scale = torch.full((g.num_kv_heads,), 1.0 / 32.0, device="cuda")
            self.k = (dev(sc.k_pool).float() * 32.0).to(torch.float8_e4m3fn)        # input preparation only
            self.v = (dev(sc.v_pool).float() * 32.0).to(torch.float8_e4m3fn)
            variant.update(kv_dtype=cf.CF_KV_FP8_E4M3, k_scale=self.k_scale, v_scale=self.v_scale)
        else:
            self.k, self.v = dev(sc.k_pool), dev(sc.v_pool)
        self.desc = cf.make_desc(g.num_q_heads, g.num_kv_heads, g.head_dim, g.block_size, g.num_blocks, **variant)
        self.its = []
        for b in sc.batches:
            it = {"b": b, "bt": torch.from_numpy(b.block_table).cuda(), "q": dev(b.q), "kn": dev(b.k_new), "vn": dev(b.v_new),
                  "out": torch.empty((b.total_q, g.num_q_heads, g.head_dim), dtype=torch.bfloat16, device="cuda"),
                  "qh": torch.from_numpy(b.q.view(np.int16)).pin_memory(),
                  "knh": torch.from_numpy(b.k_new.view(np.int16)).pin_memory(),
                  "vnh": torch.from_numpy(b.v_new.view(np.int16)).pin_memory()}
            it["outh"] = torch.empty_like(it["qh"]).pin_memory()
            self.its.append(it)

    def step(self, i: int, stream):
        it = self.its[i % len(self.its)]
        b = it["b"]
        self.cf.cf_kv_append(self.ctx, self.desc, self.k, self.v, it["kn"], it["vn"], it["bt"], b.max_blocks,
                             b.context_len, b.query_len, stream=stream)
        self.cf.cf_mixed_attention(self.ctx, self.desc, it["q"], self.k, self.v, it["bt"], b.max_blocks,
                                   b.context_len, b.query_len, it["out"], None, stream=stream)
        return 1 + self.cf.cf_get_last_launch_count(self.ctx)

    def step_host(self, i: int, stream):
        it = self.its[i % len(self.its)]
        b = it["b"]
        self.cf.cf_mixed_step_host(self.ctx, self.desc, it["qh"], it["knh"], it["vnh"], self.k, self.v, it["bt"],
                                   b.max_blocks, b.context_len, b.query_len, it["outh"], stream=stream)

    def tokens(self, i: int) -> int:
        return self.its[i % len(self.its)]["b"].total_q

    def capture_graphs(self):
        """Plan every iteration once (cf_plan_create) and capture its cf_kv_append_planned +
        cf_mixed_attention_planned pair in a CUDA graph: what a serving engine does per layer when it
        replays a captured forward pass.  Returns (graphs, plans)."""
        torch, cf = self.torch, self.cf
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graphs, plans = [], []
        with torch.cuda.stream(side):
            for it in self.its:
                b = it["b"]
                plan = cf.cf_plan_create(self.ctx, self.desc, b.context_len, b.query_len, b.max_blocks, stream=side)
                cf.cf_kv_append_planned(plan, self.k, self.v, it["kn"], it["vn"], it["bt"], stream=side)      # warm-up outside the capture
                cf.cf_mixed_attention_planned(plan, it["q"], self.k, self.v, it["bt"], it["out"], None, stream=side)
                side.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    cf.cf_kv_append_planned(plan, self.k, self.v, it["kn"], it["vn"], it["bt"], stream=side)
                    cf.cf_mixed_attention_planned(plan, it["q"], self.k, self.v, it["bt"], it["out"], None, stream=side)
                graphs.append(g)
                plans.append(plan)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        return graphs, plans


def time_region(torch, fn, steps: int, stream) -> float:
    """Milliseconds for `steps` calls of fn(i), CUDA events on `stream`, synchronised on both sides."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(steps):
        fn(i)
    e1.record(stream)
    torch.cuda.synchronize()
    return float(e0.elapsed_time(e1))


def time_repeats(torch, fn, steps: int, stream, repeats: int, clk: "ClockSampler" = None):
    """The timed region of `steps` calls, `repeats` times.  Returns a list of
    {"ms_per_step", "sm_mhz", "watts"} (the clock is the median of the samples taken while the repeat ran)."""
    out = []
    for _ in range(repeats):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ms = time_region(torch, fn, steps, stream)
        t1 = time.perf_counter()
        mhz, watts = clk.between(t0, t1) if clk is not None else (None, None)
        out.append({"ms_per_step": ms / steps, "sm_mhz": mhz, "watts": watts})
    return out


def median_of(reps):
    return float(np.median([r["ms_per_step"] for r in reps]))


def batch_accounting(sc: syn.Scenario, window: int = 0, kv_elem_bytes: int = 2):
    acc = []
    for b in sc.batches:
        acc.append({"tokens": b.total_q,
                    "decode_bytes": syn.decode_algorithmic_bytes(b.geom, b.context_len, b.query_len, window, kv_elem_bytes),
                    "decode_flops": syn.decode_flops(b.geom, b.context_len, b.query_len, window),
                    "prefill_flops": syn.prefill_flops(b.geom, b.context_len, b.query_len, window),
                    "prefill_bytes": syn.prefill_algorithmic_bytes(b.geom, b.context_len, b.query_len, window, kv_elem_bytes)})
    return acc


# nominal chip figures (HGX B200: 7.7 TB/s HBM3e, 2.25 PFLOP/s dense bf16), reported beside the measured peaks
NOMINAL_HBM_GBS = 7700.0
NOMINAL_BF16_TFLOPS = 2250.0


def measure_kernels(torch, cf, wl: DeviceWorkload, steps: int, stream, peaks, clk: "ClockSampler" = None):
    """Per-kernel CUDA-event times (inside the library, on the launching stream, serial launch sequence) over
    `steps` steps.  Fractions: `frac` against `peak` (for the prefill kernel the burst or the sustained cuBLAS figure, chosen
    by the SM clock sampled while it was timed: see below), `frac_of_burst` and `frac_of_sustained` against both,
    `frac_of_nominal`."""
    acc = batch_accounting(wl.sc, wl.window, wl.kv_elem_bytes)
    cf.cf_set_timing(wl.ctx, True)
    launches = 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        launches += wl.step(i, stream)
    ms_dec, ms_comb, ms_pre, n = cf.cf_get_timing_sums(wl.ctx)
    t1 = time.perf_counter()
    cf.cf_set_timing(wl.ctx, False)
    mhz, _ = clk.between(t0, t1) if clk is not None else (None, None)
    dec_bytes = sum(acc[i % len(acc)]["decode_bytes"] for i in range(steps))
    pre_flops = sum(acc[i % len(acc)]["prefill_flops"] for i in range(steps))
    pre_bytes = sum(acc[i % len(acc)]["prefill_bytes"] for i in range(steps))
    out = {"ms_decode": ms_dec / steps, "ms_combine": ms_comb / steps, "ms_prefill": ms_pre / steps, "sequence": "serial",
           "sm_mhz": mhz}
    if ms_dec > 0:
        gbs = dec_bytes / ((ms_dec + ms_comb) * 1e-3) / 1e9
        out["decode"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
                         "traffic": DECODE_TRAFFIC_RATIO * dec_bytes / steps,
                         "bytes_per_launch": dec_bytes / steps, "ms": (ms_dec + ms_comb) / steps}
    if ms_pre > 0:
        tf = pre_flops / (ms_pre * 1e-3) / 1e12
        out["prefill"] = {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                          "frac": tf / peaks["bf16_tflops"], "peak_kind": "burst",
                          "frac_of_burst": tf / peaks["bf16_tflops"], "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                          "frac_of_nominal": tf / NOMINAL_BF16_TFLOPS,
                          "traffic": PREFILL_TRAFFIC_RATIO * pre_bytes / steps, "bytes_per_launch": pre_bytes / steps,
                          "flops_per_launch": pre_flops / steps, "ms": ms_pre / steps,
                          "tflops_per_ghz": (tf / (mhz / 1e3)) if mhz else None}
    return out, launches


def apply_peak_rule(kern, region_mhz, peaks):
    """Denominator of the prefill kernel's roofline: the measured cuBLAS burst figure for a kernel timed at the idle
    clock, the measured sustained figure (a seconds-long cuBLAS loop under the 1000 W cap) when this kernel, too, was
    timed inside a long power-capped run - the median SM clock of the timed region that preceded the per-kernel
    measurement sits more than 10 % below the maximum.  Both fractions stay in the record."""
    pre = kern.get("prefill")
    if not pre or region_mhz is None or region_mhz >= 0.9 * peaks.get("sm_max_mhz", 1965.0):
        return
    pre["peak"] = peaks["bf16_tflops_sustained"]
    pre["frac"] = pre["achieved"] / pre["peak"]
    pre["peak_kind"] = "sustained (power-capped run: SM clock %.0f MHz over the timed region)" % region_mhz


def measure_host_time(torch, cf, wl: DeviceWorkload, steps: int, stream):
    """Host microseconds the two ABI calls of a step cost the caller's thread, with the stream idle before
    every step (so nothing waits for a plan slot): validation, planning, plan upload, tensor-map lookup, launches."""
    cf.cf_get_host_time_sums(wl.ctx)
    for i in range(steps):
        torch.cuda.synchronize()
        wl.step(i, stream)
    torch.cuda.synchronize()
    us_append, us_attn, us_plan, n = cf.cf_get_host_time_sums(wl.ctx)
    n = max(n, 1)
    return {"append": us_append / n, "attention": us_attn / n, "planner": us_plan / n, "total": (us_append + us_attn) / n}


# ------------------------------------------------------------------------------------------ CPU oracle legs
class OracleWorkload:
    """The scenario on the host with every iteration's K/V appended (by the oracle's own scatter);
    iteration t only reads tokens below its own context lengths, so one cache serves all t."""

    def __init__(self, sc: syn.Scenario):
        import oracle
        self.oracle, self.sc = oracle, sc
        self.k, self.v = sc.k_pool, sc.v_pool          # appended in place: the scenario is not reused afterwards
        for b in sc.batches:
            oracle.kv_append(self.k, self.v, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)

    def sample(self, it: int, prefill_stride: int):
        """All decode rows and every `prefill_stride`-th prefill row of iteration `it`.
        Returns (seconds, sampled visible pairs, total visible pairs, T, rows run)."""
        b = self.sc.batches[it]
        qs = b.q_start()
        rows, pairs_s, pairs_t = [], 0, 0
        for s in range(b.num_seqs):
            lq, lc = int(b.query_len[s]), int(b.context_len[s])
            idx = np.arange(lq)
            p = lc - lq + idx + 1
            pairs_t += int(p.sum())
            keep = idx if lq == 1 else idx[::prefill_stride]
            rows.append(qs[s] + keep)
            pairs_s += int(p[keep].sum())
        rows = np.concatenate(rows).astype(np.int64)
        t0 = time.perf_counter()
        self.oracle.mixed_attention(b.q, self.k, self.v, b.block_table, b.context_len, b.query_len, rows=rows)
        return time.perf_counter() - t0, pairs_s, pairs_t, b.total_q, len(rows)


def _stride_for(ow: "OracleWorkload", it: int, seconds: float):
    """Calibrates on a thin sample and picks the prefill-row stride whose sample takes about `seconds`."""
    ow.sample(it, 256)                                  # touch the pages once, untimed
    dt, ps, pt, _, _ = ow.sample(it, 256)
    rate = ps / max(dt, 1e-6)                           # visible pairs per second
    for stride in (1, 2, 4, 8, 16, 32, 64, 128):
        # pairs of the sample at this stride ~ decode pairs + prefill pairs / stride; bounded by the thin sample's own figure
        est = ps + (pt - ps) * (256.0 / stride - 1.0) / 255.0
        if est / rate <= seconds:
            return stride
    return 256


def cpu_baseline(sc: syn.Scenario, seconds: float = 15.0):
    ow = OracleWorkload(sc)
    stride = _stride_for(ow, 0, seconds)
    dt, ps, pt, T, nrows = ow.sample(0, stride)
    full = dt * pt / ps
    return {"value": T / full, "unit": UNIT, "cores": ow.oracle.num_threads(), "kind": "oracle",
            "sample": f"iteration 0: all decode rows + every {stride}th prefill row ({nrows} of {T} rows, "
                      f"{ps / pt:.4f} of the visible (query,key) pairs) in {dt:.2f} s; whole-step time extrapolated by pair count"}


def run_reference(args):
    """The fp64 oracle as the reference arm: each step is a bounded sample of the step's rows, sized
    from a calibration pass so that the whole run stays within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ow = OracleWorkload(syn.config4_agentic())
    n_it = len(ow.sc.batches)
    stride = _stride_for(ow, 0, 100.0 / max(1, args.steps + args.warmup))
    times, toks = [], []
    for i in range(args.warmup + args.steps):
        dt, ps, pt, T, nrows = ow.sample(i % n_it, stride)
        if i >= args.warmup:
            times.append(dt * pt / ps)
            toks.append(T)
    total = sum(times)
    value = sum(toks) / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": ow.oracle.num_threads(), "kind": "oracle",
                             "sample": f"per step: all decode rows + every {stride}th prefill row; "
                                       "step time extrapolated by visible-pair count"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ main arm
def reduce_max(value: float, dist, device) -> float:
    """Max over ranks of a host float (identity when not distributed)."""
    if dist is None or not dist.is_initialized():
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# (name, scenario, variant of the layer): the other workload configurations, and two configurations again as a
# sliding-window layer with sinks and on an fp8 cache (rooflines against the bytes / FLOPs those variants need)
PER_CONFIG = [("configs[1] decode-only", lambda: syn.config2_decode_only(), {}),
              ("configs[2] chat-like", lambda: syn.config3_chat(), {}),
              ("configs[2] chat-like, one TP4 rank's shard (8 q heads, 2 kv heads)", lambda: syn.config3_chat_tp4_shard(), {}),
              ("configs[4] sweep, budget 0", lambda: syn.config5_sweep_point(0, 0), {}),
              ("configs[4] sweep, budget 512 x 4 prompts", lambda: syn.config5_sweep_point(512, 4), {}),
              ("configs[4] sweep, budget 2048 x 1 prompt", lambda: syn.config5_sweep_point(2048, 1), {}),
              ("configs[4] sweep, budget 8192 x 1 prompt", lambda: syn.config5_sweep_point(8192, 1), {}),
              ("configs[4] sweep, budget 8192 x 4 prompts", lambda: syn.config5_sweep_point(8192, 4), {}),
              ("configs[3] agentic as a sliding-window layer (window 4096) with sinks", lambda: syn.config4_agentic(),
               {"window": 4096, "sinks": True}),
              ("configs[1] decode-only on an fp8 (e4m3) cache", lambda: syn.config2_decode_only(), {"fp8": True}),
              ("configs[4] sweep, budget 0, on an fp8 (e4m3) cache", lambda: syn.config5_sweep_point(0, 0), {"fp8": True})]


def measure_config(torch, cf, ctx, sc, stream, peaks, clk, steps: int, repeats: int, variant=None):
    """Default-sequence and serial-sequence step times (median of `repeats` regions of `steps` steps) and the
    per-kernel figures of one workload."""
    wl = DeviceWorkload(sc, torch, cf, ctx, **(variant or {}))
    n_it = len(sc.batches)
    for i in range(max(3, n_it)):
        wl.step(i, stream)
    reps = time_repeats(torch, lambda i: wl.step(i, stream), steps, stream, repeats, clk)
    cf.cf_set_overlap(ctx, 0)
    for i in range(max(3, n_it)):
        wl.step(i, stream)
    reps_serial = time_repeats(torch, lambda i: wl.step(i, stream), steps, stream, max(3, repeats // 2), clk)
    cf.cf_set_overlap(ctx, 1)
    kern, _ = measure_kernels(torch, cf, wl, steps, stream, peaks, clk)
    host = measure_host_time(torch, cf, wl, min(steps, 4 * n_it), stream)
    toks = sum(wl.tokens(i) for i in range(steps)) / steps
    ms = median_of(reps)
    region = [r["sm_mhz"] for r in reps if r["sm_mhz"]]
    apply_peak_rule(kern, float(np.median(region)) if region else None, peaks)
    row = {"ms_per_step": ms, "ms_per_step_min": min(r["ms_per_step"] for r in reps), "ms_per_step_serial": median_of(reps_serial),
           "query_tokens_per_s": toks / (ms * 1e-3), "steps": steps, "repeats": len(reps),
           "sm_mhz": float(np.median([r["sm_mhz"] for r in reps if r["sm_mhz"]])) if any(r["sm_mhz"] for r in reps) else None,
           "kernels": kern, "host_us_per_call": host}
    del wl
    torch.cuda.empty_cache()
    return row


def run_ours(args):
    import torch
    import paper_2609_27085_b200 as cf

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    device = torch.device("cuda", local)
    peaks = load_peaks()
    ctx = cf.cf_create(local)
    sc = syn.config4_agentic(k=rank % 3)
    wl = DeviceWorkload(sc, torch, cf, ctx)
    stream = torch.cuda.current_stream()
    steps, warmup, repeats = args.steps, max(3, args.warmup), max(1, args.repeats)

    for i in range(warmup):
        wl.step(i, stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    launches = 0

    def one(i):
        nonlocal launches
        launches += wl.step(i, stream)

    with ClockSampler(local, period_s=args.clock_period_ms * 1e-3) as clk:
        # per-kernel times before the long timed region, while the GPU is not yet held at its power cap: what the
        # kernels do at the idle clock (the figures after the region, below, are the sustained ones)
        kern_start, _ = measure_kernels(torch, cf, wl, min(steps, 8), stream, peaks, clk)
        for i in range(2):
            wl.step(i, stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        launches = 0
        t_first = time.perf_counter()
        reps = time_repeats(torch, one, steps, stream, repeats, clk)
        t_last = time.perf_counter()
        if dist is not None:
            dist.barrier()
        launches_per_region = launches // repeats
        # every repeat is a region of exactly `steps` steps; the slowest rank decides each of them
        for r in reps:
            r["ms_per_step"] = reduce_max(r["ms_per_step"], dist, device)
        ms_step = median_of(reps)
        tokens_per_step = sum(wl.tokens(i) for i in range(steps)) / steps
        value = world * tokens_per_step / (ms_step * 1e-3)
        clocks = clk.summary(t_first, t_last)

        # the same steps as the serial sequence (decode -> combine -> prefill on the caller's stream alone)
        side_reps = max(3, repeats // 3)
        cf.cf_set_overlap(ctx, 0)
        for i in range(3):
            wl.step(i, stream)
        ms_serial = reduce_max(median_of(time_repeats(torch, lambda i: wl.step(i, stream), steps, stream, side_reps, clk)), dist, device)
        cf.cf_set_overlap(ctx, 1)
        # the same steps as replays of captured graphs of the planned calls (plan once per iteration, launch per layer)
        graphs, plans = wl.capture_graphs()
        for i in range(3):
            graphs[i % len(graphs)].replay()
        ms_graph = reduce_max(median_of(time_repeats(torch, lambda i: graphs[i % len(graphs)].replay(), steps, stream, side_reps, clk)),
                              dist, device)
        del graphs
        for pl in plans:
            cf.cf_plan_destroy(pl)
        # per-kernel times on the launching stream (serial sequence), same steps
        kern, _ = measure_kernels(torch, cf, wl, steps, stream, peaks, clk)
        host = measure_host_time(torch, cf, wl, min(steps, 16), stream)
        # end to end: host buffers in, host result out, every step
        for i in range(3):
            wl.step_host(i, stream)
        cf.cf_host_steps_flush(ctx, stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()

        def host_step(i):
            wl.step_host(i, stream)
            if i == steps - 1:
                cf.cf_host_steps_flush(ctx, stream)          # the last read-backs are inside the timed region

        ms_e2e = reduce_max(median_of(time_repeats(torch, host_step, steps, stream, side_reps, clk)), dist, device)
        assert cf.cf_get_async_status(ctx) == cf.CF_OK
        g = sc.geom
        T = wl.tokens(0)
        h2d = T * (g.num_q_heads + 2 * g.num_kv_heads) * g.head_dim * 2
        d2h = T * g.num_q_heads * g.head_dim * 2
        del wl
        torch.cuda.empty_cache()

        per_config = None
        if rank == 0 and world == 1 and not args.no_per_config:
            per_config = {}
            pc_repeats = max(3, min(5, repeats))
            for name, make, variant in PER_CONFIG:
                if args.only_config and args.only_config not in name:
                    continue
                scn = make()
                n_it = len(scn.batches)
                per_config[name] = measure_config(torch, cf, ctx, scn, stream, peaks, clk, steps=max(8, 4 * n_it),
                                                  repeats=pc_repeats, variant=variant)
                del scn

    if rank == 0:
        apply_peak_rule(kern, clocks.get("sm_mhz"), peaks)
        dominant = "prefill" if kern.get("prefill", {}).get("ms", 0) >= kern.get("decode", {}).get("ms", 0) else "decode"
        roof = {k: kern[dominant].get(k) for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "frac_of_nominal",
                                                   "frac_of_burst", "frac_of_sustained", "tflops_per_ghz")}
        roof["kernel"] = "prefill_tc_kernel" if dominant == "prefill" else "decode_splitk_kernel (merge of the partials fused in)"
        roof["peak_source"] = peaks["source"] + ((" bf16, " + kern["prefill"]["peak_kind"]) if dominant == "prefill" else " copy")
        roof["sequence"] = "serial (per-kernel events need kernels that do not overlap; `value` runs the default sequence)"
        mhz = [r["sm_mhz"] for r in reps if r["sm_mhz"]]
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
                "ms_per_step": ms_step, "ms_per_step_min": min(r["ms_per_step"] for r in reps),
                "ms_per_step_first": reps[0]["ms_per_step"], "repeats": len(reps),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "l2": "inputs larger than L2: ~1.3 GB of paged K/V streamed per step",
                           "replicas": world},
                "roofline": roof,
                "kernels": {"decode": kern.get("decode"), "prefill": kern.get("prefill"), "sequence": "serial",
                            "ms_decode": kern["ms_decode"], "ms_combine": kern["ms_combine"], "ms_prefill": kern["ms_prefill"],
                            "sm_mhz": kern.get("sm_mhz")},
                "kernels_at_start": {"decode": kern_start.get("decode"), "prefill": kern_start.get("prefill"), "sequence": "serial",
                                     "sm_mhz": kern_start.get("sm_mhz"),
                                     "note": "the same per-kernel measurement taken before the timed repeats (few steps, "
                                             "GPU not yet at its power cap)"},
                "e2e": {"value": world * tokens_per_step / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
                "serial": {"value": world * tokens_per_step / (ms_serial * 1e-3), "unit": UNIT, "ms_per_step": ms_serial,
                           "note": "cf_set_overlap(0): decode -> prefill one after the other; `value` is the "
                                   "library's default sequence (prefill CTAs beside decode, joined per call)"},
                "planned_graph": {"value": world * tokens_per_step / (ms_graph * 1e-3), "unit": UNIT, "ms_per_step": ms_graph,
                                  "note": "cf_plan_create once per chunk iteration; cf_kv_append_planned + "
                                          "cf_mixed_attention_planned captured in a CUDA graph and replayed per step"},
                "host_us_per_call": host,
                "repeat_list": [{"ms_per_step": round(r["ms_per_step"], 5), "sm_mhz": r["sm_mhz"], "watts": r["watts"],
                                 "ms_x_ghz": (round(r["ms_per_step"] * r["sm_mhz"] / 1e3, 5) if r["sm_mhz"] else None)} for r in reps],
                "gpu_launches": launches_per_region, "clocks": clocks}
        if mhz:
            line["clocks"]["sm_mhz_per_repeat_min"] = min(mhz)
            line["clocks"]["sm_mhz_per_repeat_max"] = max(mhz)
        if per_config is not None:
            line["per_config"] = per_config
        if world == 1:
            line["cpu_baseline"] = cpu_baseline(sc)
        print(json.dumps(line), flush=True)
    cf.cf_destroy(ctx)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def small_case(name: str) -> syn.Scenario:
    """Reduced workloads for profiler captures (inputs still larger than L2 for the decode case,
    under 1.5 GB on the device)."""
    if name == "decode_small":
        geom = syn.Geometry(32, 8, 128, 16, 16384)
        lens = syn.uniform_int(np.random.default_rng(42), 32, 2048, 6144)
        return syn.scenario_from_lengths(name, geom, 43, lens - 1, [[1] * 32])
    if name == "decode_small_fp8":   # the same lengths on an fp8 (e4m3) cache (run_case converts the pools)
        geom = syn.Geometry(32, 8, 128, 16, 16384)
        lens = syn.uniform_int(np.random.default_rng(42), 32, 2048, 6144)
        return syn.scenario_from_lengths(name, geom, 43, lens - 1, [[1] * 32])
    if name == "prefill_small":
        geom = syn.Geometry(32, 8, 128, 16, 4096)
        return syn.scenario_from_lengths(name, geom, 44, [3072], [[1024]])
    if name == "prefill_multi":      # 32 q tiles x 16 head pairs = 512 items: every persistent CTA works through 3-4 of them
        geom = syn.Geometry(32, 8, 128, 16, 16384)
        return syn.scenario_from_lengths(name, geom, 45, [8192], [[4096]])
    if name == "agentic_small":      # the headline's first chunk iteration (2048 new over 24,576 cached) beside 4 decode sequences, in a pool of 1 GB
        geom = syn.Geometry(32, 8, 128, 16, 8192)
        return syn.scenario_from_lengths(name, geom, 46, [24576, 20000, 9000, 30000, 12000], [[2048, 1, 1, 1, 1]])
    raise SystemExit(f"unknown case {name}")


def run_shared_prefix_case(args):
    """16 decode sequences (Hq 32, Hkv 8, D 128) that share an 8192-token prefix and have 200..900 tokens of their
    own: the same batch through cf_mixed_attention (every sequence streams the shared pages) and through
    cf_mixed_attention_shared (the shared pages are streamed once per set of four sequences).  `--variant plain`
    or `--variant shared` runs only that one (for a profiler capture)."""
    import torch
    import paper_2609_27085_b200 as cf
    torch.cuda.set_device(0)
    geom = syn.Geometry(32, 8, 128, 16, 16384)
    rng = np.random.default_rng(7)
    own = [int(x) for x in rng.integers(200, 900, size=16)]
    sc, sg, sl = syn.shared_prefix_scenario("shared_prefix", geom, 47, 8192, own, [1] * 16, [0] * 16)
    b = sc.batches[0]
    ctx = cf.cf_create(0)
    wl = DeviceWorkload(sc, torch, cf, ctx)
    it = wl.its[0]
    stream = torch.cuda.current_stream()
    wl.step(0, stream)                                               # append once
    per_tok = geom.kv_bytes_per_token()
    bytes_plain = int(sum(int(x) for x in b.context_len) * per_tok)
    bytes_dedup = int((8192 + sum(int(x) - 8192 for x in b.context_len)) * per_tok)
    res = {"case": "shared_prefix", "kv_bytes_every_sequence": bytes_plain, "kv_bytes_shared_once": bytes_dedup}

    def plain(i):
        cf.cf_mixed_attention(ctx, wl.desc, it["q"], wl.k, wl.v, it["bt"], b.max_blocks, b.context_len, b.query_len,
                              it["out"], None, stream=stream)

    def shared(i):
        cf.cf_mixed_attention_shared(ctx, wl.desc, it["q"], wl.k, wl.v, it["bt"], b.max_blocks, b.context_len, b.query_len,
                                     sg, sl, it["out"], None, stream=stream)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # larger than L2: every timed call starts cold
    for name, fn in (("plain", plain), ("shared", shared)):
        if args.variant not in ("both", name):
            continue
        for i in range(args.warmup):
            fn(i)
        ts = []
        for i in range(args.steps):
            flush.zero_()
            ts.append(time_region(torch, fn, 1, stream))
        res[name] = {"ms": float(np.median(ts)), "ms_min": float(min(ts)),
                     "effective_gbs_of_all_sequences": bytes_plain / (float(np.median(ts)) * 1e-3) / 1e9,
                     "plan_counts": [int(x) for x in cf.cf_get_last_plan_counts(ctx)]}
    assert cf.cf_get_async_status(ctx) == cf.CF_OK
    print(json.dumps(res), flush=True)
    del wl
    cf.cf_destroy(ctx)


def run_case(args):
    """Runs one reduced workload for `warmup + steps` steps and prints its per-kernel times."""
    if args.case == "shared_prefix":
        return run_shared_prefix_case(args)
    import torch
    import paper_2609_27085_b200 as cf
    torch.cuda.set_device(0)
    peaks = load_peaks()
    ctx = cf.cf_create(0)
    if args.pairs:
        cf.cf_set_debug_option(ctx, cf.CF_DEBUG_PREFILL_PAIRS, 1)
    wl = DeviceWorkload(small_case(args.case), torch, cf, ctx, fp8=args.case.endswith("_fp8"))
    stream = torch.cuda.current_stream()
    for i in range(args.warmup):
        wl.step(i, stream)
    kern, launches = measure_kernels(torch, cf, wl, args.steps, stream, peaks)
    host = measure_host_time(torch, cf, wl, min(args.steps, 8), stream)
    torch.cuda.synchronize()
    print(json.dumps({"case": args.case, "pairs": bool(args.pairs), "steps": args.steps, "kernels": kern, "host_us_per_call": host, "gpu_launches": launches}),
          flush=True)
    del wl
    cf.cf_destroy(ctx)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None,
                    help="run a reduced workload (decode_small | decode_small_fp8 | prefill_small | prefill_multi | agentic_small | shared_prefix) and exit")
    ap.add_argument("--pairs", action="store_true", help="reduced workloads: chunked prefill on the two-CTA (cta_group::2) kernel")
    ap.add_argument("--variant", default="both", choices=["both", "plain", "shared"], help="shared_prefix case: which entry point")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--repeats", type=int, default=15, help="how many times the timed region of --steps steps is repeated")
    ap.add_argument("--clock-period-ms", type=float, default=10.0, help="sampling period of the SM clock (NVML, read-only)")
    ap.add_argument("--only-config", default=None, help="with per_config: measure only the configurations whose name contains this")
    ap.add_argument("--no-per-config", action="store_true", help="skip the per_config block (the other workload configurations)")
    args = ap.parse_args()
    if args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
