#!/usr/bin/env python
"""Benchmark of the mixed decode + chunked-prefill paged-attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--report]

One *step* = one unit of one layer of the chat-like mixed batch: cf_kv_append followed by
cf_mixed_attention (split-K decode with its merge, chunked prefill) over 48 decode sequences
(lognormal contexts, median 4096) plus two 512-token prefill chunks that sit on 6144 + 512*t
cached tokens; steps cycle through the four chunks t = 0..3 of the 2048-token prompts.
Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank runs
an independent replica of the batch on its own GPU: the path has no exchange step, so there is no
data-path collective; the only collective is the max-over-ranks of the device time.
`value` is measured in the library's default launch sequence (for this batch: a first grid of
prefill CTAs beside decode); the `serial` key repeats the steps with one kernel after the other,
which is also the sequence the per-kernel times under `kernels` / `roofline` are taken in.

`--impl reference` times the fp64 CPU oracle (as it stands) on the host cores instead.
`--report` additionally writes a per-configuration table (all five workload configurations) to
bench_report.json under $CF_REPORT_DIR (default: ./bench_out).
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
WORKLOAD = ("configs[2] chat-like mixed batch: 48 decode seqs (lognormal ctx, median 4096, sigma 0.8, clip [128,16384]) "
            "+ 2 prefills of 2048 new tokens over 6144 cached, 512-token chunks; Hq 32, Hkv 8, D 128, block 16, bf16; "
            "one step = kv_append + mixed attention of one chunk iteration (t cycles 0..3)")
# DRAM traffic per algorithmic byte of the split-K decode kernel, from an ncu capture on the reduced
# decode case (dram bytes read + written: 560.9 MB for 555.2 MB algorithmic); traffic grows in
# proportion to the K/V bytes, so a full launch is scaled by its algorithmic bytes.
DECODE_TRAFFIC_RATIO = 1.010
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    except Exception:
        return dict(FALLBACK_PEAKS, source="fallback")


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, torch_device_index: int, period_s: float = 0.005):
        self.period = period_s
        self.samples = []
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
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
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

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------ device workload
class DeviceWorkload:
    """A scenario resident on the GPU: pools, block table, per-iteration inputs."""

    def __init__(self, sc: syn.Scenario, torch, cf, ctx):
        self.sc, self.torch, self.cf, self.ctx = sc, torch, cf, ctx
        g = sc.geom
        self.desc = cf.make_desc(g.num_q_heads, g.num_kv_heads, g.head_dim, g.block_size, g.num_blocks)

        def dev(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

        self.k, self.v = dev(sc.k_pool), dev(sc.v_pool)
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


def batch_accounting(sc: syn.Scenario):
    acc = []
    for b in sc.batches:
        acc.append({"tokens": b.total_q,
                    "decode_bytes": syn.decode_algorithmic_bytes(b.geom, b.context_len, b.query_len),
                    "decode_flops": syn.decode_flops(b.geom, b.context_len, b.query_len),
                    "prefill_flops": syn.prefill_flops(b.geom, b.context_len, b.query_len)})
    return acc


# nominal chip figures (HGX B200: 7.7 TB/s HBM3e, 2.25 PFLOP/s dense bf16), reported beside the measured peaks
NOMINAL_HBM_GBS = 7700.0
NOMINAL_BF16_TFLOPS = 2250.0


def measure_kernels(torch, cf, wl: DeviceWorkload, steps: int, stream, peaks):
    """Per-kernel CUDA-event times (inside the library, on the launching stream) over `steps` steps."""
    acc = batch_accounting(wl.sc)
    cf.cf_set_timing(wl.ctx, True)
    launches = 0
    for i in range(steps):
        launches += wl.step(i, stream)
    ms_dec, ms_comb, ms_pre, n = cf.cf_get_timing_sums(wl.ctx)
    cf.cf_set_timing(wl.ctx, False)
    dec_bytes = sum(acc[i % len(acc)]["decode_bytes"] for i in range(steps))
    pre_flops = sum(acc[i % len(acc)]["prefill_flops"] for i in range(steps))
    out = {"ms_decode": ms_dec / steps, "ms_combine": ms_comb / steps, "ms_prefill": ms_pre / steps}
    if ms_dec > 0:
        gbs = dec_bytes / ((ms_dec + ms_comb) * 1e-3) / 1e9
        out["decode"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
                         "traffic": DECODE_TRAFFIC_RATIO * dec_bytes / steps,
                         "bytes_per_launch": dec_bytes / steps, "ms": (ms_dec + ms_comb) / steps}
    if ms_pre > 0:
        tf = pre_flops / (ms_pre * 1e-3) / 1e12
        out["prefill"] = {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                          "frac": tf / peaks["bf16_tflops"], "frac_of_nominal": tf / NOMINAL_BF16_TFLOPS, "traffic": None,
                          "flops_per_launch": pre_flops / steps, "ms": ms_pre / steps}
    return out, launches


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


def cpu_baseline(sc: syn.Scenario, prefill_stride: int = 4):
    ow = OracleWorkload(sc)
    ow.sample(0, 64)                                   # touch the pages once, untimed
    dt, ps, pt, T, nrows = ow.sample(0, prefill_stride)
    full = dt * pt / ps
    return {"value": T / full, "unit": UNIT, "cores": ow.oracle.num_threads(), "kind": "oracle",
            "sample": f"iteration 0: all decode rows + every {prefill_stride}th prefill row ({nrows} of {T} rows, "
                      f"{ps / pt:.3f} of the visible (query,key) pairs) in {dt:.2f} s; whole-step time extrapolated by pair count"}


def run_reference(args):
    """The fp64 oracle as the reference arm: each step is a bounded sample of the step's rows, sized
    from a calibration pass so that the whole run stays within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ow = OracleWorkload(syn.config3_chat())
    n_it = len(ow.sc.batches)
    dt, ps, pt, _, _ = ow.sample(0, 64)                # page-touching pass
    dt, ps, pt, _, _ = ow.sample(0, 64)
    budget = 120.0 / max(1, args.steps + args.warmup)
    stride = 64
    for cand in (4, 8, 16, 32):
        est_pairs = ps + (pt - ps) * (64.0 / cand - 1.0) / 63.0 if cand < 64 else ps
        if dt * est_pairs / ps <= budget:
            stride = cand
            break
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
    peaks = load_peaks()
    ctx = cf.cf_create(local)
    sc = syn.config3_chat(k=rank % 3)
    wl = DeviceWorkload(sc, torch, cf, ctx)
    stream = torch.cuda.current_stream()
    steps, warmup = args.steps, max(3, args.warmup)

    for i in range(warmup):
        wl.step(i, stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    launches = 0

    def one(i):
        nonlocal launches
        launches += wl.step(i, stream)

    with ClockSampler(local) as clk:
        ms = time_region(torch, one, steps, stream)
    if dist is not None:
        dist.barrier()
    ms = reduce_max(ms, dist, torch.device("cuda", local))
    tokens = sum(wl.tokens(i) for i in range(steps))
    value = world * tokens / (ms * 1e-3)

    # the same steps as the serial sequence (decode -> combine -> prefill on the caller's stream alone)
    cf.cf_set_overlap(ctx, 0)
    for i in range(3):
        wl.step(i, stream)
    ms_serial = reduce_max(time_region(torch, lambda i: wl.step(i, stream), steps, stream), dist, torch.device("cuda", local))
    cf.cf_set_overlap(ctx, 1)
    # the same steps as replays of captured graphs of the planned calls (plan once per iteration, launch per layer)
    graphs, plans = wl.capture_graphs()
    for i in range(3):
        graphs[i % len(graphs)].replay()
    ms_graph = reduce_max(time_region(torch, lambda i: graphs[i % len(graphs)].replay(), steps, stream), dist,
                          torch.device("cuda", local))
    del graphs
    for pl in plans:
        cf.cf_plan_destroy(pl)
    # per-kernel times on the launching stream, same steps
    kern, _ = measure_kernels(torch, cf, wl, steps, stream, peaks)
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

    ms_e2e = time_region(torch, host_step, steps, stream)
    ms_e2e = reduce_max(ms_e2e, dist, torch.device("cuda", local))
    assert cf.cf_get_async_status(ctx) == cf.CF_OK
    g = sc.geom
    T = wl.tokens(0)
    h2d = T * (g.num_q_heads + 2 * g.num_kv_heads) * g.head_dim * 2
    d2h = T * g.num_q_heads * g.head_dim * 2

    if rank == 0:
        dominant = "prefill" if kern.get("prefill", {}).get("ms", 0) >= kern.get("decode", {}).get("ms", 0) else "decode"
        roof = {k: kern[dominant][k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "frac_of_nominal")}
        roof["kernel"] = "prefill_tc_kernel" if dominant == "prefill" else "decode_splitk_kernel (merge of the partials fused in)"
        roof["peak_source"] = peaks["source"] + (" burst bf16" if dominant == "prefill" else " copy")
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
                "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "l2": "inputs larger than L2: ~1.0 GB of paged K/V streamed per step",
                           "replicas": world},
                "roofline": roof,
                "kernels": {"decode": kern.get("decode"), "prefill": kern.get("prefill"),
                            "ms_decode": kern["ms_decode"], "ms_combine": kern["ms_combine"], "ms_prefill": kern["ms_prefill"]},
                "e2e": {"value": world * tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / steps},
                "serial": {"value": world * tokens / (ms_serial * 1e-3), "unit": UNIT, "ms_per_step": ms_serial / steps,
                           "note": "cf_set_overlap(0): decode -> prefill one after the other; `value` is the "
                                   "library's default sequence (prefill CTAs beside decode, joined per call); the per-kernel "
                                   "times under `kernels` are taken in the serial sequence"},
                "planned_graph": {"value": world * tokens / (ms_graph * 1e-3), "unit": UNIT, "ms_per_step": ms_graph / steps,
                                  "note": "cf_plan_create once per chunk iteration; cf_kv_append_planned + "
                                          "cf_mixed_attention_planned captured in a CUDA graph and replayed per step"},
                "gpu_launches": launches, "clocks": clk.summary()}
        if world == 1:
            line["cpu_baseline"] = cpu_baseline(sc)
        print(json.dumps(line), flush=True)
        if args.report:
            write_report(torch, cf, ctx, stream, peaks)
    del wl
    cf.cf_destroy(ctx)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def write_report(torch, cf, ctx, stream, peaks):
    """Per-configuration table over the workload configurations (device times only)."""
    rows = []
    scenarios = [("cfg2_decode", lambda: syn.config2_decode_only()), ("cfg3_chat", lambda: syn.config3_chat()),
                 ("cfg3_tp4_shard", lambda: syn.config3_chat_tp4_shard()), ("cfg4_agentic", lambda: syn.config4_agentic())]
    scenarios += [(f"cfg5_b{b}_n{n}", (lambda b=b, n=n: syn.config5_sweep_point(b, n))) for b, n in
                  [(0, 0), (512, 4), (2048, 1), (8192, 1), (8192, 4)]]
    only = [x for x in os.environ.get("CF_REPORT_ONLY", "").split(",") if x]
    for name, make in scenarios:
        if only and name not in only:
            continue
        sc = make()
        wl = DeviceWorkload(sc, torch, cf, ctx)
        n_it = len(sc.batches)
        for i in range(3 * n_it):
            wl.step(i, stream)
        steps = 5 * n_it
        ms = time_region(torch, lambda i: wl.step(i, stream), steps, stream)
        cf.cf_set_overlap(ctx, 0)
        for i in range(n_it):
            wl.step(i, stream)
        ms_serial = time_region(torch, lambda i: wl.step(i, stream), steps, stream)
        cf.cf_set_overlap(ctx, 1)
        kern, _ = measure_kernels(torch, cf, wl, steps, stream, peaks)
        toks = sum(wl.tokens(i) for i in range(steps))
        rows.append({"config": name, "ms_per_step": ms / steps, "ms_per_step_serial": ms_serial / steps,
                     "query_tokens_per_s": toks / (ms * 1e-3), **kern})
        del wl
        torch.cuda.empty_cache()
    out_dir = os.environ.get("CF_REPORT_DIR", os.path.join(ROOT, "bench_out"))
    os.makedirs(out_dir, exist_ok=True)
    with open(os.path.join(out_dir, "bench_report.json"), "w") as f:
        json.dump({"peaks": peaks, "rows": rows}, f, indent=1)
    for r in rows:
        d, p = r.get("decode"), r.get("prefill")
        print(f"# {r['config']:16s} step {r['ms_per_step'] * 1e3:8.1f} us (serial {r['ms_per_step_serial'] * 1e3:8.1f})  "
              f"{r['query_tokens_per_s']:12.0f} tok/s | "
              f"decode {r['ms_decode'] * 1e3:7.1f}+{r['ms_combine'] * 1e3:5.1f} us "
              f"{(d['achieved'] if d else 0):7.0f} GB/s ({(d['frac'] if d else 0):.2f}) | "
              f"prefill {r['ms_prefill'] * 1e3:8.1f} us {(p['achieved'] if p else 0):7.1f} TF/s ({(p['frac'] if p else 0):.2f})",
              file=sys.stderr, flush=True)


def small_case(name: str) -> syn.Scenario:
    """Reduced workloads for profiler captures (inputs still larger than L2 for the decode case,
    under 1.5 GB on the device)."""
    if name == "decode_small":
        geom = syn.Geometry(32, 8, 128, 16, 16384)
        lens = syn.uniform_int(np.random.default_rng(42), 32, 2048, 6144)
        return syn.scenario_from_lengths(name, geom, 43, lens - 1, [[1] * 32])
    if name == "prefill_small":
        geom = syn.Geometry(32, 8, 128, 16, 4096)
        return syn.scenario_from_lengths(name, geom, 44, [3072], [[1024]])
    if name == "prefill_multi":      # 32 q tiles x 16 head pairs = 512 items: every persistent CTA works through 3-4 of them
        geom = syn.Geometry(32, 8, 128, 16, 16384)
        return syn.scenario_from_lengths(name, geom, 45, [8192], [[4096]])
    raise SystemExit(f"unknown case {name}")


def run_case(args):
    """Runs one reduced workload for `warmup + steps` steps and prints its per-kernel times."""
    import torch
    import paper_2609_27085_b200 as cf
    torch.cuda.set_device(0)
    peaks = load_peaks()
    ctx = cf.cf_create(0)
    wl = DeviceWorkload(small_case(args.case), torch, cf, ctx)
    stream = torch.cuda.current_stream()
    for i in range(args.warmup):
        wl.step(i, stream)
    kern, launches = measure_kernels(torch, cf, wl, args.steps, stream, peaks)
    torch.cuda.synchronize()
    print(json.dumps({"case": args.case, "steps": args.steps, "kernels": kern, "gpu_launches": launches}), flush=True)
    del wl
    cf.cf_destroy(ctx)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, help="run a reduced workload (decode_small | prefill_small | prefill_multi) and exit")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--report", action="store_true")
    args = ap.parse_args()
    if args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
