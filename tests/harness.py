"""Shared plumbing for the GPU parity tests: runs one scenario through the CUDA library (via the
C ABI) and through the CPU oracle on the same seeded inputs and compares them.

Tolerances (bf16 inputs, fp32 accumulation, one bf16 rounding of the output), per batch:
    max |O_gpu - O_oracle| <= 2e-2     mean |O_gpu - O_oracle| <= 2e-3
and, because those bounds are loose at long context (one lost key moves O by less than 2e-2 at a
context of 4096), also
    max |lse_gpu - lse_oracle| <= LSE_TOL = 1e-5  (lse never passes through bf16; a lost key moves it by >= 3e-4)
    error ratio: max/mean error relative to the oracle's own bf16 rounding error <= 4 / 2.
"""
from __future__ import annotations

import numpy as np
import torch

import cf_synth as syn
import oracle
import paper_2609_27085_b200 as cf

MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3
LSE_TOL = 1e-5


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class GpuScenario:
    """Device copy of a scenario's pools plus a library context."""

    def __init__(self, sc: syn.Scenario, ctx=None, softmax_scale: float = 0.0, layout: str = "HND", debug=None,
                 window: int = 0, sinks=None, fp8=None):
        """debug: {CF_DEBUG_* option: value} applied to a context created here (test-only planner switches).
        window / sinks: the sliding-window and attention-sink variant (sinks: host fp32 array [Hq]).
        fp8: (k_scale, v_scale) host fp32 arrays [Hkv]: the cache is an e4m3 cache; the scenario's bf16 prefix is
        quantised on the host by the oracle's encoder (NaN sentinels stay NaN codes)."""
        self.geom = g = sc.geom
        self.fp8 = fp8
        self.sinks_dev = None if sinks is None else torch.from_numpy(np.ascontiguousarray(sinks, dtype=np.float32)).cuda()
        variant = dict(window_size=window, sink_logits=self.sinks_dev)
        self.layout = layout
        self.own_ctx = ctx is None
        self.ctx = cf.cf_create(0) if ctx is None else ctx
        for opt, val in (debug or {}).items():
            cf.cf_set_debug_option(self.ctx, opt, val)
        if fp8 is not None:
            assert layout == "HND"
            self.k_scale = np.ascontiguousarray(fp8[0], dtype=np.float32)
            self.v_scale = np.ascontiguousarray(fp8[1], dtype=np.float32)
            self.k_scale_dev, self.v_scale_dev = torch.from_numpy(self.k_scale).cuda(), torch.from_numpy(self.v_scale).cuda()
            self.k = torch.from_numpy(quantise_pool(sc.k_pool, self.k_scale)).cuda()
            self.v = torch.from_numpy(quantise_pool(sc.v_pool, self.v_scale)).cuda()
            self.desc = cf.make_desc(g.num_q_heads, g.num_kv_heads, g.head_dim, g.block_size, g.num_blocks,
                                     softmax_scale=softmax_scale, kv_dtype=cf.CF_KV_FP8_E4M3, k_scale=self.k_scale_dev,
                                     v_scale=self.v_scale_dev, **variant)
        elif layout == "HND":
            self.k = to_dev_bf16(sc.k_pool)
            self.v = to_dev_bf16(sc.v_pool)
            self.desc = cf.make_desc(g.num_q_heads, g.num_kv_heads, g.head_dim, g.block_size, g.num_blocks,
                                     softmax_scale=softmax_scale, **variant)
        else:  # NHD: [NB, B, Hkv, D] storage
            self.k = to_dev_bf16(np.ascontiguousarray(sc.k_pool.transpose(0, 2, 1, 3)))
            self.v = to_dev_bf16(np.ascontiguousarray(sc.v_pool.transpose(0, 2, 1, 3)))
            H, B, D = g.num_kv_heads, g.block_size, g.head_dim
            st = (B * H * D, D, H * D)
            self.desc = cf.make_desc(g.num_q_heads, g.num_kv_heads, g.head_dim, g.block_size, g.num_blocks,
                                     k_strides=st, v_strides=st, softmax_scale=softmax_scale, **variant)

    def pools_host(self):
        if self.fp8 is not None:
            return self.k.cpu().numpy(), self.v.cpu().numpy()
        k, v = to_host_bits(self.k), to_host_bits(self.v)
        if self.layout != "HND":
            k, v = k.transpose(0, 2, 1, 3), v.transpose(0, 2, 1, 3)
        return k, v

    def append(self, b: syn.Batch):
        bt = torch.from_numpy(b.block_table).cuda()
        cf.cf_kv_append(self.ctx, self.desc, self.k, self.v, to_dev_bf16(b.k_new), to_dev_bf16(b.v_new), bt,
                        b.max_blocks, b.context_len, b.query_len)
        torch.cuda.synchronize()

    def attend(self, b: syn.Batch, want_lse: bool = True, poison: bool = True):
        g = self.geom
        bt = torch.from_numpy(b.block_table).cuda()
        q = to_dev_bf16(b.q)
        T = b.total_q
        out = torch.full((T, g.num_q_heads, g.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda") if poison \
            else torch.empty((T, g.num_q_heads, g.head_dim), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((T, g.num_q_heads), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
        cf.cf_mixed_attention(self.ctx, self.desc, q, self.k, self.v, bt, b.max_blocks, b.context_len, b.query_len,
                              out, lse)
        torch.cuda.synchronize()
        assert cf.cf_get_async_status(self.ctx) == cf.CF_OK
        return to_host_bits(out), (lse.cpu().numpy() if want_lse else None)

    def close(self):
        if self.own_ctx and self.ctx is not None:
            cf.cf_destroy(self.ctx)
            self.ctx = None


def quantise_pool(pool_bits: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """bf16 pool [NB, Hkv, B, D] -> e4m3 codes of value / scale[head] (the oracle's encoder; fp32 division)."""
    vals = syn.bf16_bits_to_f32(pool_bits) / np.asarray(scale, dtype=np.float32)[None, :, None, None]
    return oracle.e4m3_encode(vals.astype(np.float32))


def compare(o_bits: np.ndarray, lse: np.ndarray, ref_o: np.ndarray, ref_lse: np.ndarray, rows=None, label=""):
    """Element-by-element comparison against the oracle (on `rows` if given)."""
    o = syn.bf16_bits_to_f64(o_bits if rows is None else o_bits[rows])
    assert np.isfinite(o).all(), f"{label}: non-finite output"
    err = np.abs(o - ref_o)
    own = np.abs(syn.bf16_bits_to_f64(syn.f32_to_bf16_bits(ref_o.astype(np.float32))) - ref_o)
    stats = {"max_abs": float(err.max()), "mean_abs": float(err.mean()),
             "ratio_max": float(err.max() / max(own.max(), 1e-30)), "ratio_mean": float(err.mean() / max(own.mean(), 1e-30))}
    assert stats["max_abs"] <= MAX_ABS_TOL, f"{label}: {stats}"
    assert stats["mean_abs"] <= MEAN_ABS_TOL, f"{label}: {stats}"
    assert stats["ratio_max"] <= 4.0 and stats["ratio_mean"] <= 2.0, f"{label}: {stats}"
    if lse is not None:
        l = lse if rows is None else lse[rows]
        assert np.isfinite(l).all(), f"{label}: non-finite lse"
        stats["lse_max"] = float(np.abs(l.astype(np.float64) - ref_lse).max())
        assert stats["lse_max"] <= LSE_TOL, f"{label}: {stats}"
    return stats


def run_and_check(sc: syn.Scenario, max_prefill_rows: int = 0, layout: str = "HND", softmax_scale: float = 0.0,
                  check_append: bool = True, ctx=None, debug=None, tile_rows: bool = False, window: int = 0, sinks=None,
                  fp8=None):
    """Every iteration of the scenario: append + attention on both sides, compare.
    Rows compared: all of them, or (max_prefill_rows) a thinned sample per prefill sequence, or (tile_rows) the
    first and last row of every 128-row q tile plus every 41st row of each prefill sequence, all heads."""
    gpu = GpuScenario(sc, ctx=ctx, softmax_scale=softmax_scale, layout=layout, debug=debug, window=window, sinks=sinks, fp8=fp8)
    scales = {}
    if fp8 is None:
        k_ref, v_ref = sc.k_pool.copy(), sc.v_pool.copy()
    else:
        k_ref, v_ref = quantise_pool(sc.k_pool, gpu.k_scale), quantise_pool(sc.v_pool, gpu.v_scale)
        scales = dict(k_scale=gpu.k_scale, v_scale=gpu.v_scale)
    all_stats = []
    try:
        for b in sc.batches:
            gpu.append(b)
            oracle.kv_append(k_ref, v_ref, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len, **scales)
            if check_append:
                kg, vg = gpu.pools_host()
                assert np.array_equal(kg, k_ref) and np.array_equal(vg, v_ref), f"{b.label}: kv_append not bit-exact"
            o_bits, lse = gpu.attend(b)
            rows = syn.tile_edge_rows(b) if tile_rows else (syn.sample_rows(b, max_prefill_rows) if max_prefill_rows else None)
            ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len,
                                                    scale=(softmax_scale or None), rows=rows, window=window,
                                                    sinks=None if sinks is None else np.asarray(sinks, dtype=np.float32).astype(np.float64),
                                                    **scales)
            all_stats.append(compare(o_bits, lse, ref_o, ref_lse, rows=rows, label=b.label))
    finally:
        gpu.close()
    return all_stats
