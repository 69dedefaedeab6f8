"""Thin Python binding of libcrossflow_attn.so (argument marshalling only).

Every step of the path — KV append, split-K decode, combine, chunked prefill, the planner —
runs inside the CUDA library; this module converts tensors to pointers and checks statuses.
There is no CPU fallback: if the library is missing, loading raises.

Names mirror the C ABI (``include/crossflow_attn.h``): ``cf_create``, ``cf_kv_append``,
``cf_mixed_attention``, ``cf_mixed_step_host``, ``cf_get_async_status``, ``cf_set_timing``,
``cf_get_timing_sums``, ``cf_get_last_launch_count``, ``cf_plan_inspect``, ``cf_decode_attention_static``, ``cf_status_string``, ...

Device arguments may be torch tensors (their ``data_ptr()`` is used) or integer addresses; the
length arrays are host ``int32`` numpy arrays (anything array-like is converted).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcrossflow_attn.so")

CF_OK = 0
CF_ERR_INVALID_ARG = 1
CF_ERR_UNSUPPORTED = 2
CF_ERR_OUT_OF_RANGE = 3
CF_ERR_WORKSPACE = 4
CF_ERR_CUDA = 5
CF_ERR_TIMEOUT = 6
CF_ERR_ARCH = 7
CF_ERR_BUSY = 8

CF_KV_BF16 = 0
CF_KV_FP8_E4M3 = 1

# cf_debug_option (test-only switches)
CF_DEBUG_PREFILL_SPLIT = 0
CF_DEBUG_SEPARATE_COMBINE = 1
CF_DEBUG_DECODE_WAVES = 2
CF_DEBUG_DECODE_MIN_CHUNK_PAGES = 3
CF_DEBUG_SPATIAL_NO_WAIT = 4
CF_DEBUG_PREFILL_PAIRS = 5

EXPORTS = ("cf_create", "cf_destroy", "cf_kv_append", "cf_mixed_attention", "cf_mixed_step_host", "cf_host_steps_flush",
           "cf_get_async_status", "cf_set_timing", "cf_get_timing_sums", "cf_get_last_launch_count", "cf_plan_inspect",
           "cf_decode_attention_static", "cf_selftest_bounded_wait", "cf_set_overlap", "cf_plan_create", "cf_plan_destroy",
           "cf_kv_append_planned", "cf_mixed_attention_planned", "cf_estimate_us", "cf_validate_block_table", "cf_set_debug_option", "cf_get_host_time_sums", "cf_mixed_attention_shared", "cf_get_last_plan_counts", "cf_spatial_share",
           "cf_status_string")


class CacheDesc(ctypes.Structure):
    """Mirror of ``cf_cache_desc``."""
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("block_size", ctypes.c_int32), ("num_blocks", ctypes.c_int32),
                ("k_stride_block", ctypes.c_int64), ("k_stride_head", ctypes.c_int64), ("k_stride_token", ctypes.c_int64),
                ("v_stride_block", ctypes.c_int64), ("v_stride_head", ctypes.c_int64), ("v_stride_token", ctypes.c_int64),
                ("softmax_scale", ctypes.c_float), ("window_size", ctypes.c_int32), ("sink_logits", ctypes.c_void_p),
                ("kv_dtype", ctypes.c_int32), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p)]


class PlanOptions(ctypes.Structure):
    """Mirror of ``cf_plan_options`` (zero = default)."""
    _fields_ = [("num_sms", ctypes.c_int32), ("prefill_sms_mixed", ctypes.c_int32), ("prefill_force_split", ctypes.c_int32),
                ("decode_waves", ctypes.c_int32), ("decode_min_chunk_pages", ctypes.c_int32), ("prefill_pairs", ctypes.c_int32)]


class CfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {cf_status_string(status)} ({status})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the C-ABI library; raises if it has not been built (no fallback of any kind)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_27085_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i32p, fp = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float)
    dp = ctypes.POINTER(CacheDesc)
    lib.cf_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, ctypes.c_size_t]
    lib.cf_destroy.argtypes = [vp]
    lib.cf_kv_append.argtypes = [vp, dp, vp, vp, vp, vp, vp, i32, vp, vp, i32, vp]
    lib.cf_mixed_attention.argtypes = [vp, dp, vp, vp, vp, vp, i32, vp, vp, i32, vp, vp, vp]
    lib.cf_mixed_attention_shared.argtypes = [vp, dp, vp, vp, vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, vp]
    lib.cf_get_last_plan_counts.argtypes = [vp, vp]
    lib.cf_mixed_step_host.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, i32, vp, vp, i32, vp, vp]
    lib.cf_host_steps_flush.argtypes = [vp, vp]
    lib.cf_get_async_status.argtypes = [vp]
    lib.cf_set_timing.argtypes = [vp, ctypes.c_int]
    lib.cf_get_timing_sums.argtypes = [vp, fp, fp, fp, i32p]
    lib.cf_get_last_launch_count.argtypes = [vp, i32p]
    lib.cf_plan_inspect.argtypes = [dp, vp, vp, i32, i32, ctypes.POINTER(PlanOptions), vp, vp, vp, i32, vp]
    lib.cf_set_debug_option.argtypes = [vp, ctypes.c_int, ctypes.c_int]
    dbl = ctypes.POINTER(ctypes.c_double)
    lib.cf_get_host_time_sums.argtypes = [vp, dbl, dbl, dbl, i32p]
    lib.cf_decode_attention_static.argtypes = [dp, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp]
    lib.cf_selftest_bounded_wait.argtypes = [vp, vp]
    lib.cf_set_overlap.argtypes = [vp, ctypes.c_int]
    lib.cf_validate_block_table.argtypes = [vp, dp, vp, i32, vp, vp, i32, vp, i32p]
    lib.cf_estimate_us.argtypes = [dp, vp, vp, i32, i32, i32, fp, fp, fp]
    lib.cf_spatial_share.argtypes = [dp, vp, vp, i32, i32]
    lib.cf_spatial_share.restype = ctypes.c_int32
    lib.cf_plan_create.argtypes = [vp, dp, vp, vp, i32, i32, vp, ctypes.POINTER(vp)]
    lib.cf_plan_destroy.argtypes = [vp]
    lib.cf_kv_append_planned.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.cf_mixed_attention_planned.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.cf_status_string.argtypes = [ctypes.c_int]
    lib.cf_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "cf_status_string":
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def cf_status_string(status: int) -> str:
    return load_library().cf_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != CF_OK:
        raise CfError(status, where)


def _dev(x) -> Optional[int]:
    """Device address of a torch tensor, or an integer address, or None."""
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    return int(x)


def _host_i32(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.int32)


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    return int(getattr(stream, "cuda_stream", stream)) or None


def make_desc(num_q_heads: int, num_kv_heads: int, head_dim: int, block_size: int, num_blocks: int,
              k_strides: Optional[Tuple[int, int, int]] = None, v_strides: Optional[Tuple[int, int, int]] = None,
              softmax_scale: float = 0.0, window_size: int = 0, sink_logits=None, kv_dtype: int = 0, k_scale=None,
              v_scale=None) -> CacheDesc:
    """Descriptor for pools laid out [num_blocks, num_kv_heads, block_size, head_dim] unless
    (block, head, token) element strides are given.  window_size > 0: sliding-window attention;
    sink_logits: device fp32 tensor [num_q_heads] (or address) of per-head sink logits.  The caller keeps
    the sink tensor alive for as long as the descriptor is used.  kv_dtype = CF_KV_FP8_E4M3: the pools hold e4m3
    codes (one byte per element) and k_scale / v_scale are device fp32 tensors [num_kv_heads]."""
    default = (num_kv_heads * block_size * head_dim, block_size * head_dim, head_dim)
    ks = k_strides or default
    vs = v_strides or default
    return CacheDesc(num_q_heads, num_kv_heads, head_dim, block_size, num_blocks,
                     ks[0], ks[1], ks[2], vs[0], vs[1], vs[2], softmax_scale, int(window_size), _dev(sink_logits),
                     int(kv_dtype), _dev(k_scale), _dev(v_scale))


def cf_create(device: int = 0, workspace_bytes: int = 0) -> ctypes.c_void_p:
    lib = load_library()
    ctx = ctypes.c_void_p()
    _check(lib.cf_create(ctypes.byref(ctx), int(device), int(workspace_bytes)), "cf_create")
    return ctx


def cf_destroy(ctx) -> None:
    _check(load_library().cf_destroy(ctx), "cf_destroy")


def cf_kv_append(ctx, desc: CacheDesc, k_cache, v_cache, k_new, v_new, block_table, max_blocks_per_seq: int,
                 context_len, query_len, stream=None, check: bool = True) -> int:
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    st = load_library().cf_kv_append(ctx, ctypes.byref(desc), _dev(k_cache), _dev(v_cache), _dev(k_new), _dev(v_new),
                                     _dev(block_table), int(max_blocks_per_seq), lc.ctypes.data, lq.ctypes.data,
                                     int(lc.shape[0]), _stream(stream))
    if check:
        _check(st, "cf_kv_append")
    return st


def cf_mixed_attention(ctx, desc: CacheDesc, q, k_cache, v_cache, block_table, max_blocks_per_seq: int,
                       context_len, query_len, out, lse=None, stream=None, check: bool = True) -> int:
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    st = load_library().cf_mixed_attention(ctx, ctypes.byref(desc), _dev(q), _dev(k_cache), _dev(v_cache),
                                           _dev(block_table), int(max_blocks_per_seq), lc.ctypes.data, lq.ctypes.data,
                                           int(lc.shape[0]), _dev(out), _dev(lse), _stream(stream))
    if check:
        _check(st, "cf_mixed_attention")
    return st


def cf_mixed_attention_shared(ctx, desc: CacheDesc, q, k_cache, v_cache, block_table, max_blocks_per_seq: int,
                              context_len, query_len, share_group, shared_len, out, lse=None, stream=None,
                              check: bool = True) -> int:
    """cf_mixed_attention with shared prefixes described: share_group[s] >= 0 names the group whose members have
    the same pages for their first shared_len[s] tokens (host int32 arrays)."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    sg, sl = _host_i32(share_group), _host_i32(shared_len)
    st = load_library().cf_mixed_attention_shared(ctx, ctypes.byref(desc), _dev(q), _dev(k_cache), _dev(v_cache),
                                                  _dev(block_table), int(max_blocks_per_seq), lc.ctypes.data, lq.ctypes.data,
                                                  sg.ctypes.data, sl.ctypes.data, int(lc.shape[0]), _dev(out), _dev(lse),
                                                  _stream(stream))
    if check:
        _check(st, "cf_mixed_attention_shared")
    return st


def cf_get_last_plan_counts(ctx) -> np.ndarray:
    """Item counts of the last plan built by cf_mixed_attention(_shared): see the header."""
    counts = np.zeros(8, dtype=np.int32)
    _check(load_library().cf_get_last_plan_counts(ctx, counts.ctypes.data), "cf_get_last_plan_counts")
    return counts


def cf_mixed_step_host(ctx, desc: CacheDesc, q_host, k_new_host, v_new_host, k_cache, v_cache, block_table,
                       max_blocks_per_seq: int, context_len, query_len, out_host, stream=None, check: bool = True) -> int:
    """q_host / k_new_host / v_new_host / out_host: host tensors (pinned recommended) or addresses."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    st = load_library().cf_mixed_step_host(ctx, ctypes.byref(desc), _dev(q_host), _dev(k_new_host), _dev(v_new_host),
                                           _dev(k_cache), _dev(v_cache), _dev(block_table), int(max_blocks_per_seq),
                                           lc.ctypes.data, lq.ctypes.data, int(lc.shape[0]), _dev(out_host),
                                           _stream(stream))
    if check:
        _check(st, "cf_mixed_step_host")
    return st


def cf_host_steps_flush(ctx, stream=None) -> None:
    """Makes `stream` wait for the read-backs of every cf_mixed_step_host call issued so far."""
    _check(load_library().cf_host_steps_flush(ctx, _stream(stream)), "cf_host_steps_flush")


def cf_get_async_status(ctx) -> int:
    return int(load_library().cf_get_async_status(ctx))


def cf_selftest_bounded_wait(ctx, stream=None) -> None:
    """Enqueues the kernel whose bounded wait must expire (see cf_get_async_status)."""
    _check(load_library().cf_selftest_bounded_wait(ctx, _stream(stream)), "cf_selftest_bounded_wait")


def cf_set_overlap(ctx, n) -> None:
    """Spatial launch sequence: n > 0 persistent prefill CTAs take their SMs first (1 or True = the
    library's default share), decode + combine run beside them; 0 = the serial sequence."""
    _check(load_library().cf_set_overlap(ctx, int(n)), "cf_set_overlap")


def cf_set_debug_option(ctx, option: int, value: int) -> None:
    """Test-only planner / launch-sequence switches (CF_DEBUG_*); value <= 0 restores the default."""
    _check(load_library().cf_set_debug_option(ctx, int(option), int(value)), "cf_set_debug_option")


def cf_set_timing(ctx, enabled: bool) -> None:
    _check(load_library().cf_set_timing(ctx, int(bool(enabled))), "cf_set_timing")


def cf_get_timing_sums(ctx) -> Tuple[float, float, float, int]:
    """(ms_decode, ms_combine, ms_prefill, num_calls) summed over the calls timed since the last query."""
    a, b, c, n = ctypes.c_float(), ctypes.c_float(), ctypes.c_float(), ctypes.c_int32()
    _check(load_library().cf_get_timing_sums(ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(n)),
           "cf_get_timing_sums")
    return a.value, b.value, c.value, n.value


def cf_get_host_time_sums(ctx) -> Tuple[float, float, float, int]:
    """(us in cf_kv_append, us in cf_mixed_attention, us of that in the planner, attention calls) since the last query."""
    a, b, c, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_double(), ctypes.c_int32()
    _check(load_library().cf_get_host_time_sums(ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(n)),
           "cf_get_host_time_sums")
    return a.value, b.value, c.value, n.value


def cf_get_last_launch_count(ctx) -> int:
    n = ctypes.c_int32()
    _check(load_library().cf_get_last_launch_count(ctx, ctypes.byref(n)), "cf_get_last_launch_count")
    return n.value


def cf_plan_inspect(desc: CacheDesc, context_len, query_len, max_blocks_per_seq: int, num_sms: int = 148,
                    cap: int = 1 << 16, check: bool = True, prefill_sms_mixed: int = 0, prefill_force_split: int = 0,
                    decode_waves: int = 0, decode_min_chunk_pages: int = 0, want_counts: bool = False, prefill_pairs: int = 0):
    """Returns (status, decode_items [n,6], combine_items [n,3], prefill_items [n,8], n_partial_slots)
    and, with want_counts, the six counters as a last element."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    dec = np.zeros((cap, 6), dtype=np.int32)
    comb = np.zeros((cap, 3), dtype=np.int32)
    pre = np.zeros((cap, 8), dtype=np.int32)
    counts = np.zeros(6, dtype=np.int32)
    opts = PlanOptions(int(num_sms), int(prefill_sms_mixed), int(prefill_force_split), int(decode_waves),
                       int(decode_min_chunk_pages), int(prefill_pairs))
    st = load_library().cf_plan_inspect(ctypes.byref(desc), lc.ctypes.data, lq.ctypes.data, int(lc.shape[0]),
                                        int(max_blocks_per_seq), ctypes.byref(opts), dec.ctypes.data, comb.ctypes.data,
                                        pre.ctypes.data, cap, counts.ctypes.data)
    if check:
        _check(st, "cf_plan_inspect")
    res = (st, dec[:counts[0]], comb[:counts[1]], pre[:counts[2]], int(counts[3]))
    return res + (counts,) if want_counts else res


def cf_decode_attention_static(desc: CacheDesc, q, k_cache, v_cache, block_table, max_blocks_per_seq: int,
                               context_len, out, lse=None, stream=None, check: bool = True) -> int:
    """All-decode attention for callers that must not allocate device memory (a plugin that only
    receives its buffers, a process whose GPU memory belongs to another allocator): no context, the
    split-K scratch is a fixed 16 MiB array inside the library.  One query token per sequence;
    runs on the current device; calls sharing the array must not overlap on the GPU.  Batches beyond
    the fixed limits return CF_ERR_WORKSPACE."""
    lc = _host_i32(context_len)
    st = load_library().cf_decode_attention_static(ctypes.byref(desc), _dev(q), _dev(k_cache), _dev(v_cache),
                                                   _dev(block_table), int(max_blocks_per_seq), lc.ctypes.data,
                                                   int(lc.shape[0]), _dev(out), _dev(lse), _stream(stream))
    if check:
        _check(st, "cf_decode_attention_static")
    return st


def cf_plan_create(ctx, desc: CacheDesc, context_len, query_len, max_blocks_per_seq: int, stream=None) -> ctypes.c_void_p:
    """Plans one set of lengths once; the returned handle serves every layer's planned calls."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    plan = ctypes.c_void_p()
    _check(load_library().cf_plan_create(ctx, ctypes.byref(desc), lc.ctypes.data, lq.ctypes.data, int(lc.shape[0]),
                                         int(max_blocks_per_seq), _stream(stream), ctypes.byref(plan)), "cf_plan_create")
    return plan


def cf_plan_destroy(plan) -> None:
    _check(load_library().cf_plan_destroy(plan), "cf_plan_destroy")


def cf_kv_append_planned(plan, k_cache, v_cache, k_new, v_new, block_table, stream=None) -> None:
    _check(load_library().cf_kv_append_planned(plan, _dev(k_cache), _dev(v_cache), _dev(k_new), _dev(v_new),
                                               _dev(block_table), _stream(stream)), "cf_kv_append_planned")


def cf_mixed_attention_planned(plan, q, k_cache, v_cache, block_table, out, lse=None, stream=None) -> None:
    _check(load_library().cf_mixed_attention_planned(plan, _dev(q), _dev(k_cache), _dev(v_cache), _dev(block_table),
                                                     _dev(out), _dev(lse), _stream(stream)), "cf_mixed_attention_planned")


def cf_spatial_share(desc: CacheDesc, context_len, query_len, num_sms: int = 148) -> int:
    """SMs the first prefill grid of the spatial sequence takes for these lengths (0: no mixed batch)."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    return int(load_library().cf_spatial_share(ctypes.byref(desc), lc.ctypes.data, lq.ctypes.data, int(lc.shape[0]), int(num_sms)))


def cf_estimate_us(desc: CacheDesc, context_len, query_len, max_blocks_per_seq: int, num_sms: int = 148) -> Tuple[float, float, float]:
    """Predicted (us_decode, us_combine, us_prefill) of one cf_mixed_attention call on a B200 (host only)."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    a, b, c = ctypes.c_float(), ctypes.c_float(), ctypes.c_float()
    _check(load_library().cf_estimate_us(ctypes.byref(desc), lc.ctypes.data, lq.ctypes.data, int(lc.shape[0]),
                                         int(max_blocks_per_seq), int(num_sms), ctypes.byref(a), ctypes.byref(b),
                                         ctypes.byref(c)), "cf_estimate_us")
    return a.value, b.value, c.value


def cf_validate_block_table(ctx, desc: CacheDesc, block_table, max_blocks_per_seq: int, context_len, query_len,
                            stream=None) -> int:
    """Number of block-table entries in use that fall outside the pool (0 = table is safe to use)."""
    lc, lq = _host_i32(context_len), _host_i32(query_len)
    bad = ctypes.c_int32()
    st = load_library().cf_validate_block_table(ctx, ctypes.byref(desc), _dev(block_table), int(max_blocks_per_seq),
                                                lc.ctypes.data, lq.ctypes.data, int(lc.shape[0]), _stream(stream),
                                                ctypes.byref(bad))
    if st not in (CF_OK, CF_ERR_OUT_OF_RANGE):
        raise CfError(st, "cf_validate_block_table")
    return bad.value
