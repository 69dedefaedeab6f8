"""Loader for the CPU oracle (``cf_oracle.c``).

TEST INFRASTRUCTURE ONLY: the fp64 definition the CUDA library is checked against.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; it imports nothing from the CUDA package and shares no code with it.

``mixed_attention`` evaluates textbook softmax attention through the block table in
fp64 (see the header of ``cf_oracle.c`` for the formula and the passages of the
paper that fix the shapes); ``kv_append`` is the byte scatter of new K/V rows.
Inputs are numpy arrays; bf16 tensors are ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import hashlib
import math
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cf_oracle.c")


def _cpu_tag() -> str:
    """The oracle is compiled -march=native, so the binary is keyed by the host's CPU flags."""
    try:
        with open("/proc/cpuinfo") as f:
            flags = next((ln for ln in f if ln.startswith("flags")), "")
    except OSError:
        flags = ""
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


_LIB = os.path.join(_HERE, f"libcf_oracle_{_cpu_tag()}.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-march=native", "-fopenmp", "-fPIC", "-shared",
                               "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.cf_oracle_mixed_attention.restype = ctypes.c_int
        lib.cf_oracle_mixed_attention.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i64, vp, i32, vp, vp, i32,
                                                  i32, i32, i32, i32, f64, vp, i64, vp, vp, vp, i64, i32, vp, i32, vp, vp]
        lib.cf_oracle_kv_append_fp8.restype = ctypes.c_int
        lib.cf_oracle_kv_append_fp8.argtypes = [vp, vp, i64, i64, i64, i64, i64, i64, vp, vp, vp, i32, vp, vp, i32,
                                                i32, i32, i32, vp, vp]
        lib.cf_oracle_e4m3_decode.argtypes = [vp, i64, vp]
        lib.cf_oracle_e4m3_encode.argtypes = [vp, i64, vp]
        lib.cf_oracle_kv_append.restype = ctypes.c_int
        lib.cf_oracle_kv_append.argtypes = [vp, vp, i64, i64, i64, i64, i64, i64, vp, vp, vp, i32, vp, vp, i32,
                                            i32, i32, i32]
        lib.cf_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().cf_oracle_num_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _pool_strides(pool: np.ndarray) -> Tuple[int, int, int]:
    """Element strides (block, head, token) of a [NB, Hkv, B, D] pool view (uint16: bf16 bits; uint8: e4m3 codes)."""
    es = pool.dtype.itemsize
    assert pool.dtype in (np.uint16, np.uint8) and pool.ndim == 4 and pool.strides[3] == es
    return pool.strides[0] // es, pool.strides[1] // es, pool.strides[2] // es


def _base(pool: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(pool.__array_interface__["data"][0])


def mixed_attention(q: np.ndarray, k_pool: np.ndarray, v_pool: np.ndarray, block_table: np.ndarray,
                    context_len: np.ndarray, query_len: np.ndarray, scale: Optional[float] = None,
                    rows: Optional[np.ndarray] = None, want_weights: int = 0, window: int = 0,
                    sinks: Optional[np.ndarray] = None, k_scale: Optional[np.ndarray] = None,
                    v_scale: Optional[np.ndarray] = None):
    """fp64 paged attention.  q: uint16 [T, Hq, D]; pools: uint16 [NB, Hkv, B, D] (any strides with
    a contiguous last axis).  Returns (out [n, Hq, D], lse [n, Hq]) and, if want_weights > 0, the
    softmax weights [n, Hq, want_weights].
    window > 0: sliding window (the query at position p sees keys (p - window, p]); sinks: per-query-head
    logits [Hq] that join the softmax denominator only (see the header of cf_oracle.c).
    uint8 pools hold e4m3 codes and need k_scale / v_scale (per KV head, [Hkv])."""
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.uint16)
    T, Hq, D = q.shape
    NB, Hkv, B, D2 = k_pool.shape
    assert D2 == D and v_pool.shape == k_pool.shape
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    lc = np.ascontiguousarray(context_len, dtype=np.int32)
    lq = np.ascontiguousarray(query_len, dtype=np.int32)
    S = lc.shape[0]
    assert bt.shape[0] == S and lq.shape[0] == S and int(lq.sum()) == T
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.shape[0]
    else:
        n = T
    out = np.empty((n, Hq, D), dtype=np.float64)
    lse = np.empty((n, Hq), dtype=np.float64)
    w = np.empty((n, Hq, want_weights), dtype=np.float64) if want_weights else None
    if sinks is not None:
        sinks = np.ascontiguousarray(sinks, dtype=np.float64)
        assert sinks.shape == (Hq,)
    fp8 = k_pool.dtype == np.uint8
    assert v_pool.dtype == k_pool.dtype
    if fp8:
        k_scale = np.ascontiguousarray(k_scale, dtype=np.float64)
        v_scale = np.ascontiguousarray(v_scale, dtype=np.float64)
        assert k_scale.shape == (Hkv,) and v_scale.shape == (Hkv,)
    ks, vs = _pool_strides(k_pool), _pool_strides(v_pool)
    rc = lib.cf_oracle_mixed_attention(
        _ptr(q), _base(k_pool), _base(v_pool), ks[0], ks[1], ks[2], vs[0], vs[1], vs[2],
        _ptr(bt), bt.shape[1], _ptr(lc), _ptr(lq), S, Hq, Hkv, D, B,
        float(1.0 / math.sqrt(D) if scale is None else scale),
        _ptr(rows), n, _ptr(out), _ptr(lse), _ptr(w), want_weights, int(window), _ptr(sinks),
        int(fp8), _ptr(k_scale) if fp8 else None, _ptr(v_scale) if fp8 else None)
    if rc != 0:
        raise ValueError(f"cf_oracle_mixed_attention rejected its arguments (code {rc})")
    return (out, lse, w) if want_weights else (out, lse)


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(codes.shape, dtype=np.float64)
    _load().cf_oracle_e4m3_decode(_ptr(codes), codes.size, _ptr(out))
    return out


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint8)
    _load().cf_oracle_e4m3_encode(_ptr(x), x.size, _ptr(out))
    return out


def kv_append(k_pool: np.ndarray, v_pool: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
              block_table: np.ndarray, context_len: np.ndarray, query_len: np.ndarray,
              k_scale: Optional[np.ndarray] = None, v_scale: Optional[np.ndarray] = None) -> None:
    """In-place scatter of the new rows (uint16 [T, Hkv, D]) into the pools; uint8 pools are fp8 caches and the
    rows are quantised with the per-head scales (see the header of cf_oracle.c)."""
    lib = _load()
    if k_pool.dtype == np.uint8:
        k_new = np.ascontiguousarray(k_new, dtype=np.uint16)
        v_new = np.ascontiguousarray(v_new, dtype=np.uint16)
        NB, Hkv, B, D = k_pool.shape
        bt = np.ascontiguousarray(block_table, dtype=np.int32)
        lc = np.ascontiguousarray(context_len, dtype=np.int32)
        lq = np.ascontiguousarray(query_len, dtype=np.int32)
        ksc = np.ascontiguousarray(k_scale, dtype=np.float32)
        vsc = np.ascontiguousarray(v_scale, dtype=np.float32)
        assert ksc.shape == (Hkv,) and vsc.shape == (Hkv,) and v_pool.dtype == np.uint8
        assert k_new.shape == (int(lq.sum()), Hkv, D) and v_new.shape == k_new.shape
        ks, vs = _pool_strides(k_pool), _pool_strides(v_pool)
        rc = lib.cf_oracle_kv_append_fp8(_base(k_pool), _base(v_pool), ks[0], ks[1], ks[2], vs[0], vs[1], vs[2],
                                         _ptr(k_new), _ptr(v_new), _ptr(bt), bt.shape[1], _ptr(lc), _ptr(lq),
                                         lc.shape[0], Hkv, D, B, _ptr(ksc), _ptr(vsc))
        if rc != 0:
            raise ValueError(f"cf_oracle_kv_append_fp8 rejected its arguments (code {rc})")
        return
    k_new = np.ascontiguousarray(k_new, dtype=np.uint16)
    v_new = np.ascontiguousarray(v_new, dtype=np.uint16)
    NB, Hkv, B, D = k_pool.shape
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    lc = np.ascontiguousarray(context_len, dtype=np.int32)
    lq = np.ascontiguousarray(query_len, dtype=np.int32)
    assert k_new.shape == (int(lq.sum()), Hkv, D) and v_new.shape == k_new.shape
    assert k_pool.flags.writeable and v_pool.flags.writeable
    ks, vs = _pool_strides(k_pool), _pool_strides(v_pool)
    rc = lib.cf_oracle_kv_append(_base(k_pool), _base(v_pool), ks[0], ks[1], ks[2], vs[0], vs[1], vs[2],
                                 _ptr(k_new), _ptr(v_new), _ptr(bt), bt.shape[1], _ptr(lc), _ptr(lq),
                                 lc.shape[0], Hkv, D, B)
    if rc != 0:
        raise ValueError(f"cf_oracle_kv_append rejected its arguments (code {rc})")
