"""The allocation-free decode entry point, for integrators that cannot call cudaMalloc where they
need attention (they are handed buffers only, or another allocator owns the GPU's memory).  It must
give what the context-based entry point gives on the same all-decode batch, on back-to-back calls
that reuse the library's fixed scratch array, and refuse batches beyond its fixed limits.

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

import cf_synth as syn
import paper_2609_27085_b200 as cf
from harness import GpuScenario, to_dev_bf16, to_host_bits

pytestmark = pytest.mark.gpu


def _decode_scenario(seed, lens, Hq=32, Hkv=8, D=128, NB=8192):
    geom = syn.Geometry(Hq, Hkv, D, 16, NB)
    return syn.scenario_from_lengths("na", geom, seed, [l - 1 for l in lens], [[1] * len(lens)])


def _both_ways(sc):
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    ref_o, ref_lse = g.attend(b)                                   # context-based entry point
    geom = sc.geom
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.full((b.total_q, geom.num_q_heads, geom.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((b.total_q, geom.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, out, lse)
    torch.cuda.synchronize()
    g.close()
    return ref_o, ref_lse, to_host_bits(out), lse.cpu().numpy()


def _check(ref_o, ref_lse, o, lse):
    a, r = syn.bf16_bits_to_f64(o), syn.bf16_bits_to_f64(ref_o)
    assert np.isfinite(a).all() and np.isfinite(lse).all()
    err = np.abs(a - r)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3            # the tolerance of the parity tests
    assert np.abs(lse - ref_lse).max() <= 1e-4


def test_static_scratch_entry_matches_context_entry_twice_in_a_row():
    # first call: long sequences that are split into several chunks (partials + combine) next to short ones
    first = _decode_scenario(31, [30000, 17, 4096, 1, 9001, 640, 12345, 16])
    _check(*_both_ways(first))
    # second call straight after, different shapes: the scratch still holds the first call's partials
    second = _decode_scenario(32, [5000, 22000, 3, 700, 15999], Hq=64)
    _check(*_both_ways(second))
    # and the first batch again
    _check(*_both_ways(first))


def test_static_scratch_entry_rejects_what_does_not_fit():
    sc = _decode_scenario(33, [100, 200])
    b = sc.batches[0]
    g = GpuScenario(sc)
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.zeros_like(q)
    too_many = np.full(2000, 64, dtype=np.int32)                      # more than 1024 sequences
    st = cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, b.max_blocks, too_many, out, check=False)
    assert st == cf.CF_ERR_WORKSPACE
    st = cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, b.max_blocks, [0, 5], out, check=False)
    assert st == cf.CF_ERR_INVALID_ARG                                # a decode sequence has at least its own token
    st = cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, 1, [100, 200], out, check=False)
    assert st == cf.CF_ERR_OUT_OF_RANGE
    torch.cuda.synchronize()
    assert (out == 0).all()
    g.close()
