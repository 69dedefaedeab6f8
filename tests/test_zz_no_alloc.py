"""The allocation-free decode entry point, for integrators that cannot call cudaMalloc where they
need attention (they are handed buffers only, or another allocator owns the GPU's memory).  It is
held to the fp64 oracle like every other path, must give the bits of the context-based entry point on
the same all-decode batch, on back-to-back calls that reuse the library's fixed scratch array, must
not change the amount of free device memory, and must refuse batches beyond its fixed limits.

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

import cf_synth as syn
import oracle
import paper_2609_27085_b200 as cf
from harness import GpuScenario, compare, to_dev_bf16, to_host_bits

pytestmark = pytest.mark.gpu


def _decode_scenario(seed, lens, Hq=32, Hkv=8, D=128, NB=8192):
    geom = syn.Geometry(Hq, Hkv, D, 16, NB)
    return syn.scenario_from_lengths("na", geom, seed, [l - 1 for l in lens], [[1] * len(lens)])


def _both_ways(sc):
    """Runs the batch through the context entry point and through the static one; checks the static one
    against the oracle and against the context entry point's bits."""
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    ctx_o, ctx_lse = g.attend(b)                                   # context-based entry point
    geom = sc.geom
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.full((b.total_q, geom.num_q_heads, geom.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((b.total_q, geom.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, out, lse)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                               # the call allocated nothing on the device
    k_ref, v_ref = g.pools_host()
    g.close()
    o_bits, lse_h = to_host_bits(out), lse.cpu().numpy()
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len)
    compare(o_bits, lse_h, ref_o, ref_lse, label="static entry vs oracle")
    assert np.array_equal(o_bits, ctx_o) and np.array_equal(lse_h, ctx_lse)     # same chunking, same merge order


def test_static_scratch_entry_matches_oracle_and_context_entry_twice_in_a_row():
    # first call: long sequences that are split into several chunks (partials + combine) next to short ones
    first = _decode_scenario(31, [30000, 17, 4096, 1, 9001, 640, 12345, 16])
    _both_ways(first)
    # second call straight after, different shapes: the scratch still holds the first call's partials
    second = _decode_scenario(32, [5000, 22000, 3, 700, 15999], Hq=64)
    _both_ways(second)
    # and the first batch again
    _both_ways(first)


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
    # (The other two limits - 3584 KV chunks, 16 MiB of partials - bound the planner's output, which for S
    # sequences never exceeds S + 4 waves x 2 CTAs x SMs / Hkv chunks; on a 148-SM device they cannot be reached
    # and are there for devices with more SMs.)
    torch.cuda.synchronize()
    assert (out == 0).all()
    g.close()


def test_static_scratch_entry_refuses_a_capturing_stream():
    """The call copies its plan from the caller's stack, so it cannot become a graph node: on a stream that
    is being captured it returns CF_ERR_UNSUPPORTED and records nothing."""
    sc = _decode_scenario(34, [300, 40])
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.zeros_like(q)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            st = cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, out, stream=side,
                                               check=False)
    assert st == cf.CF_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    del graph
    g.close()
