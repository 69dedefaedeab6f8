"""GPU parity at the full sizes of the five workload configurations, in the launch configuration
the benchmark times: every chunk iteration of configs 3 and 4, all 13 sweep points of config 5.
Decode rows are all checked; prefill rows are checked on a deterministic sample - the first and
last row of every 128-row q tile, the last row and every 41st row of each chunk, all heads - because
the fp64 oracle needs ~1 TFLOP per iteration for the long chunks."""
import pytest

import cf_synth as syn
from harness import run_and_check

pytestmark = pytest.mark.gpu


def test_config2_decode_only_full_size():
    print(run_and_check(syn.config2_decode_only(), check_append=True))


def test_config3_chat_all_iterations():
    print(run_and_check(syn.config3_chat(), tile_rows=True, check_append=False))


def test_config4_agentic_all_iterations():
    sc = syn.config4_agentic()
    print(run_and_check(sc, tile_rows=True, check_append=False))


@pytest.mark.parametrize("budget,n", syn.CONFIG5_POINTS)
def test_config5_sweep_points(budget, n):
    print(run_and_check(syn.config5_sweep_point(budget, n), tile_rows=True, check_append=False))


@pytest.mark.parametrize("make", [lambda: syn.config3_chat(iterations=(3,)), lambda: syn.config5_sweep_point(2048, 3)])
def test_launch_sequences_agree_bit_for_bit_on_one_plan_at_full_size(make):
    """One plan of a full-size mixed batch run as the serial sequence, the default spatial sequence and with a
    20-CTA front grid (every CTA works through many items, the second grid takes part): identical output
    and lse bits.  (Unplanned calls plan per launch sequence - the spatial one balances the prefill items
    over the front grid's SMs and may cut other items into KV ranges - so across sequences they agree to
    rounding, not to the bit; each of them is held to the oracle by the tests above.)"""
    import numpy as np
    import torch
    import paper_2609_27085_b200 as cf
    from harness import GpuScenario, to_dev_bf16, to_host_bits
    sc = make()
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    plan = cf.cf_plan_create(g.ctx, g.desc, b.context_len, b.query_len, b.max_blocks)
    outs = []
    for mode in (0, 1, 20):
        cf.cf_set_overlap(g.ctx, mode)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((b.total_q, sc.geom.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        cf.cf_mixed_attention_planned(plan, q, g.k, g.v, bt, out, lse)
        torch.cuda.synchronize()
        outs.append((to_host_bits(out), lse.cpu().numpy()))
    cf.cf_set_overlap(g.ctx, 1)
    assert np.isfinite(outs[0][1]).all()
    for o, l in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(l, outs[0][1])
    assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
    cf.cf_plan_destroy(plan)
    g.close()


def test_paper_context_limit_128k():
    """The paper's workers run a 128K-token context with 512 reserved (Section 6.1): one decode sequence
    at that limit, one at a page boundary below it, and a 300-token prefill chunk that ends at the limit."""
    geom = syn.Geometry(32, 8, 128, 16, 32768)
    limit = 131072 - 512
    sc = syn.scenario_from_lengths("ctx128k", geom, 4242, [limit - 1, 65536 - 1, limit - 300], [[1, 1, 300]])
    print(run_and_check(sc, tile_rows=True, check_append=False))
