"""GPU parity of the model-specific attention variant - sliding window and per-head attention sinks -
against the oracle's statement of it, on the decode kernel, the tcgen05 prefill kernel (whole items and
KV ranges) and mixed batches."""
import numpy as np
import pytest
import torch

import cf_synth as syn
import oracle
import paper_2609_27085_b200 as cf
from harness import GpuScenario, compare, run_and_check, to_dev_bf16, to_host_bits

pytestmark = pytest.mark.gpu


def small(seed, Hq, Hkv, D, prefix, qlens, NB=2048, shuffle=False):
    return syn.scenario_from_lengths("v", syn.Geometry(Hq, Hkv, D, 16, NB), seed, prefix, qlens, shuffle_seqs=shuffle)


def sink_values(Hq, seed=0):
    return np.random.default_rng(100 + seed).normal(0.0, 2.0, size=Hq).astype(np.float32)


@pytest.mark.parametrize("window", [1, 16, 17, 100, 128, 1000, 5000])
@pytest.mark.parametrize("Hq,Hkv,D,with_sinks", [(32, 8, 128, True), (8, 2, 64, False), (64, 8, 128, True)])
def test_windowed_decode(window, Hq, Hkv, D, with_sinks):
    lens = [1, 2, 15, 16, 17, 31, 33, 127, 129, 255, 700, 1025, 2500, 4097, 9000, 20000]
    sc = small(3, Hq, Hkv, D, [l - 1 for l in lens], [[1] * len(lens)], NB=4096)
    run_and_check(sc, window=window, sinks=sink_values(Hq) if with_sinks else None)


@pytest.mark.parametrize("window", [1, 17, 128, 129, 300, 1024])
@pytest.mark.parametrize("Hq,Hkv,D,with_sinks", [(32, 8, 128, True), (4, 4, 128, False), (8, 2, 64, True), (16, 2, 128, False)])
def test_windowed_prefill(window, Hq, Hkv, D, with_sinks):
    prefix = [0, 0, 5, 16, 63, 64, 100, 1000, 0, 333, 2000]
    qlen = [2, 64, 65, 17, 1, 128, 129, 200, 300, 31, 700]
    run_and_check(small(5, Hq, Hkv, D, prefix, [qlen]), window=window, sinks=sink_values(Hq, 1) if with_sinks else None)


def test_sinks_without_a_window():
    prefix = [10, 0, 500, 77, 0, 2000, 31, 640, 5, 1, 9000]
    qlen = [1, 90, 1, 0, 1, 1, 130, 1, 0, 64, 1]
    run_and_check(small(7, 32, 8, 128, prefix, [qlen], shuffle=True), sinks=sink_values(32, 2))
    # a huge sink swallows nearly all of the probability: outputs shrink towards zero, lse follows the sink
    run_and_check(small(7, 8, 2, 64, prefix, [qlen], shuffle=True), sinks=np.full(8, 30.0, dtype=np.float32))
    run_and_check(small(7, 8, 2, 64, prefix, [qlen], shuffle=True), sinks=np.full(8, -30.0, dtype=np.float32))


@pytest.mark.parametrize("split", [2, 3])
def test_windowed_prefill_items_cut_into_kv_ranges(split):
    """A window long enough for the band to hold several KV ranges per item (forced split), with sinks (joined in
    the combine pass), beside decode sequences."""
    prefix = [6000, 300, 4097, 50, 8000]
    qlen = [300, 700, 129, 1, 1]
    sinks = sink_values(32, 3)
    for window in (2048, 3000):
        sc = small(43, 32, 8, 128, prefix, [qlen], NB=2048)
        b = sc.batches[0]
        d = cf.make_desc(32, 8, 128, 16, 2048, window_size=window)
        counts = cf.cf_plan_inspect(d, b.context_len, b.query_len, b.max_blocks, prefill_force_split=split, want_counts=True)[5]
        assert counts[5] > 0
        run_and_check(sc, window=window, sinks=sinks, debug={cf.CF_DEBUG_PREFILL_SPLIT: split})


def test_pages_left_of_the_window_are_never_touched():
    """An engine that serves a sliding-window layer releases the pages that no query can see any more.  Here their
    block-table entries are -1 and their contents NaN: the kernels must neither dereference the entries (the
    status word would report a block id outside the pool) nor let the contents reach a result."""
    window = 200
    prefix = [3000, 5000, 700, 130, 0]
    qlen = [300, 1, 1, 150, 64]
    sc = small(45, 32, 8, 128, prefix, [qlen], NB=1024)
    b = sc.batches[0]
    g = GpuScenario(sc, window=window, sinks=sink_values(32, 4))
    g.append(b)
    k_ref, v_ref = g.pools_host()
    table = b.block_table.copy()
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device="cuda")
    for s in range(b.num_seqs):
        first_visible = int(b.context_len[s]) - int(b.query_len[s]) - window + 1      # left edge of the first row's window
        for pg in range(max(0, first_visible) // 16):
            blk = int(table[s, pg])
            g.k[blk] = nan
            g.v[blk] = nan
            k_ref[blk] = syn.BF16_NAN_BITS
            v_ref[blk] = syn.BF16_NAN_BITS
            table[s, pg] = -1
    dead = syn.Batch(b.geom, b.context_len, b.query_len, table, b.q, b.k_new, b.v_new)
    o_bits, lse = g.attend(dead)
    assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, table, b.context_len, b.query_len, window=window,
                                            sinks=sink_values(32, 4).astype(np.float64))
    assert np.isfinite(ref_o).all()
    compare(o_bits, lse, ref_o, ref_lse)
    g.close()


def test_window_edges_with_a_spike_key():
    """A key that towers over the rest, planted on both sides of the window's left edge of several rows: inside
    the window it must dominate the row, one position further left it must not be seen."""
    Hq, Hkv, D, window = 8, 2, 128, 300
    Lq, P = 400, 1500
    sc = small(47, Hq, Hkv, D, [P, 2000], [[Lq, 1]], NB=1024)
    b = sc.batches[0]
    g = GpuScenario(sc, window=window)
    g.append(b)
    k0 = g.k.clone()
    big = torch.zeros(D, dtype=torch.bfloat16, device="cuda")
    big[0] = 96.0
    q = b.q.copy()
    q[:, :, 0] = syn.f32_to_bf16_bits(np.float32(8.0))
    bq = syn.Batch(b.geom, b.context_len, b.query_len, b.block_table, q, b.k_new, b.v_new)
    v_host = to_host_bits(g.v)
    rows = [0, 1, 127, 128, 255, 256, Lq - 1]
    cand = set()
    for i in rows:
        left = P + i - window + 1
        cand.update({left - 1, left, left + 1, P + i, P + i + 1})
    for j in sorted(c for c in cand if 0 <= c < P + Lq):
        g.k.copy_(k0)
        blk, slot = int(b.block_table[0, j // 16]), j % 16
        g.k[blk, :, slot, :] = big
        o, _ = g.attend(bq, want_lse=False)
        o = syn.bf16_bits_to_f64(o)
        want = np.repeat(syn.bf16_bits_to_f64(v_host[blk, :, slot, :]), Hq // Hkv, axis=0)
        for i in rows:
            visible = P + i - window + 1 <= j <= P + i
            assert (np.abs(o[i] - want).max() <= 2e-2) == visible, (j, i)
    # the decode sequence: position 2000, window [1701, 2000]
    for j, visible in ((1700, False), (1701, True), (2000, True)):
        g.k.copy_(k0)
        blk, slot = int(b.block_table[1, j // 16]), j % 16
        g.k[blk, :, slot, :] = big
        o, _ = g.attend(bq, want_lse=False)
        o = syn.bf16_bits_to_f64(o)
        want = np.repeat(syn.bf16_bits_to_f64(v_host[blk, :, slot, :]), Hq // Hkv, axis=0)
        assert (np.abs(o[Lq] - want).max() <= 2e-2) == visible, j
    g.close()


def test_windowed_agentic_configuration_at_full_size():
    """configs[3] (16 decode sequences of 8K..32K, a 2048-token chunk over 24,576 cached tokens) as a sliding-window
    layer of 128 tokens with sinks - the geometry of the windowed layers of GPT-OSS - and with a 4096-token window:
    first chunk iteration, decode rows and the edge rows of every q tile against the oracle."""
    for window in (128, 4096):
        sc = syn.config4_agentic(iterations=(0,))
        run_and_check(sc, tile_rows=True, check_append=False, window=window, sinks=sink_values(32, 5))


def test_static_entry_point_honours_window_and_sinks():
    lens = [30000, 17, 4096, 1, 9001, 640]
    sc = small(49, 32, 8, 128, [l - 1 for l in lens], [[1] * len(lens)], NB=4096)
    b = sc.batches[0]
    sinks = sink_values(32, 6)
    g = GpuScenario(sc, window=1000, sinks=sinks)
    g.append(b)
    ctx_o, ctx_lse = g.attend(b)
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((b.total_q, 32), float("nan"), dtype=torch.float32, device="cuda")
    cf.cf_decode_attention_static(g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, out, lse)
    torch.cuda.synchronize()
    assert np.array_equal(to_host_bits(out), ctx_o) and np.array_equal(lse.cpu().numpy(), ctx_lse)
    k_ref, v_ref = g.pools_host()
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len, window=1000,
                                            sinks=sinks.astype(np.float64))
    compare(ctx_o, ctx_lse, ref_o, ref_lse)
    g.close()


# ------------------------------------------------------------------ tensor-parallel head sharding (Section 6.1: one TP4 worker per server)
def _run_shard(ctx, sc, b, g_full, r, ranks, debug_single_partition):
    """Rank r's share of the heads through the ABI: strided views of the SAME pools (the descriptor keeps the
    pool's block stride and says Hkv / ranks heads; the base pointer is moved to the shard's first KV head)."""
    geom = sc.geom
    Hq, Hkv, D, B = geom.num_q_heads, geom.num_kv_heads, geom.head_dim, geom.block_size
    hq, hkv = Hq // ranks, Hkv // ranks
    st = (Hkv * B * D, B * D, D)
    desc = cf.make_desc(hq, hkv, D, B, geom.num_blocks, k_strides=st, v_strides=st)
    k_ptr = g_full.k.data_ptr() + r * hkv * B * D * 2
    v_ptr = g_full.v.data_ptr() + r * hkv * B * D * 2
    q = to_dev_bf16(np.ascontiguousarray(b.q[:, r * hq:(r + 1) * hq, :]))
    bt = torch.from_numpy(b.block_table).cuda()
    out = torch.full((b.total_q, hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((b.total_q, hq), float("nan"), dtype=torch.float32, device="cuda")
    cf.cf_mixed_attention(ctx, desc, q, k_ptr, v_ptr, bt, b.max_blocks, b.context_len, b.query_len, out, lse)
    torch.cuda.synchronize()
    assert cf.cf_get_async_status(ctx) == cf.CF_OK
    return to_host_bits(out), lse.cpu().numpy()


@pytest.mark.parametrize("same_partition", [True, False])
def test_four_head_shards_reproduce_the_unsharded_result(same_partition):
    """The chat-like configuration split four ways by KV-head group, each shard run on its own through the ABI
    on strided views of the same pools, concatenated along the head axis.  With the planner held to one
    partition (one KV chunk per decode sequence, no KV split of prefill items) a head's arithmetic does not
    depend on which other heads ride in the call: the concatenation equals the unsharded call bit for bit.  With
    the planner left to itself the shards are cut differently (fewer heads per call) and agree to rounding;
    both ways the shards match the oracle."""
    sc = syn.config3_chat(iterations=(0,))
    b = sc.batches[0]
    debug = {cf.CF_DEBUG_PREFILL_SPLIT: 1, cf.CF_DEBUG_DECODE_MIN_CHUNK_PAGES: 1 << 20} if same_partition else None
    g = GpuScenario(sc, debug=debug)
    g.append(b)
    full_o, full_lse = g.attend(b)
    shards = [_run_shard(g.ctx, sc, b, g, r, 4, same_partition) for r in range(4)]
    cat_o = np.concatenate([o for o, _ in shards], axis=1)
    cat_lse = np.concatenate([l for _, l in shards], axis=1)
    if same_partition:
        assert np.array_equal(cat_o, full_o) and np.array_equal(cat_lse, full_lse)
    else:
        diff = np.abs(syn.bf16_bits_to_f64(cat_o) - syn.bf16_bits_to_f64(full_o))
        assert diff.max() <= 2e-2 and diff.mean() <= 2e-3
    k_ref, v_ref = g.pools_host()
    rows = syn.tile_edge_rows(b)
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len, rows=rows)
    compare(cat_o, cat_lse, ref_o, ref_lse, rows=rows, label="concatenated shards vs oracle")
    g.close()


# ------------------------------------------------------------------ shared prefixes read once
def _run_shared(sc, share_group, shared_len, expect_shared_items=True):
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    plain_o, plain_lse = g.attend(b)                      # aliased block tables alone already define the result
    geom = sc.geom
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.full((b.total_q, geom.num_q_heads, geom.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((b.total_q, geom.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):                                    # twice: the ticket counters must be back at zero
        out.fill_(float("nan"))
        cf.cf_mixed_attention_shared(g.ctx, g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, b.query_len,
                                     share_group, shared_len, out, lse)
        torch.cuda.synchronize()
        assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
        counts = cf.cf_get_last_plan_counts(g.ctx)
        assert (counts[5] > 0) == expect_shared_items, counts
        k_ref, v_ref = g.pools_host()
        ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len)
        o_bits, lse_h = to_host_bits(out), lse.cpu().numpy()
        compare(o_bits, lse_h, ref_o, ref_lse, label="shared-prefix path vs oracle")
    diff = np.abs(syn.bf16_bits_to_f64(o_bits) - syn.bf16_bits_to_f64(plain_o))
    assert diff.max() <= 2e-2 and diff.mean() <= 2e-3
    g.close()
    return counts


@pytest.mark.parametrize("n_sharers", [2, 4, 8, 16])
@pytest.mark.parametrize("Hq,Hkv,D", [(4, 4, 128), (32, 8, 128), (64, 8, 128), (8, 2, 64)])
def test_shared_prefix_is_read_once_for_all_sharers(n_sharers, Hq, Hkv, D):
    """2 to 16 decode sequences that share a 2048-token prefix (group sizes 1, 4 and 8, both head dims), each with
    a suffix of its own, beside sequences that share nothing and a prefill chunk of the same group."""
    geom = syn.Geometry(Hq, Hkv, D, 16, 4096)
    rng = np.random.default_rng(n_sharers)
    own = [int(x) for x in rng.integers(0, 700, size=n_sharers)] + [900, 3000, 40]
    qlen = [1] * n_sharers + [1, 1, 150]
    group = [0] * n_sharers + [-1, -1, 0]
    sc, sg, sl = syn.shared_prefix_scenario("shared", geom, 61 + n_sharers, 2048, own, qlen, group)
    counts = _run_shared(sc, sg, sl)
    per_set = max(1, 16 // (Hq // Hkv))
    assert counts[6] == n_sharers and counts[5] % ((n_sharers + per_set - 1) // per_set) == 0


def test_two_share_groups_and_a_short_prefix():
    """Two groups with prefixes of their own; a group whose common prefix is shorter than the threshold, a group
    with a single decode member and a member whose shared_len exceeds its context are served the ordinary way."""
    geom = syn.Geometry(32, 8, 128, 16, 4096)
    own = [10, 500, 33, 0, 1200, 77, 5, 300]
    qlen = [1, 1, 1, 1, 1, 1, 1, 1]
    sc, sg, sl = syn.shared_prefix_scenario("two-groups", geom, 71, 4096, own, qlen, [0, 0, 0, 1, 1, 1, 1, -1])
    counts = _run_shared(sc, sg, sl)
    assert counts[6] == 7
    sc, sg, sl = syn.shared_prefix_scenario("short", geom, 72, 128, own[:4], qlen[:4], [0, 0, 0, 0])
    _run_shared(sc, sg, sl, expect_shared_items=False)
    sc, sg, sl = syn.shared_prefix_scenario("lonely", geom, 73, 2048, own[:3], [1, 40, 1], [0, 0, -1])
    _run_shared(sc, sg, sl, expect_shared_items=False)
    # shared_len claims more than a member has: clamped to the member's context minus its new token
    sc, sg, sl = syn.shared_prefix_scenario("clamped", geom, 74, 1024, [0, 0, 0], [1, 1, 1], [0, 0, 0])
    sl[:] = 1 << 20
    counts = _run_shared(sc, sg, sl)
    assert counts[6] == 3


def test_shared_prefix_with_many_chunks_and_the_separate_combine_kernel():
    """A 40K-token shared prefix (many shared chunks per member) with short and long suffixes, merged by the fused
    merge and by the separate combine kernel: identical bits."""
    geom = syn.Geometry(32, 8, 128, 16, 8192)
    sc, sg, sl = syn.shared_prefix_scenario("long-shared", geom, 75, 40000 // 16 * 16, [0, 15, 3000, 9000, 17, 600], [1] * 6, [0] * 6)
    b = sc.batches[0]
    outs = []
    for debug in (None, {cf.CF_DEBUG_SEPARATE_COMBINE: 1}):
        g = GpuScenario(sc, debug=debug)
        g.append(b)
        bt = torch.from_numpy(b.block_table).cuda()
        q = to_dev_bf16(b.q)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((b.total_q, 32), float("nan"), dtype=torch.float32, device="cuda")
        cf.cf_mixed_attention_shared(g.ctx, g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, b.query_len, sg, sl, out, lse)
        torch.cuda.synchronize()
        assert cf.cf_get_last_plan_counts(g.ctx)[5] > 1
        outs.append((to_host_bits(out), lse.cpu().numpy()))
        k_ref, v_ref = g.pools_host()
        g.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len)
    compare(outs[0][0], outs[0][1], ref_o, ref_lse)


# ------------------------------------------------------------------ chunked prefill on pairs of SMs (opt-in kernel)
PAIRS = {cf.CF_DEBUG_PREFILL_PAIRS: 1}


@pytest.mark.parametrize("Hq,Hkv", [(4, 1), (32, 8), (16, 2), (64, 8)])
def test_pair_kernel_ragged_prefill(Hq, Hkv):
    """The two-CTA prefill kernel (four heads of a group per work item, K/V tiles split between two SMs) on ragged
    chunks: group sizes 4 and 8, chunks shorter than a tile, without a prefix, ending in the middle of a page."""
    prefix = [0, 0, 5, 16, 63, 64, 100, 1000, 0, 333, 2000]
    qlen = [2, 64, 65, 17, 1, 128, 129, 200, 300, 31, 700]
    sc = small(5, Hq, Hkv, 128, prefix, [qlen])
    g = GpuScenario(sc, debug=PAIRS)
    g.append(sc.batches[0])
    g.attend(sc.batches[0])
    assert cf.cf_get_last_plan_counts(g.ctx)[7] == 1          # the plan really was a pair plan
    g.close()
    run_and_check(sc, debug=PAIRS)


def test_pair_kernel_mixed_batches_kv_split_window_and_sinks():
    mixed = small(8, 32, 8, 128, [3000, 700, 9000, 50, 0], [[1, 300, 1, 1, 130]])
    run_and_check(mixed, debug=PAIRS)
    for split in (2, 3):
        run_and_check(small(7, 32, 8, 128, [2000, 0, 700, 4097, 300], [[300, 700, 129, 64, 1]]),
                      debug={**PAIRS, cf.CF_DEBUG_PREFILL_SPLIT: split})
    run_and_check(small(9, 32, 8, 128, [3000, 700, 100], [[300, 700, 64]]), window=300, sinks=sink_values(32, 7), debug=PAIRS)
    # more items than pairs of SMs (11 x 8 + 2 x 8 = 104 four-head items for 74 pairs), in the serial and the spatial sequence
    many = small(41, 32, 8, 128, [700, 40, 5000, 300, 17], [[1300, 130, 1, 1, 1]])
    b = many.batches[0]
    g = GpuScenario(many, debug={**PAIRS, cf.CF_DEBUG_PREFILL_SPLIT: 1})
    g.append(b)
    outs = []
    for mode in (0, 1, 10):
        cf.cf_set_overlap(g.ctx, mode)
        outs.append(g.attend(b))
    for o, l in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(l, outs[0][1])
    k_ref, v_ref = g.pools_host()
    rows = syn.tile_edge_rows(b)
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len, rows=rows)
    compare(outs[0][0], outs[0][1], ref_o, ref_lse, rows=rows)
    assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
    g.close()


def test_pair_kernel_chat_configuration_at_full_size():
    sc = syn.config3_chat(iterations=(0, 3))
    run_and_check(sc, tile_rows=True, check_append=False, debug=PAIRS)


# ------------------------------------------------------------------ fp8 (e4m3) KV cache
def scales(Hkv, seed=0, pow2=False):
    rng = np.random.default_rng(200 + seed)
    if pow2:
        return (2.0 ** rng.integers(-6, -2, size=Hkv)).astype(np.float32), (2.0 ** rng.integers(-6, -2, size=Hkv)).astype(np.float32)
    return rng.uniform(0.01, 0.05, size=Hkv).astype(np.float32), rng.uniform(0.01, 0.05, size=Hkv).astype(np.float32)


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (8, 8), (16, 2), (64, 8)])
def test_fp8_cache_decode(Hq, Hkv):
    """Decode over an e4m3 cache: the append stores the oracle's codes bit for bit (whole-pool compare), attention
    matches the oracle's reading of the same codes; ragged lengths, split and unsplit sequences."""
    lens = [1, 2, 15, 16, 17, 31, 33, 127, 129, 255, 700, 1025, 2500, 4097, 9000, 20000]
    sc = small(3, Hq, Hkv, 128, [l - 1 for l in lens], [[1] * len(lens)], NB=4096)
    run_and_check(sc, fp8=scales(Hkv, 1))


def test_fp8_cache_mixed_batches_and_chunked_prefill():
    """Prefill chunks over an e4m3 cache (their pages are expanded into the bf16 staging area first), beside decode
    sequences, over several iterations; with KV-split items, with a sliding window and sinks."""
    prefix = [300, 40, 999, 0, 5000]
    qlens = [[100, 1, 1, 64, 1], [37, 1, 1, 64, 1], [200, 1, 1, 1, 300]]
    run_and_check(small(9, 32, 8, 128, prefix, qlens), fp8=scales(8, 2))
    run_and_check(small(9, 32, 8, 128, prefix, qlens), fp8=scales(8, 3, pow2=True), window=150, sinks=sink_values(32, 8))
    run_and_check(small(7, 32, 8, 128, [2000, 0, 700, 4097, 300], [[300, 700, 129, 64, 1]]), fp8=scales(8, 4),
                  debug={cf.CF_DEBUG_PREFILL_SPLIT: 3})
    run_and_check(small(7, 4, 4, 128, [2000, 0, 700], [[300, 700, 1]]), fp8=scales(4, 5))


def test_fp8_cache_values_at_the_edges_of_the_format():
    """New K/V values far outside the format's range saturate at +-448 * scale and tiny ones fall on the subnormal
    grid - on both sides alike, because the rounding decision is taken in fp32 by both."""
    sc = small(11, 8, 2, 128, [100, 40], [[60, 1]])
    b = sc.batches[0]
    rng = np.random.default_rng(1)
    kn = syn.bf16_bits_to_f32(b.k_new) * rng.choice([1e-4, 1.0, 300.0], size=b.k_new.shape).astype(np.float32)
    vn = syn.bf16_bits_to_f32(b.v_new) * rng.choice([1e-4, 1.0, 40.0], size=b.v_new.shape).astype(np.float32)
    b.k_new[...] = syn.f32_to_bf16_bits(kn)
    b.v_new[...] = syn.f32_to_bf16_bits(vn)
    # (scales small enough that the saturated values, +-448 * scale, keep scores and outputs of order one: the
    # comparison's absolute tolerances on the output and on lse are meant for such magnitudes)
    stats = run_and_check(sc, fp8=(np.array([0.004, 0.003], np.float32), np.array([0.004, 0.003], np.float32)))
    print(stats)


def test_fp8_cache_at_full_size_and_what_is_refused():
    sc = syn.config3_chat(iterations=(0,))
    run_and_check(sc, tile_rows=True, check_append=False, fp8=scales(8, 6))
    # head_dim 64 and the allocation-free entry point do not take an fp8 cache
    ks = torch.ones(2, device="cuda")
    d64 = cf.make_desc(8, 2, 64, 16, 64, kv_dtype=cf.CF_KV_FP8_E4M3, k_scale=ks, v_scale=ks)
    assert cf.cf_plan_inspect(d64, [5], [1], 8, check=False)[0] == cf.CF_ERR_UNSUPPORTED
    d128 = cf.make_desc(8, 2, 128, 16, 64, kv_dtype=cf.CF_KV_FP8_E4M3, k_scale=ks, v_scale=ks)
    assert cf.cf_decode_attention_static(d128, 1, 1, 1, 1, 8, [5], 1, check=False) == cf.CF_ERR_UNSUPPORTED
    no_scale = cf.make_desc(8, 2, 128, 16, 64, kv_dtype=cf.CF_KV_FP8_E4M3)
    assert cf.cf_plan_inspect(no_scale, [5], [1], 8, check=False)[0] == cf.CF_ERR_INVALID_ARG


def test_property_random_batches_of_every_variant():
    """Seeded random geometries, lengths and launch sequences, each with a random variant of the layer: a sliding
    window, sinks, an fp8 cache (head_dim 128), or several at once.  Every row against the oracle."""
    rng = np.random.default_rng(4242)
    ctx = cf.cf_create(0)
    try:
        for trial in range(36):
            fp8 = rng.random() < 0.3
            Hkv = int(rng.choice([1, 2, 4, 8]))
            G = int(rng.choice([1, 2, 4, 8]))
            D = 128 if fp8 else int(rng.choice([64, 128]))
            S = int(rng.integers(1, 9))
            kind = int(rng.integers(0, 3))
            if kind == 0:      # many small chunks and decode sequences
                qlen = [int(x) for x in rng.choice([0, 1, 1, 1, 2, 31, 128, 129, 300, 513], size=S)]
                prefix = [int(x) for x in rng.integers(0, 1500, size=S)]
            elif kind == 1:    # long decode sequences (many KV chunks) beside one chunk
                qlen = [1] * S
                qlen[0] = int(rng.integers(2, 700))
                prefix = [int(x) for x in rng.integers(0, 12000, size=S)]
            else:              # one large chunk (sometimes more work items than SMs)
                qlen = [int(rng.integers(300, 1500))] + [1] * (S - 1)
                prefix = [int(rng.integers(0, 3000))] + [int(x) for x in rng.integers(0, 6000, size=S - 1)]
            if sum(qlen) == 0:
                qlen[0] = 1
            window = int(rng.choice([0, 0, 1, 16, 100, 128, 1000, 4096]))
            sinks = (rng.standard_normal(Hkv * G) * 2).astype(np.float32) if rng.random() < 0.5 else None
            need = sum((p + q + 15) // 16 for p, q in zip(prefix, qlen)) + 8
            sc = syn.scenario_from_lengths("rv", syn.Geometry(Hkv * G, Hkv, D, 16, max(256, int(need * 1.1))), 5100 + trial,
                                           prefix, [qlen], shuffle_seqs=True)
            cf.cf_set_overlap(ctx, int(rng.choice([0, 1, 1, 7, 40, 129])))
            scales = ((0.004 + 0.004 * rng.random(Hkv)).astype(np.float32),
                      (0.003 + 0.003 * rng.random(Hkv)).astype(np.float32)) if fp8 else None
            run_and_check(sc, ctx=ctx, window=window, sinks=sinks, fp8=scales, max_prefill_rows=(24 if sum(qlen) > 400 else 0))
    finally:
        cf.cf_set_overlap(ctx, 1)
        cf.cf_destroy(ctx)
