"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on seeded inputs that span several tiles, ragged tails and the degenerate cases."""
import numpy as np
import pytest
import torch

import cf_synth as syn
import oracle
import paper_2609_27085_b200 as cf
from harness import GpuScenario, compare, run_and_check, to_dev_bf16, to_host_bits

pytestmark = pytest.mark.gpu


def small(seed, Hq, Hkv, D, prefix, qlens, NB=2048, shuffle=False):
    return syn.scenario_from_lengths("t", syn.Geometry(Hq, Hkv, D, 16, NB), seed, prefix, qlens, shuffle_seqs=shuffle)


def test_config1_tiny():
    stats = run_and_check(syn.config1_tiny())
    print(stats)


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 64), (8, 8, 128), (8, 4, 128), (32, 8, 128), (64, 8, 128), (16, 2, 64), (8, 1, 64)])
def test_decode_only_ragged(Hq, Hkv, D):
    lens = [1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 127, 129, 255, 700, 1023, 1025, 2500, 4097, 9000]
    run_and_check(small(3, Hq, Hkv, D, [l - 1 for l in lens], [[1] * len(lens)]))


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 64), (4, 4, 128), (32, 8, 128), (16, 2, 128)])
def test_prefill_only_ragged(Hq, Hkv, D):
    prefix = [0, 0, 5, 16, 63, 64, 100, 1000, 0, 333]
    qlen = [2, 64, 65, 17, 1, 128, 129, 200, 300, 31]
    run_and_check(small(5, Hq, Hkv, D, prefix, [qlen]))


def test_mixed_shuffled_order_with_empty_sequences():
    prefix = [10, 0, 500, 77, 0, 2000, 31, 640, 5, 1]
    qlen = [1, 90, 1, 0, 1, 1, 130, 1, 0, 64]
    run_and_check(small(7, 32, 8, 128, prefix, [qlen], shuffle=True))


def test_multi_iteration_chunked_prefill_with_growing_decodes():
    prefix = [300, 40, 999, 0]
    qlens = [[100, 1, 1, 64], [37, 1, 1, 64], [200, 1, 1, 1]]
    run_and_check(small(9, 8, 2, 64, prefix, qlens))
    run_and_check(small(9, 32, 8, 128, prefix, qlens))


def test_nhd_layout_and_custom_scale():
    prefix = [10, 700, 0, 2047]
    qlen = [1, 1, 80, 1]
    run_and_check(small(11, 32, 8, 128, prefix, [qlen]), layout="NHD")
    run_and_check(small(11, 8, 2, 64, prefix, [qlen]), layout="NHD", softmax_scale=0.2)


def test_long_split_decode_uses_partials_and_combine():
    sc = small(13, 32, 8, 128, [40000 - 1, 123], [[1, 1]], NB=4096)
    d = cf.make_desc(32, 8, 128, 16, 4096)
    _, dec, comb, _, parts = cf.cf_plan_inspect(d, sc.batches[0].context_len, sc.batches[0].query_len, sc.batches[0].max_blocks)
    assert parts >= 2 and len(comb) == 1
    run_and_check(sc)


@pytest.mark.parametrize("Hq,Hkv,D", [(16, 2, 64), (8, 1, 128), (64, 8, 128)])
def test_many_chunk_merge_other_geometries(Hq, Hkv, D):
    """Sequences cut into up to ~40 chunks (the fused merge folds its partials eight at a time) beside
    one- and two-chunk sequences, for head_dim 64, a single KV head and group size 8."""
    sc = small(17, Hq, Hkv, D, [20000 - 1, 9000 - 1, 511, 513, 4100], [[1, 1, 1, 1, 1]], NB=4096)
    d = cf.make_desc(Hq, Hkv, D, 16, 4096)
    b = sc.batches[0]
    _, dec, comb, _, parts = cf.cf_plan_inspect(d, b.context_len, b.query_len, b.max_blocks)
    assert max(c[2] for c in comb) > 8
    run_and_check(sc)


def test_chunking_invariance_on_gpu():
    """One 300-token unit vs. three ragged units (Section 4.4): same rows within tolerance, and both match the oracle."""
    one = small(15, 8, 2, 64, [77], [[300]])
    cut = small(15, 8, 2, 64, [77], [[300]])
    b = one.batches[0]
    g1 = GpuScenario(one)
    g1.append(b)
    o_full, _ = g1.attend(b)
    g1.close()
    g2 = GpuScenario(cut)
    at, have = 0, 77
    outs = []
    for c in (130, 1, 169):
        have += c
        part = syn.Batch(b.geom, np.array([have], np.int32), np.array([c], np.int32), b.block_table,
                         b.q[at:at + c], b.k_new[at:at + c], b.v_new[at:at + c])
        g2.append(part)
        outs.append(g2.attend(part)[0])
        at += c
    g2.close()
    o_cut = np.concatenate(outs)
    diff = np.abs(syn.bf16_bits_to_f64(o_full) - syn.bf16_bits_to_f64(o_cut))
    assert diff.max() <= 2e-2 and diff.mean() <= 2e-3


def test_determinism_and_unrelated_calls():
    sc = small(17, 32, 8, 128, [5000, 20, 300], [[1, 1, 150]])
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    first, lse0 = g.attend(b)
    other = small(18, 8, 2, 64, [900], [[1]])
    g_other = GpuScenario(other, ctx=g.ctx)
    g_other.append(other.batches[0])
    g_other.attend(other.batches[0])
    for _ in range(10):
        o, lse = g.attend(b)
        assert np.array_equal(o, first) and np.array_equal(lse, lse0)
    g.close()


def _spike_run(sc, cand, rows_to_check, spike, debug=None):
    """Plants, at each candidate position in turn, a key whose score towers over the rest and checks
    that every listed row returns that key's value if it can see the key and is unaffected if not."""
    b = sc.batches[0]
    geom = sc.geom
    Hq, Hkv, D = geom.num_q_heads, geom.num_kv_heads, geom.head_dim
    Lc, Lq = int(b.context_len[0]), int(b.query_len[0])
    P = Lc - Lq
    g = GpuScenario(sc, debug=debug)
    g.append(b)
    k0 = g.k.clone()
    big = torch.zeros(D, dtype=torch.bfloat16, device="cuda")
    big[0] = spike
    q = b.q.copy()
    q[:, :, 0] = syn.f32_to_bf16_bits(np.float32(8.0))       # every row: score of the planted key = 8 * spike / sqrt(D)
    bq = syn.Batch(b.geom, b.context_len, b.query_len, b.block_table, q, b.k_new, b.v_new)
    v_host = to_host_bits(g.v)
    for j in sorted(set(int(x) for x in cand if 0 <= x < Lc)):
        g.k.copy_(k0)
        blk, slot = int(b.block_table[0, j // 16]), j % 16
        g.k[blk, :, slot, :] = big
        o, _ = g.attend(bq, want_lse=False)
        o = syn.bf16_bits_to_f64(o)                          # [Lq, Hq, D]
        vj = syn.bf16_bits_to_f64(v_host[blk, :, slot, :])   # [Hkv, D]
        want = np.repeat(vj, Hq // Hkv, axis=0)
        for i in rows_to_check:
            if j <= P + i:
                assert np.abs(o[i] - want).max() <= 2e-2, (j, i)
            else:
                assert np.abs(o[i] - want).max() > 0.5, (j, i)   # invisible key: output is the ordinary average
    g.close()


def test_spike_keys_decode():
    """A key planted ~68 nats above the rest must be found wherever it sits in a split decode sequence: page
    edges, both sides of every chunk edge of the plan, the last positions."""
    Hq, Hkv, D = 8, 2, 128
    Lc = 20000
    sc = small(19, Hq, Hkv, D, [Lc - 1], [[1]], NB=2048)
    b = sc.batches[0]
    d = cf.make_desc(Hq, Hkv, D, 16, 2048)
    _, dec, _, _, _ = cf.cf_plan_inspect(d, b.context_len, b.query_len, b.max_blocks)
    assert len(dec) > 2
    cand = {0, 15, 16, 63, 64, 127, 128, Lc - 2, Lc - 1}
    for e in sorted(set(int(x) for x in dec[:, 2]) | set(int(x) for x in dec[:, 3])):
        cand.update({e - 1, e, e + 1})
    _spike_run(sc, cand, [0], 96.0)


@pytest.mark.parametrize("split", [1, 0, 3])
@pytest.mark.parametrize("spike", [96.0, 192.0])
def test_spike_keys_prefill(split, spike):
    """Chunked prefill, 700 new tokens over a 3100-token prefix (interior tiles of the lean MMA loop, a ragged
    last q tile): the planted key sits on both sides of every 128-token KV tile boundary, of every KV-range
    boundary of the KV split (none, the cost model's, a forced 3-way one), of the prefix/chunk boundary and of the diagonal, and on the columns of
    later tiles whose exponentials are evaluated by the polynomial route (14, 15, 30, 31 of every 32).  spike =
    192 puts the key ~136 nats (196 in log2 units) above the rest: far outside what an exponent field can
    hold against a stale reference maximum, so the rescale path must catch it in every column."""
    Hq, Hkv, D = 8, 2, 128
    Lq, P = 700, 3100
    Lc = P + Lq
    sc = small(19, Hq, Hkv, D, [P], [[Lq]], NB=2048)
    b = sc.batches[0]
    d = cf.make_desc(Hq, Hkv, D, 16, 2048)
    _, _, _, pre, _, counts = cf.cf_plan_inspect(d, b.context_len, b.query_len, b.max_blocks, prefill_force_split=split,
                                                 want_counts=True)
    assert (counts[5] > 0) == (split != 1)        # 1: never split; 0: the cost model splits these 24 items; 3: forced
    cand = {0, 15, 16, 63, 64, P - 1, P, P + 1, Lc - 2, Lc - 1}
    for t in range(0, Lc + 128, 128):
        cand.update({t - 1, t, t + 1})
    for e in sorted(set(int(x) * 128 for x in pre[:, 6]) | set(int(x) * 128 for x in pre[:, 7])):
        cand.update({e - 1, e, e + 1})
    for t in (1, 2, 7, 13, P // 128, (Lc - 1) // 128):
        cand.update({128 * t + c for c in (14, 15, 30, 31, 46, 47, 126, 127)})
    rows = [0, 1, 127, 128, 300, 511, 512, Lq - 2, Lq - 1]
    _spike_run(sc, cand, rows, spike, debug={cf.CF_DEBUG_PREFILL_SPLIT: split} if split else None)


def test_abi_rejects_bad_arguments_without_launching():
    sc = small(21, 8, 2, 64, [10], [[1]])
    b = sc.batches[0]
    g = GpuScenario(sc)
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.zeros_like(q)
    A = dict(check=False)
    assert cf.cf_mixed_attention(g.ctx, g.desc, q, g.k, g.v, bt, b.max_blocks, [5], [6], out, **A) == cf.CF_ERR_INVALID_ARG
    assert cf.cf_mixed_attention(g.ctx, g.desc, q, g.k, g.v, bt, 0, [11], [1], out, **A) == cf.CF_ERR_OUT_OF_RANGE
    assert cf.cf_mixed_attention(g.ctx, g.desc, None, g.k, g.v, bt, b.max_blocks, [11], [1], out, **A) == cf.CF_ERR_INVALID_ARG
    assert cf.cf_mixed_attention(g.ctx, g.desc, q, g.k, g.v, bt, b.max_blocks, [11], [1], None, **A) == cf.CF_ERR_INVALID_ARG
    bad = cf.make_desc(8, 2, 96, 16, 2048)
    assert cf.cf_mixed_attention(g.ctx, bad, q, g.k, g.v, bt, b.max_blocks, [11], [1], out, **A) == cf.CF_ERR_UNSUPPORTED
    assert cf.cf_kv_append(g.ctx, g.desc, g.k, g.v, None, None, bt, b.max_blocks, [11], [1], **A) == cf.CF_ERR_INVALID_ARG
    assert cf.cf_kv_append(g.ctx, g.desc, g.k, g.v, q, q, bt, b.max_blocks, [11], [12], **A) == cf.CF_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert (out == 0).all()
    assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
    g.close()


def test_fixed_workspace_too_small_is_reported():
    sc = small(23, 32, 8, 128, [60000, 60000, 60000], [[1, 1, 1]], NB=12288)     # ~90 partial slots x 16 KB: more than the 1 MB a tiny request is rounded up to
    b = sc.batches[0]
    ctx = cf.cf_create(0, workspace_bytes=4096)
    g = GpuScenario(sc, ctx=ctx)
    bt = torch.from_numpy(b.block_table).cuda()
    q = to_dev_bf16(b.q)
    out = torch.zeros_like(q)
    st = cf.cf_mixed_attention(ctx, g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, b.query_len, out, check=False)
    assert st == cf.CF_ERR_WORKSPACE
    cf.cf_destroy(ctx)


def test_host_step_matches_device_step():
    sc = small(25, 32, 8, 128, [100, 3000, 50], [[70, 1, 1]])
    b = sc.batches[0]
    g = GpuScenario(sc)
    bt = torch.from_numpy(b.block_table).cuda()
    qh = torch.from_numpy(b.q.view(np.int16)).pin_memory()
    kh = torch.from_numpy(b.k_new.view(np.int16)).pin_memory()
    vh = torch.from_numpy(b.v_new.view(np.int16)).pin_memory()
    oh = torch.zeros_like(qh).pin_memory()
    cf.cf_mixed_step_host(g.ctx, g.desc, qh, kh, vh, g.k, g.v, bt, b.max_blocks, b.context_len, b.query_len, oh)
    cf.cf_host_steps_flush(g.ctx)
    torch.cuda.synchronize()
    o_dev, _ = g.attend(b, want_lse=False)          # caches were appended by the host step
    assert np.array_equal(oh.numpy().view(np.uint16), o_dev)
    k_ref, v_ref = sc.k_pool.copy(), sc.v_pool.copy()
    oracle.kv_append(k_ref, v_ref, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len)
    compare(o_dev, None, ref_o, ref_lse)
    g.close()


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait that nothing satisfies gives up by itself; the host reads CF_ERR_TIMEOUT and the same
    context then still computes correct attention."""
    sc = small(27, 32, 8, 128, [300, 40], [[130, 1]])
    b = sc.batches[0]
    g = GpuScenario(sc)
    cf.cf_selftest_bounded_wait(g.ctx)
    torch.cuda.synchronize()
    assert cf.cf_get_async_status(g.ctx) == cf.CF_ERR_TIMEOUT
    assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
    g.append(b)
    o_bits, lse = g.attend(b)
    k_ref, v_ref = sc.k_pool.copy(), sc.v_pool.copy()
    oracle.kv_append(k_ref, v_ref, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len)
    compare(o_bits, lse, ref_o, ref_lse)
    g.close()


def test_property_random_batches():
    """Random small batches: sequence counts, chunk lengths, prefixes, group sizes, head dims, and the launch
    sequence (serial, default spatial share, a 7-CTA front grid)."""
    rng = np.random.default_rng(2024)
    ctx = cf.cf_create(0)
    for trial in range(36):
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 4, 8]))
        D = int(rng.choice([64, 128]))
        S = int(rng.integers(1, 9))
        qlen = [int(x) for x in rng.choice([0, 1, 1, 1, 2, 7, 31, 64, 127, 128, 129, 200, 300], size=S)]
        prefix = [int(x) for x in rng.integers(0, 601, size=S)]
        prefix = [p if q > 0 else max(p, 0) for p, q in zip(prefix, qlen)]
        if sum(qlen) == 0:
            qlen[0] = 1
        cf.cf_set_overlap(ctx, int(rng.choice([0, 1, 7])))
        run_and_check(small(3000 + trial, Hkv * G, Hkv, D, prefix, [qlen], NB=1024, shuffle=True), ctx=ctx)
    cf.cf_destroy(ctx)


def test_separate_combine_kernel_gives_the_bits_of_the_fused_merge():
    """The split-K merge runs inside the decode kernel by default; the test-only switch CF_DEBUG_SEPARATE_COMBINE
    keeps the separate combine kernel.  Same merge routine, same chunk order: identical bits."""
    sc = small(47, 32, 8, 128, [9000, 5000, 300, 16000, 2047], [[1, 1, 1, 1, 1]], NB=4096)
    b = sc.batches[0]
    fused = GpuScenario(sc)
    fused.append(b)
    o1, l1 = fused.attend(b)
    assert cf.cf_get_last_launch_count(fused.ctx) == 1
    sep = GpuScenario(sc, debug={cf.CF_DEBUG_SEPARATE_COMBINE: 1})
    sep.append(b)
    o2, l2 = sep.attend(b)
    assert cf.cf_get_last_launch_count(sep.ctx) == 2
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)
    for _ in range(3):                       # the ticket counters are back at zero after every launch
        o3, l3 = fused.attend(b)
        assert np.array_equal(o1, o3) and np.array_equal(l1, l3)
    fused.close()
    sep.close()


def test_more_prefill_items_than_sms():
    """A chunk whose q tiles x head pairs exceed the SM count (11 tiles x 16 pairs + 2 x 16 = 208 items, ragged
    last tiles): every persistent CTA works through several items, in the serial and in the spatial sequence,
    with and without decode sequences beside it (KV split off, so that all sequences run one plan)."""
    for qlen in ([[1300, 130]], [[1300, 130, 1, 1, 1]]):
        prefix = [700, 40, 5000, 300, 17][:len(qlen[0])]
        sc = small(41, 32, 8, 128, prefix, qlen, NB=2048)
        b = sc.batches[0]
        g = GpuScenario(sc, debug={cf.CF_DEBUG_PREFILL_SPLIT: 1})
        g.append(b)
        outs = []
        for mode in (0, 1, 5):
            cf.cf_set_overlap(g.ctx, mode)
            outs.append(g.attend(b))
        cf.cf_set_overlap(g.ctx, 1)
        for o, l in outs[1:]:
            assert np.array_equal(o, outs[0][0]) and np.array_equal(l, outs[0][1])
        k_ref, v_ref = sc.k_pool.copy(), sc.v_pool.copy()
        oracle.kv_append(k_ref, v_ref, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
        rows = syn.sample_rows(b, 96)
        ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len, rows=rows)
        compare(outs[0][0], outs[0][1], ref_o, ref_lse, rows=rows)
        assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
        g.close()


def test_spatial_sequence_is_bit_identical_to_the_serial_sequence():
    """With the planner's KV split switched off the plan does not depend on the launch sequence, and then
    neither does any bit of the result: which CTA runs an item, and when, never matters."""
    sc = small(29, 32, 8, 128, [3000, 700, 9000, 50, 0], [[1, 300, 1, 1, 130]], NB=2048)
    b = sc.batches[0]
    g = GpuScenario(sc, debug={cf.CF_DEBUG_PREFILL_SPLIT: 1})
    g.append(b)
    cf.cf_set_overlap(g.ctx, 0)
    serial, lse0 = g.attend(b)
    # default share of the SMs; then 8 and 3 front CTAs, so that every CTA works through several items and
    # the second grid (behind decode, same queue) takes part
    for n in (1, 1, 8, 3, 8):
        cf.cf_set_overlap(g.ctx, n)
        o, lse = g.attend(b)
        assert np.array_equal(o, serial) and np.array_equal(lse, lse0)
    cf.cf_set_overlap(g.ctx, 1)
    assert cf.cf_get_async_status(g.ctx) == 0
    k_ref, v_ref = sc.k_pool.copy(), sc.v_pool.copy()
    oracle.kv_append(k_ref, v_ref, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_ref, v_ref, b.block_table, b.context_len, b.query_len)
    compare(serial, lse0, ref_o, ref_lse)
    g.close()


def test_spatial_sequence_without_the_resident_wait():
    """By default decode waits, through a stream memory operation, until the front prefill CTAs hold their SMs;
    CF_DEBUG_SPATIAL_NO_WAIT (test-only switch) leaves the order to the launches.  Same plan, same bits either
    way, over repeated calls."""
    sc = small(31, 32, 8, 128, [3000, 700, 9000, 50, 0], [[1, 300, 1, 1, 130]], NB=2048)
    b = sc.batches[0]
    plain = GpuScenario(sc)
    plain.append(b)
    o0, l0 = plain.attend(b)
    waited = GpuScenario(sc, debug={cf.CF_DEBUG_SPATIAL_NO_WAIT: 1})      # (the variable keeps its name: this is the one without the wait)
    waited.append(b)
    for n in (1, 1, 5, 1):
        cf.cf_set_overlap(waited.ctx, n)
        o1, l1 = waited.attend(b)
        if n == 1:
            assert np.array_equal(o0, o1) and np.array_equal(l0, l1)
    assert cf.cf_get_async_status(waited.ctx) == 0
    plain.close()
    waited.close()


def test_pipelined_host_steps_keep_their_order():
    """Six host-buffer steps back to back (copies of neighbouring steps overlap the kernels): every
    step's read-back equals the device-buffer path run step by step on a second copy of the caches."""
    prefix = [300, 40, 999, 0]
    qlens = [[100, 1, 1, 64], [37, 1, 1, 64], [200, 1, 1, 1], [1, 1, 1, 1], [64, 1, 1, 130], [5, 1, 1, 1]]
    sc = small(31, 32, 8, 128, prefix, qlens, NB=1024)
    ga, gb = GpuScenario(sc), GpuScenario(sc)
    outs, keep = [], []
    for b in sc.batches:
        bt = torch.from_numpy(b.block_table).cuda()
        qh = torch.from_numpy(b.q.view(np.int16)).pin_memory()
        kh = torch.from_numpy(b.k_new.view(np.int16)).pin_memory()
        vh = torch.from_numpy(b.v_new.view(np.int16)).pin_memory()
        oh = torch.zeros_like(qh).pin_memory()
        cf.cf_mixed_step_host(ga.ctx, ga.desc, qh, kh, vh, ga.k, ga.v, bt, b.max_blocks, b.context_len, b.query_len, oh)
        outs.append(oh)
        keep.append((bt, qh, kh, vh))
    cf.cf_host_steps_flush(ga.ctx)
    torch.cuda.synchronize()
    for b, oh in zip(sc.batches, outs):
        gb.append(b)
        ref, _ = gb.attend(b, want_lse=False)
        assert np.array_equal(oh.numpy().view(np.uint16), ref), b.label
    ga.close()
    gb.close()


def test_planned_calls_match_and_replay_from_a_cuda_graph():
    """Plan once, launch per layer: the planned calls give the bits of the unplanned ones, and a CUDA
    graph captured around them replays with the same result."""
    sc = small(33, 32, 8, 128, [3000, 700, 9000, 50, 0], [[1, 300, 1, 1, 130]], NB=2048)
    b = sc.batches[0]
    ga, gb = GpuScenario(sc), GpuScenario(sc)
    ga.append(b)
    ref, ref_lse = ga.attend(b)
    bt = torch.from_numpy(b.block_table).cuda()
    q, kn, vn = to_dev_bf16(b.q), to_dev_bf16(b.k_new), to_dev_bf16(b.v_new)
    out = torch.zeros_like(q)
    lse = torch.zeros((b.total_q, 32), dtype=torch.float32, device="cuda")
    plan = cf.cf_plan_create(gb.ctx, gb.desc, b.context_len, b.query_len, b.max_blocks)
    cf.cf_kv_append_planned(plan, gb.k, gb.v, kn, vn, bt)
    cf.cf_mixed_attention_planned(plan, q, gb.k, gb.v, bt, out, lse)
    torch.cuda.synchronize()
    assert np.array_equal(to_host_bits(gb.k), to_host_bits(ga.k)) and np.array_equal(to_host_bits(gb.v), to_host_bits(ga.v))
    assert np.array_equal(to_host_bits(out), ref) and np.array_equal(lse.cpu().numpy(), ref_lse)
    # capture the two planned calls of one layer and replay them
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        out.zero_()
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            cf.cf_kv_append_planned(plan, gb.k, gb.v, kn, vn, bt, stream=side)
            cf.cf_mixed_attention_planned(plan, q, gb.k, gb.v, bt, out, lse, stream=side)
    for _ in range(3):       # the prefill work queue is put back to zero by the kernel itself between replays
        out.zero_()
        lse.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(to_host_bits(out), ref) and np.array_equal(lse.cpu().numpy(), ref_lse)
    assert cf.cf_get_async_status(gb.ctx) == cf.CF_OK
    del graph
    cf.cf_plan_destroy(plan)
    ga.close()
    gb.close()


def test_cost_model_tracks_measured_kernel_times():
    """cf_estimate_us (host model, Section 4.2's compute credit) against CUDA-event times of the
    kernels on two reduced workloads: within 30 %."""
    import bench
    for case in ("decode_small", "prefill_small"):
        sc = bench.small_case(case)
        b = sc.batches[0]
        g = GpuScenario(sc)
        g.append(b)
        for _ in range(3):
            g.attend(b, want_lse=False, poison=False)
        cf.cf_set_timing(g.ctx, True)
        for _ in range(5):
            g.attend(b, want_lse=False, poison=False)
        ms_dec, ms_comb, ms_pre, n = cf.cf_get_timing_sums(g.ctx)
        cf.cf_set_timing(g.ctx, False)
        est_dec, est_comb, est_pre = cf.cf_estimate_us(g.desc, b.context_len, b.query_len, b.max_blocks, 148)
        if case == "decode_small":
            assert abs(est_dec / (1e3 * ms_dec / n) - 1.0) < 0.3, (est_dec, ms_dec / n)
        else:
            assert abs(est_pre / (1e3 * ms_pre / n) - 1.0) < 0.3, (est_pre, ms_pre / n)
        g.close()


def test_validate_block_table_finds_entries_outside_the_pool():
    sc = small(35, 8, 2, 64, [100, 40, 0], [[1, 20, 5]], NB=64)
    b = sc.batches[0]
    g = GpuScenario(sc)
    bt = torch.from_numpy(b.block_table).cuda()
    assert cf.cf_validate_block_table(g.ctx, g.desc, bt, b.max_blocks, b.context_len, b.query_len) == 0
    bad = b.block_table.copy()
    bad[0, 3] = 64            # one past the pool
    bad[1, 0] = -5
    bad[2, 3] = 9999          # beyond this sequence's used entries: not dereferenced, not counted
    assert cf.cf_validate_block_table(g.ctx, g.desc, torch.from_numpy(bad).cuda(), b.max_blocks, b.context_len, b.query_len) == 2
    g.close()


def test_sequences_sharing_prefix_pages():
    """Radix-cache reuse: several sequences whose block tables point at the same prefix pages
    (Section 4.4: a lookup determines how much of the prompt is reusable)."""
    geom = syn.Geometry(32, 8, 128, 16, 512)
    rng = np.random.default_rng(37)
    k_pool, v_pool = syn.empty_pools(geom)
    shared = np.arange(100, 100 + 40, dtype=np.int32)            # 640 shared prefix tokens
    syn.fill_prefix(rng, geom, k_pool, shared, 640)
    syn.fill_prefix(rng, geom, v_pool, shared, 640)
    prefix = [640 + 35, 640 + 300, 640]                          # own suffixes beyond the shared pages
    qlen = [1, 150, 1]
    table = np.full((3, 80), -1, dtype=np.int32)
    nxt = 200
    for s in range(3):
        table[s, :40] = shared
        own = (prefix[s] + qlen[s] + 15) // 16 - 40
        table[s, 40:40 + own] = np.arange(nxt, nxt + own)
        nxt += own
        n_own = prefix[s] - 640
        if n_own:
            syn.fill_prefix(rng, geom, k_pool, table[s, 40:], n_own)
            syn.fill_prefix(rng, geom, v_pool, table[s, 40:], n_own)
    # sequence 2 appends its new token into a fresh page; the shared pages are never written
    b = syn.make_batch(rng, geom, np.array(prefix) + np.array(qlen), qlen, table, label="shared-prefix")
    sc = syn.Scenario("shared", geom, k_pool, v_pool, [b])
    run_and_check(sc)


@pytest.mark.parametrize("k", [2, 3])
def test_kv_split_prefill_items_match_the_oracle(k):
    """Every tcgen05 prefill item cut into k KV ranges (fp32 partials + the prefill combine kernel):
    group sizes 1, 4 and 8, ragged chunks, a chunk with no prefix."""
    prefix = [2000, 0, 700, 4097, 300]
    qlen = [300, 700, 129, 64, 1]
    for Hq, Hkv in ((4, 4), (32, 8), (16, 2)):
        sc = small(41 + Hq, Hq, Hkv, 128, prefix, [qlen], NB=2048)
        d = cf.make_desc(Hq, Hkv, 128, 16, 2048)
        b = sc.batches[0]
        counts = cf.cf_plan_inspect(d, b.context_len, b.query_len, b.max_blocks, prefill_force_split=k, want_counts=True)[5]
        assert counts[5] > 0                                  # some items really were split
        run_and_check(sc, debug={cf.CF_DEBUG_PREFILL_SPLIT: k})


def test_block_ids_outside_the_pool_are_reported_not_dereferenced():
    """A block-table entry in use that lies outside the pool: nothing is read or written through it, and
    cf_get_async_status reports CF_ERR_OUT_OF_RANGE once (decode, prefill and append paths)."""
    sc = small(51, 8, 2, 128, [100, 700, 300], [[1, 1, 140]], NB=128)
    b = sc.batches[0]
    g = GpuScenario(sc)
    g.append(b)
    k_before, v_before = to_host_bits(g.k), to_host_bits(g.v)
    for s, col, val in ((0, 2, 128), (1, 40, -7), (2, 5, 1 << 28)):
        bad = b.block_table.copy()
        bad[s, col] = val
        bt = torch.from_numpy(bad).cuda()
        q = to_dev_bf16(b.q)
        out = torch.zeros_like(q)
        cf.cf_mixed_attention(g.ctx, g.desc, q, g.k, g.v, bt, b.max_blocks, b.context_len, b.query_len, out)
        torch.cuda.synchronize()
        assert cf.cf_get_async_status(g.ctx) == cf.CF_ERR_OUT_OF_RANGE
        assert cf.cf_get_async_status(g.ctx) == cf.CF_OK
    # append aimed at a page outside the pool: the row is not written anywhere
    bad = b.block_table.copy()
    bad[0, (int(b.context_len[0]) - 1) // 16] = 4096
    cf.cf_kv_append(g.ctx, g.desc, g.k, g.v, to_dev_bf16(b.k_new), to_dev_bf16(b.v_new), torch.from_numpy(bad).cuda(),
                    b.max_blocks, b.context_len, b.query_len)
    torch.cuda.synchronize()
    assert cf.cf_get_async_status(g.ctx) == cf.CF_ERR_OUT_OF_RANGE
    assert np.array_equal(to_host_bits(g.k), k_before) and np.array_equal(to_host_bits(g.v), v_before)
    o_bits, lse = g.attend(b)                                  # the context is still good
    ref_o, ref_lse = oracle.mixed_attention(b.q, k_before, v_before, b.block_table, b.context_len, b.query_len)
    compare(o_bits, lse, ref_o, ref_lse)
    g.close()


def test_destroy_is_refused_while_a_plan_is_alive():
    sc = small(53, 8, 2, 64, [100], [[1]], NB=64)
    b = sc.batches[0]
    ctx = cf.cf_create(0)
    d = cf.make_desc(8, 2, 64, 16, 64)
    plan = cf.cf_plan_create(ctx, d, b.context_len, b.query_len, b.max_blocks)
    assert cf.load_library().cf_destroy(ctx) == cf.CF_ERR_BUSY
    cf.cf_plan_destroy(plan)
    cf.cf_destroy(ctx)


def test_set_overlap_one_returns_to_the_default_share():
    """cf_set_overlap(ctx, n > 1) then cf_set_overlap(ctx, 1): the default share again, i.e. the bits of a fresh
    context on a batch whose plan depends on the share (KV split balanced over the front grid)."""
    sc = small(55, 32, 8, 128, [4000, 3000, 800], [[300, 1, 1]], NB=2048)
    b = sc.batches[0]
    fresh = GpuScenario(sc)
    fresh.append(b)
    o0, l0 = fresh.attend(b)
    g = GpuScenario(sc)
    g.append(b)
    cf.cf_set_overlap(g.ctx, 9)
    g.attend(b)
    cf.cf_set_overlap(g.ctx, 1)
    o1, l1 = g.attend(b)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)
    fresh.close()
    g.close()
