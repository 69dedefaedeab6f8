"""Pins for the CPU oracle: it is checked against things other than itself.

The paper prints no worked attention value (it adds no kernels, Section 5), so the pins are:
  * brute force: gather K/V into contiguous arrays, build the dense [Lq, Lc] mask, evaluate
    softmax(QK^T * scale + mask) V with numpy matrices;
  * a library routine: torch scaled_dot_product_attention in fp64 (with its own GQA head mapping);
  * closed forms: Lc = 1, q = 0, constant V, V = 1, a dominant key;
  * invariants: page permutation, chunking, decode == 1-token prefill, GQA == MHA with duplicated
    KV heads, causal-mask / slack-slot / unassigned-page insensitivity, batch-order permutation.
"""
import math

import numpy as np
import pytest
import torch

import cf_synth as syn
import oracle


# ------------------------------------------------------------------ independent brute force
def gather_contiguous(pool, block_row, n_tokens):
    """[NB, Hkv, B, D] pool -> [Hkv, n_tokens, D] fp64 for one sequence."""
    NB, H, B, D = pool.shape
    nb = (n_tokens + B - 1) // B
    pages = pool[block_row[:nb]]                                  # [nb, H, B, D]
    flat = pages.transpose(1, 0, 2, 3).reshape(H, nb * B, D)[:, :n_tokens]
    return syn.bf16_bits_to_f64(flat)


def brute_force(batch, k_pool, v_pool, scale=None):
    g = batch.geom
    G = g.num_q_heads // g.num_kv_heads
    scale = 1.0 / math.sqrt(g.head_dim) if scale is None else scale
    qs = batch.q_start()
    out = np.zeros((batch.total_q, g.num_q_heads, g.head_dim))
    lse = np.zeros((batch.total_q, g.num_q_heads))
    for s in range(batch.num_seqs):
        Lq, Lc = int(batch.query_len[s]), int(batch.context_len[s])
        if Lq == 0:
            continue
        K = gather_contiguous(k_pool, batch.block_table[s], Lc)
        V = gather_contiguous(v_pool, batch.block_table[s], Lc)
        Q = syn.bf16_bits_to_f64(batch.q[qs[s]:qs[s + 1]])          # [Lq, Hq, D]
        mask = np.arange(Lc)[None, :] > (Lc - Lq + np.arange(Lq))[:, None]
        for h in range(g.num_q_heads):
            scores = Q[:, h, :] @ K[h // G].T * scale
            scores[mask] = -np.inf
            mx = scores.max(axis=1, keepdims=True)
            e = np.exp(scores - mx)
            out[qs[s]:qs[s + 1], h] = (e / e.sum(axis=1, keepdims=True)) @ V[h // G]
            lse[qs[s]:qs[s + 1], h] = mx[:, 0] + np.log(e.sum(axis=1))
    return out, lse


def run_oracle(batch, k_pool, v_pool, append=True, **kw):
    k, v = k_pool.copy(), v_pool.copy()
    if append:
        oracle.kv_append(k, v, batch.k_new, batch.v_new, batch.block_table, batch.context_len, batch.query_len)
    return oracle.mixed_attention(batch.q, k, v, batch.block_table, batch.context_len, batch.query_len, **kw), (k, v)


def small_scenario(seed, Hq, Hkv, D, prefix, qlens, NB=64, B=16, shuffle=False):
    geom = syn.Geometry(Hq, Hkv, D, B, NB)
    return syn.scenario_from_lengths("t", geom, seed, prefix, qlens, shuffle_seqs=shuffle)


# ------------------------------------------------------------------ T1 brute force
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 64), (4, 4, 32), (8, 1, 128), (6, 3, 16), (2, 2, 128)])
def test_oracle_matches_brute_force(Hq, Hkv, D):
    sc = small_scenario(11 + Hq, Hq, Hkv, D, prefix=[0, 5, 37, 16, 99, 0, 31], qlens=[[1, 1, 23, 16, 1, 40, 1]])
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    bo, blse = brute_force(b, k, v)
    assert np.abs(o - bo).max() < 1e-12
    assert np.abs(lse - blse).max() < 1e-12


def test_oracle_matches_brute_force_config1():
    sc = syn.config1_tiny()
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    bo, blse = brute_force(b, k, v)
    assert np.abs(o - bo).max() < 1e-12
    assert np.abs(lse - blse).max() < 1e-12
    assert np.isfinite(o).all()


def test_oracle_custom_scale_matches_brute_force():
    sc = small_scenario(5, 4, 2, 32, prefix=[10, 3], qlens=[[7, 1]])
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool, scale=0.37)
    bo, blse = brute_force(b, k, v, scale=0.37)
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - blse).max() < 1e-12


# ------------------------------------------------------------------ T2 library special case
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4), (8, 1)])
def test_oracle_matches_torch_sdpa_identity_table(Hq, Hkv):
    D, B, Lq, P = 64, 16, 37, 59
    Lc = P + Lq
    nb = (Lc + B - 1) // B
    geom = syn.Geometry(Hq, Hkv, D, B, nb)
    rng = np.random.default_rng(77)
    k_pool, v_pool = syn.empty_pools(geom)
    ident = np.arange(nb, dtype=np.int32)
    syn.fill_prefix(rng, geom, k_pool, ident, Lc)
    syn.fill_prefix(rng, geom, v_pool, ident, Lc)
    q = syn.normal_bf16(rng, (Lq, Hq, D))
    o, lse = oracle.mixed_attention(q, k_pool, v_pool, ident[None, :], [Lc], [Lq])

    K = torch.from_numpy(gather_contiguous(k_pool, ident, Lc))[None]     # [1, Hkv, Lc, D]
    V = torch.from_numpy(gather_contiguous(v_pool, ident, Lc))[None]
    Q = torch.from_numpy(syn.bf16_bits_to_f64(q)).permute(1, 0, 2)[None]  # [1, Hq, Lq, D]
    allow = torch.ones(Lq, Lc, dtype=torch.bool).tril(diagonal=P)
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=allow, enable_gqa=True)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(o - ref).max() < 1e-12


# ------------------------------------------------------------------ T3 closed forms
def _single_seq(Hq, Hkv, D, Lc, Lq, seed=3, NB=40, B=16):
    sc = small_scenario(seed, Hq, Hkv, D, prefix=[Lc - Lq], qlens=[[Lq]], NB=NB, B=B)
    b = sc.batches[0]
    k, v = sc.k_pool.copy(), sc.v_pool.copy()
    oracle.kv_append(k, v, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
    return b, k, v


def test_context_length_one_returns_v0():
    b, k, v = _single_seq(8, 2, 64, 1, 1)
    o, lse = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len)
    v0 = syn.bf16_bits_to_f64(v[b.block_table[0, 0], :, 0, :])            # [Hkv, D]
    for h in range(8):
        assert np.array_equal(o[0, h], v0[h // 4])
    # lse = the single score itself
    qf = syn.bf16_bits_to_f64(b.q)[0]
    k0 = syn.bf16_bits_to_f64(k[b.block_table[0, 0], :, 0, :])
    for h in range(8):
        assert abs(lse[0, h] - (qf[h] @ k0[h // 4]) / 8.0) < 1e-13


def test_zero_query_gives_mean_of_visible_values():
    b, k, v = _single_seq(4, 2, 32, 45, 13)
    q0 = np.zeros_like(b.q)
    o, lse = oracle.mixed_attention(q0, k, v, b.block_table, b.context_len, b.query_len)
    V = gather_contiguous(v, b.block_table[0], 45)
    for i in range(13):
        p = 45 - 13 + i
        for h in range(4):
            assert np.abs(o[i, h] - V[h // 2, :p + 1].mean(axis=0)).max() < 1e-13
            assert abs(lse[i, h] - math.log(p + 1)) < 1e-13


def test_equal_keys_give_mean_and_constant_v_is_returned():
    b, k, v = _single_seq(4, 1, 32, 33, 5)
    k2 = k.copy()
    k2[...] = k[b.block_table[0, 0], 0, 0][None, None, None, :]             # every key identical
    o, _ = oracle.mixed_attention(b.q, k2, v, b.block_table, b.context_len, b.query_len)
    V = gather_contiguous(v, b.block_table[0], 33)
    for i in range(5):
        assert np.abs(o[i, 2] - V[0, :33 - 5 + i + 1].mean(axis=0)).max() < 1e-13
    v2 = v.copy()
    v2[...] = syn.f32_to_bf16_bits(np.float32(1.0))
    o, _ = oracle.mixed_attention(b.q, k, v2, b.block_table, b.context_len, b.query_len)
    assert np.abs(o - 1.0).max() < 1e-14


def test_weights_rows_sum_to_one_and_respect_mask():
    b, k, v = _single_seq(4, 2, 32, 50, 9)
    o, lse, w = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len, want_weights=50)
    assert np.abs(w.sum(axis=-1) - 1.0).max() < 1e-14
    for i in range(9):
        p = 50 - 9 + i
        assert (w[i, :, p + 1:] == 0).all() and (w[i, :, :p + 1] > 0).all()
    # weights reproduce O as a plain weighted sum of gathered V
    V = gather_contiguous(v, b.block_table[0], 50)
    ref = np.einsum("ihj,hjd->ihd", w.reshape(9, 2, 2, 50).reshape(9, 4, 50)[:, [0, 1], :], V)  # heads 0,1 -> kv 0
    assert np.abs(o[:, 0] - w[:, 0] @ V[0]).max() < 1e-13
    assert np.abs(o[:, 3] - w[:, 3] @ V[1]).max() < 1e-13
    del ref


@pytest.mark.parametrize("jstar", [0, 15, 16, 40, 46])
def test_dominant_key_selects_its_value(jstar):
    Lc, Lq, D = 47, 1, 64
    b, k, v = _single_seq(2, 1, D, Lc, Lq, seed=9)
    # q = 8 * e_0 ; planted key = 64 * e_0 -> score 8*64/8 = 64 ; other keys have |k_0| <~ 5 -> score <~ 5
    q = np.zeros_like(b.q)
    q[0, :, 0] = syn.f32_to_bf16_bits(np.float32(8.0))
    blk, slot = b.block_table[0, jstar // 16], jstar % 16
    k[blk, 0, slot, :] = 0
    k[blk, 0, slot, 0] = syn.f32_to_bf16_bits(np.float32(64.0))
    o, _ = oracle.mixed_attention(q, k, v, b.block_table, b.context_len, b.query_len)
    vj = syn.bf16_bits_to_f64(v[blk, 0, slot])
    assert np.abs(o[0, 0] - vj).max() < 1e-15 * 1e3


# ------------------------------------------------------------------ T4 invariants
def test_page_permutation_leaves_output_bit_identical():
    sc = small_scenario(21, 8, 2, 64, prefix=[20, 70, 0], qlens=[[1, 30, 17]])
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    perm = np.random.default_rng(0).permutation(sc.geom.num_blocks)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.size)
    k2, v2 = k[perm], v[perm]                                   # new page i holds old page perm[i]
    bt2 = np.where(b.block_table >= 0, inv[np.maximum(b.block_table, 0)], -1).astype(np.int32)
    o2, lse2 = oracle.mixed_attention(b.q, k2, v2, bt2, b.context_len, b.query_len)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)


def test_chunking_invariance():
    """A prompt cut into any bounded units gives the same rows (Section 4.4: units may be paused between)."""
    Hq, Hkv, D, P, N = 4, 2, 32, 21, 90
    one = small_scenario(31, Hq, Hkv, D, prefix=[P], qlens=[[N]], NB=16)
    b1 = one.batches[0]
    (o1, l1), (kf, vf) = run_oracle(b1, one.k_pool, one.v_pool)
    for cuts in ([30, 30, 30], [1, 50, 39], [89, 1]):
        k, v = one.k_pool.copy(), one.v_pool.copy()
        at, have = 0, P
        for c in cuts:
            have += c
            oracle.kv_append(k, v, b1.k_new[at:at + c], b1.v_new[at:at + c], b1.block_table, [have], [c])
            o, l = oracle.mixed_attention(b1.q[at:at + c], k, v, b1.block_table, [have], [c])
            assert np.array_equal(o, o1[at:at + c]) and np.array_equal(l, l1[at:at + c])
            at += c
        assert np.array_equal(k, kf) and np.array_equal(v, vf)


def test_decode_equals_one_token_prefill_and_batch_order():
    sc = small_scenario(41, 8, 4, 32, prefix=[12, 0, 33, 64], qlens=[[1, 9, 1, 16]])
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    qs = b.q_start()
    order = [2, 0, 3, 1]
    q2 = np.concatenate([b.q[qs[s]:qs[s + 1]] for s in order])
    o2, lse2 = oracle.mixed_attention(q2, k, v, b.block_table[order], b.context_len[order], b.query_len[order])
    at = 0
    for s in order:
        n = int(b.query_len[s])
        assert np.array_equal(o2[at:at + n], o[qs[s]:qs[s + 1]])
        assert np.array_equal(lse2[at:at + n], lse[qs[s]:qs[s + 1]])
        at += n
    # last row of a prefill chunk == the same token issued alone as a decode step
    s = 3
    o3, _ = oracle.mixed_attention(b.q[qs[s + 1] - 1:qs[s + 1]], k, v, b.block_table[s:s + 1], b.context_len[s:s + 1], [1])
    assert np.array_equal(o3[0], o[qs[s + 1] - 1])


def test_gqa_equals_mha_with_duplicated_kv_heads():
    sc = small_scenario(51, 8, 2, 32, prefix=[19, 40], qlens=[[1, 11]])
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    k8, v8 = np.repeat(k, 4, axis=1), np.repeat(v, 4, axis=1)
    o8, lse8 = oracle.mixed_attention(b.q, k8, v8, b.block_table, b.context_len, b.query_len)
    assert np.array_equal(o, o8) and np.array_equal(lse, lse8)


def test_invisible_positions_do_not_matter():
    """Keys after the query position, slack slots of the last page, unassigned pages and the unused
    tail of the block table may hold anything (NaN included)."""
    sc = small_scenario(61, 4, 2, 32, prefix=[10, 37], qlens=[[1, 20]], NB=32)
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    assert np.isfinite(o).all()          # pools were NaN-filled outside the visible range already
    k2, v2 = k.copy(), v.copy()
    used = set(int(x) for x in b.block_table.ravel() if x >= 0)
    for blk in range(32):
        if blk not in used:
            k2[blk] = 0x7F80             # +inf
            v2[blk] = 0xFF80
    # slack slots of the last page of seq 1 (Lc = 57 -> slots 9..15 of page 3)
    last = b.block_table[1, 3]
    k2[last, :, 9:, :] = 0x4000
    v2[last, :, 9:, :] = 0x4000
    bt2 = b.block_table.copy()
    bt2[bt2 < 0] = 123456
    o2, lse2 = oracle.mixed_attention(b.q, k2, v2, bt2, b.context_len, b.query_len)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)
    # changing keys at positions > p changes only later rows
    qs = b.q_start()
    k3 = k.copy()
    pos = 37 + 10                        # visible to chunk rows i >= 10 only
    k3[b.block_table[1, pos // 16], :, pos % 16, :] ^= 0x8000
    o3, _ = oracle.mixed_attention(b.q, k3, v, b.block_table, b.context_len, b.query_len)
    assert np.array_equal(o3[qs[1]:qs[1] + 10], o[qs[1]:qs[1] + 10])
    assert not np.array_equal(o3[qs[1] + 10:], o[qs[1] + 10:])
    assert np.array_equal(o3[:qs[1]], o[:qs[1]])


def test_row_subset_matches_full_run():
    sc = small_scenario(71, 4, 2, 32, prefix=[5, 80, 9], qlens=[[1, 50, 3]])
    b = sc.batches[0]
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    rows = np.array([0, 1, 17, 50, 51, 53], dtype=np.int64)
    o2, lse2 = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len, rows=rows)
    assert np.array_equal(o2, o[rows]) and np.array_equal(lse2, lse[rows])


# ------------------------------------------------------------------ kv_append against a numpy scatter
def test_kv_append_matches_python_scatter_and_touches_nothing_else():
    sc = small_scenario(81, 4, 2, 32, prefix=[0, 15, 16, 37, 5], qlens=[[3, 1, 40, 0, 16]], NB=32)
    b = sc.batches[0]
    k, v = sc.k_pool.copy(), sc.v_pool.copy()
    oracle.kv_append(k, v, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
    k_ref, v_ref = sc.k_pool.copy(), sc.v_pool.copy()
    row = 0
    for s in range(b.num_seqs):
        P = int(b.context_len[s] - b.query_len[s])
        for i in range(int(b.query_len[s])):
            blk, slot = b.block_table[s, (P + i) // 16], (P + i) % 16
            k_ref[blk, :, slot, :] = b.k_new[row]
            v_ref[blk, :, slot, :] = b.v_new[row]
            row += 1
    assert np.array_equal(k, k_ref) and np.array_equal(v, v_ref)


def test_oracle_rejects_bad_lengths():
    sc = small_scenario(91, 4, 2, 32, prefix=[5], qlens=[[2]])
    b = sc.batches[0]
    with pytest.raises(ValueError):
        oracle.mixed_attention(b.q, sc.k_pool, sc.v_pool, b.block_table, [1], [2])
    with pytest.raises(ValueError):
        oracle.mixed_attention(b.q, sc.k_pool, sc.v_pool, b.block_table[:, :0], [7], [2])


# ------------------------------------------------------------------ error model used for the GPU tolerance
def test_bf16_pipeline_error_is_inside_the_stated_tolerance():
    """A numpy model of the obvious GPU scheme (fp32 scores, bf16 probabilities, fp32 accumulate, bf16
    output) stays well inside max-abs 2e-2 / mean-abs 2e-3, so those bounds are attainable."""
    rng = np.random.default_rng(5)
    D = 128
    for Lc in (2, 256, 4096):
        q = syn.bf16_bits_to_f32(syn.normal_bf16(rng, (8, D)))
        K = syn.bf16_bits_to_f32(syn.normal_bf16(rng, (Lc, D)))
        V = syn.bf16_bits_to_f32(syn.normal_bf16(rng, (Lc, D)))
        s = (q @ K.T) * np.float32(1 / math.sqrt(D))
        e = np.exp(s - s.max(axis=1, keepdims=True)).astype(np.float32)
        p16 = syn.bf16_bits_to_f32(syn.f32_to_bf16_bits(e))
        o = syn.bf16_bits_to_f64(syn.f32_to_bf16_bits(((p16 @ V) / e.sum(axis=1, keepdims=True)).astype(np.float32)))
        s64 = (q.astype(np.float64) @ K.astype(np.float64).T) / math.sqrt(D)
        e64 = np.exp(s64 - s64.max(axis=1, keepdims=True))
        o64 = (e64 / e64.sum(axis=1, keepdims=True)) @ V.astype(np.float64)
        assert np.abs(o - o64).max() < 2e-2 and np.abs(o - o64).mean() < 2e-3


def test_empty_sequences_inside_the_batch_match_brute_force():
    """Sequences with no new tokens (Lq = 0), at the front, in the middle and at the end of the batch, own no
    packed rows: the rows of the sequences around them must still be found (row -> sequence lookup) and match
    the dense brute force; asking for an explicit row list gives the same rows."""
    sc = small_scenario(71, 8, 2, 64, prefix=[40, 3, 0, 77, 19, 5, 60], qlens=[[0, 1, 25, 0, 0, 17, 0]])
    b = sc.batches[0]
    assert b.total_q == 43
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    bo, blse = brute_force(b, k, v)
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - blse).max() < 1e-12
    rows = np.array([0, 1, 25, 26, 42], dtype=np.int64)          # the decode row, first/last rows of both chunks
    o2, lse2 = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len, rows=rows)
    assert np.array_equal(o2, o[rows]) and np.array_equal(lse2, lse[rows])
    # the scatter skips them too: slots of the empty sequences keep their sentinel
    kk, vv = sc.k_pool.copy(), sc.v_pool.copy()
    oracle.kv_append(kk, vv, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len)
    blk = int(b.block_table[0, 40 // 16])
    assert (kk[blk, :, 40 % 16:, :] == syn.BF16_NAN_BITS).all()


# ------------------------------------------------------------------ variant: sliding window + attention sinks
def brute_force_variant(batch, k_pool, v_pool, window=0, sinks=None, scale=None):
    """Dense statement of the variant: an explicit [Lq, Lc] boolean band mask (causal edge on the right, the
    window's edge on the left) and the sink as one extra softmax column that carries a zero value row."""
    g = batch.geom
    G = g.num_q_heads // g.num_kv_heads
    scale = 1.0 / math.sqrt(g.head_dim) if scale is None else scale
    qs = batch.q_start()
    out = np.zeros((batch.total_q, g.num_q_heads, g.head_dim))
    lse = np.zeros((batch.total_q, g.num_q_heads))
    for s in range(batch.num_seqs):
        Lq, Lc = int(batch.query_len[s]), int(batch.context_len[s])
        if Lq == 0:
            continue
        K = gather_contiguous(k_pool, batch.block_table[s], Lc)
        V = gather_contiguous(v_pool, batch.block_table[s], Lc)
        Q = syn.bf16_bits_to_f64(batch.q[qs[s]:qs[s + 1]])
        pos = (Lc - Lq + np.arange(Lq))[:, None]
        keys = np.arange(Lc)[None, :]
        hidden = keys > pos
        if window > 0:
            hidden |= keys <= pos - window
        for h in range(g.num_q_heads):
            scores = Q[:, h, :] @ K[h // G].T * scale
            scores[hidden] = -np.inf
            vals = V[h // G]
            if sinks is not None:
                scores = np.concatenate([scores, np.full((Lq, 1), float(sinks[h]))], axis=1)
                vals = np.concatenate([vals, np.zeros((1, g.head_dim))], axis=0)
            logsum = np.logaddexp.reduce(scores, axis=1)
            out[qs[s]:qs[s + 1], h] = np.exp(scores - logsum[:, None]) @ vals
            lse[qs[s]:qs[s + 1], h] = logsum
    return out, lse


@pytest.mark.parametrize("window,with_sinks", [(1, False), (7, False), (16, True), (33, True), (0, True), (1000, True)])
def test_variant_matches_brute_force(window, with_sinks):
    sc = small_scenario(91, 8, 2, 64, prefix=[0, 5, 37, 16, 99, 0, 31], qlens=[[1, 1, 23, 16, 1, 40, 1]])
    b = sc.batches[0]
    sinks = np.random.default_rng(4).normal(0.0, 2.0, size=8) if with_sinks else None
    (o, lse), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool, window=window, sinks=sinks)
    bo, blse = brute_force_variant(b, k, v, window=window, sinks=sinks)
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - blse).max() < 1e-12


def test_variant_matches_torch_sdpa_with_band_mask_and_sink_column():
    """Library statement: scaled_dot_product_attention over the gathered keys plus one extra zero key / zero
    value per KV head, with an additive float mask that is -inf outside the band and the head's sink logit on
    the extra column (GQA by repeating the KV heads, since the mask is per query head)."""
    Hq, Hkv, D, B, Lq, P, W = 8, 2, 64, 16, 37, 59, 20
    Lc = P + Lq
    nb = (Lc + B - 1) // B
    geom = syn.Geometry(Hq, Hkv, D, B, nb)
    rng = np.random.default_rng(78)
    k_pool, v_pool = syn.empty_pools(geom)
    ident = np.arange(nb, dtype=np.int32)
    syn.fill_prefix(rng, geom, k_pool, ident, Lc)
    syn.fill_prefix(rng, geom, v_pool, ident, Lc)
    q = syn.normal_bf16(rng, (Lq, Hq, D))
    sinks = rng.normal(0.0, 1.5, size=Hq)
    o, lse = oracle.mixed_attention(q, k_pool, v_pool, ident[None, :], [Lc], [Lq], window=W, sinks=sinks)

    G = Hq // Hkv
    K = torch.from_numpy(gather_contiguous(k_pool, ident, Lc)).repeat_interleave(G, dim=0)      # [Hq, Lc, D]
    V = torch.from_numpy(gather_contiguous(v_pool, ident, Lc)).repeat_interleave(G, dim=0)
    K = torch.cat([K, torch.zeros(Hq, 1, D, dtype=torch.float64)], dim=1)[None]
    V = torch.cat([V, torch.zeros(Hq, 1, D, dtype=torch.float64)], dim=1)[None]
    Q = torch.from_numpy(syn.bf16_bits_to_f64(q)).permute(1, 0, 2)[None]
    pos = P + torch.arange(Lq)[:, None]
    keys = torch.arange(Lc)[None, :]
    band = (keys <= pos) & (keys > pos - W)
    bias = torch.full((Hq, Lq, Lc + 1), float("-inf"), dtype=torch.float64)
    bias[:, :, :Lc][band[None].expand(Hq, -1, -1)] = 0.0
    bias[:, :, Lc] = torch.from_numpy(sinks)[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=bias[None])
    assert np.abs(o - ref[0].permute(1, 0, 2).numpy()).max() < 1e-12


def test_variant_reduces_to_the_plain_definition():
    """A window at least as long as the context, and sinks of -inf, give the bits of the plain path."""
    sc = small_scenario(93, 8, 2, 64, prefix=[10, 77, 0], qlens=[[1, 30, 19]])
    b = sc.batches[0]
    (o0, l0), (k, v) = run_oracle(b, sc.k_pool, sc.v_pool)
    for W in (int(b.context_len.max()), 10 ** 6):
        o1, l1 = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len, window=W)
        assert np.array_equal(o0, o1) and np.array_equal(l0, l1)
    o2, l2 = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len, sinks=np.full(8, -np.inf))
    assert np.array_equal(o0, o2) and np.array_equal(l0, l2)


def test_variant_closed_forms_with_zero_query():
    """q = 0: every visible key weighs the same.  Window W -> the mean of the last min(W, p + 1) values and
    lse = ln min(W, p + 1); with a sink s the n visible keys weigh 1 / (n + e^s) each and lse = ln(n + e^s)."""
    b, k, v = _single_seq(4, 2, 32, 45, 13)
    q0 = np.zeros_like(b.q)
    V = gather_contiguous(v, b.block_table[0], 45)
    W = 10
    o, lse = oracle.mixed_attention(q0, k, v, b.block_table, b.context_len, b.query_len, window=W)
    sinks = np.array([0.0, 1.0, -2.0, 3.5])
    os_, lses = oracle.mixed_attention(q0, k, v, b.block_table, b.context_len, b.query_len, window=W, sinks=sinks)
    for i in range(13):
        p = 45 - 13 + i
        n = min(W, p + 1)
        for h in range(4):
            mean = V[h // 2, p + 1 - n:p + 1].mean(axis=0)
            assert np.abs(o[i, h] - mean).max() < 1e-13 and abs(lse[i, h] - math.log(n)) < 1e-13
            assert np.abs(os_[i, h] - mean * n / (n + math.exp(sinks[h]))).max() < 1e-13
            assert abs(lses[i, h] - math.log(n + math.exp(sinks[h]))) < 1e-13


def test_variant_weights_vanish_left_of_the_window():
    b, k, v = _single_seq(4, 2, 32, 50, 9)
    sinks = np.array([0.5, -1.0, 2.0, 0.0])
    o, lse, w = oracle.mixed_attention(b.q, k, v, b.block_table, b.context_len, b.query_len, want_weights=50, window=12,
                                       sinks=sinks)
    for i in range(9):
        p = 50 - 9 + i
        assert (w[i, :, :p - 11] == 0).all() and (w[i, :, p + 1:] == 0).all() and (w[i, :, p - 11:p + 1] > 0).all()
    # the key weights plus the sink's share exp(s - lse) sum to one
    assert np.abs(w.sum(axis=-1) + np.exp(sinks[None, :] - lse) - 1.0).max() < 1e-14
    # keys left of the window may hold anything (here: Inf) without reaching the result
    k2, v2 = k.copy(), v.copy()
    first_page = b.block_table[0, 0]
    k2[first_page] = 0x7F80
    v2[first_page] = 0x7F80
    o2, lse2 = oracle.mixed_attention(b.q, k2, v2, b.block_table, b.context_len, b.query_len, window=12, sinks=sinks)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)


# ------------------------------------------------------------------ variant: fp8 (e4m3) KV cache
def test_e4m3_decode_matches_the_library_type_for_every_code():
    codes = np.arange(256, dtype=np.uint8)
    mine = oracle.e4m3_decode(codes)
    lib = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    nan = np.isnan(lib)
    assert list(np.nonzero(nan)[0]) == [0x7F, 0xFF] and np.isnan(mine[nan]).all()
    assert np.array_equal(mine[~nan], lib[~nan])
    assert mine[0x7E] == 448.0 and mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6       # the format's corner values


def test_e4m3_encode_rounds_to_nearest_even_and_saturates():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 100, 20000), rng.uniform(-0.02, 0.02, 20000),
                        # every representable value and every midpoint between neighbours (the ties)
                        oracle.e4m3_decode(np.arange(0x7F, dtype=np.uint8)),
                        (oracle.e4m3_decode(np.arange(0x7E, dtype=np.uint8)) + oracle.e4m3_decode(np.arange(1, 0x7F, dtype=np.uint8))) / 2,
                        [0.0, -0.0, 447.9, 448.0, 463.9]]).astype(np.float32)
    x = np.concatenate([x, -x])
    mine = oracle.e4m3_encode(x)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()        # the library's cast: nearest even inside the range
    assert np.array_equal(mine, lib)
    # nearest: no other code is closer (brute force over the whole grid)
    grid = oracle.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    sample = np.abs(x[:2000]).astype(np.float64)
    best = np.abs(sample[:, None] - grid[None, :]).min(axis=1)
    assert np.allclose(np.abs(oracle.e4m3_decode(mine[:2000] & 0x7F) - sample), best, rtol=0, atol=0)
    # beyond the largest finite value the library's cast gives NaN; this one saturates
    big = np.array([464.0, 500.0, 1e9, -480.0, np.inf, -np.inf], dtype=np.float32)
    assert list(oracle.e4m3_encode(big)) == [0x7E, 0x7E, 0x7E, 0xFE, 0x7E, 0xFE]
    assert oracle.e4m3_encode(np.array([np.nan], dtype=np.float32))[0] == 0x7F


def _fp8_case(seed=21):
    sc = small_scenario(seed, 8, 2, 64, prefix=[40, 3, 0, 77], qlens=[[1, 25, 17, 1]])
    b = sc.batches[0]
    k8 = np.zeros(sc.k_pool.shape, dtype=np.uint8)
    v8 = np.zeros(sc.v_pool.shape, dtype=np.uint8)
    return sc, b, k8, v8


def test_fp8_append_matches_a_python_loop():
    sc, b, k8, v8 = _fp8_case()
    k_scale, v_scale = np.array([0.5, 0.013], dtype=np.float32), np.array([2.0, 0.3], dtype=np.float32)
    k8[...] = 0xAA
    v8[...] = 0x55
    oracle.kv_append(k8, v8, b.k_new, b.v_new, b.block_table, b.context_len, b.query_len, k_scale, v_scale)
    want_k, want_v = np.full_like(k8, 0xAA), np.full_like(v8, 0x55)
    kn, vn = syn.bf16_bits_to_f32(b.k_new), syn.bf16_bits_to_f32(b.v_new)
    row = 0
    for s in range(b.num_seqs):
        P = int(b.context_len[s] - b.query_len[s])
        for i in range(int(b.query_len[s])):
            blk, slot = b.block_table[s, (P + i) // 16], (P + i) % 16
            for g in range(2):
                want_k[blk, g, slot] = oracle.e4m3_encode((kn[row, g] / k_scale[g]).astype(np.float32))
                want_v[blk, g, slot] = oracle.e4m3_encode((vn[row, g] / v_scale[g]).astype(np.float32))
            row += 1
    assert np.array_equal(k8, want_k) and np.array_equal(v8, want_v)


def test_fp8_cache_reduces_to_the_bf16_path_when_the_values_fit():
    """With power-of-two scales every dequantised value e4m3(code) * scale is exactly a bf16 number: the fp8 read
    path must give the bits of the (already pinned) bf16 path on a pool that holds those values."""
    sc, b, k8, v8 = _fp8_case()
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 256, size=k8.shape, dtype=np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x10                       # no NaN codes
    k8[...] = codes
    v8[...] = rng.permutation(codes.reshape(-1)).reshape(codes.shape)
    k_scale, v_scale = np.array([0.25, 4.0]), np.array([1.0, 0.125])
    o8, lse8 = oracle.mixed_attention(b.q, k8, v8, b.block_table, b.context_len, b.query_len, k_scale=k_scale, v_scale=v_scale,
                                      window=20, sinks=np.linspace(-1, 1, 8))
    kb = syn.f32_to_bf16_bits((oracle.e4m3_decode(k8) * k_scale[None, :, None, None]).astype(np.float32))
    vb = syn.f32_to_bf16_bits((oracle.e4m3_decode(v8) * v_scale[None, :, None, None]).astype(np.float32))
    assert np.array_equal(syn.bf16_bits_to_f64(kb), oracle.e4m3_decode(k8) * k_scale[None, :, None, None])   # exact in bf16
    ob, lseb = oracle.mixed_attention(b.q, kb, vb, b.block_table, b.context_len, b.query_len, window=20, sinks=np.linspace(-1, 1, 8))
    assert np.array_equal(o8, ob) and np.array_equal(lse8, lseb)


def test_fp8_scales_are_per_kv_head():
    """Doubling one KV head's k_scale is the same as doubling the softmax scale for its query heads only; doubling
    v_scale doubles those heads' outputs."""
    sc, b, k8, v8 = _fp8_case()
    rng = np.random.default_rng(9)
    k8[...] = rng.integers(0x20, 0x50, size=k8.shape, dtype=np.uint8)
    v8[...] = rng.integers(0x20, 0x50, size=v8.shape, dtype=np.uint8)
    base = dict(k_scale=np.array([1.0, 1.0]), v_scale=np.array([1.0, 1.0]))
    o0, _ = oracle.mixed_attention(b.q, k8, v8, b.block_table, b.context_len, b.query_len, **base)
    o1, _ = oracle.mixed_attention(b.q, k8, v8, b.block_table, b.context_len, b.query_len, k_scale=np.array([1.0, 1.0]),
                                   v_scale=np.array([1.0, 2.0]))
    assert np.array_equal(o1[:, :4], o0[:, :4]) and np.array_equal(o1[:, 4:], 2.0 * o0[:, 4:])
    o2, _ = oracle.mixed_attention(b.q, k8, v8, b.block_table, b.context_len, b.query_len, k_scale=np.array([2.0, 1.0]),
                                   v_scale=np.array([1.0, 1.0]))
    o3, _ = oracle.mixed_attention(b.q, k8, v8, b.block_table, b.context_len, b.query_len, scale=2.0 / 8.0, **base)
    assert np.array_equal(o2[:, 4:], o0[:, 4:]) and np.abs(o2[:, :4] - o3[:, :4]).max() < 1e-13
