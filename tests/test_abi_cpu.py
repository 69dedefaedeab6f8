"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, rejects bad
arguments on the host before touching a device, and its planner covers every token exactly once."""
import ctypes
import os
import re

import numpy as np
import pytest

import cf_synth as syn
import paper_2609_27085_b200 as cf
from paper_2609_27085_b200 import build as cf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    cf_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "crossflow_attn.h")).read()
    declared = set(re.findall(r"\b(cf_[a-z_]+)\s*\(", header))
    assert declared == set(cf.EXPORTS)
    lib = cf.load_library()
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings():
    assert cf.cf_status_string(cf.CF_OK) == "CF_OK"
    assert cf.cf_status_string(cf.CF_ERR_TIMEOUT) == "CF_ERR_TIMEOUT"
    assert cf.cf_status_string(99) == "CF_ERR_UNKNOWN"


def _plan(desc, lc, lq, max_blocks=4096, sms=148, check=True):
    return cf.cf_plan_inspect(desc, lc, lq, max_blocks, sms, check=check)


def test_desc_validation():
    ok = cf.make_desc(32, 8, 128, 16, 1024)
    assert _plan(ok, [5], [1])[0] == cf.CF_OK
    for bad, want in [
        (cf.make_desc(32, 8, 96, 16, 1024), cf.CF_ERR_UNSUPPORTED),      # head_dim
        (cf.make_desc(32, 8, 128, 32, 1024), cf.CF_ERR_UNSUPPORTED),     # block_size
        (cf.make_desc(48, 8, 128, 16, 1024), cf.CF_ERR_UNSUPPORTED),     # group 6
        (cf.make_desc(30, 8, 128, 16, 1024), cf.CF_ERR_INVALID_ARG),     # Hq % Hkv
        (cf.make_desc(32, 8, 128, 16, 1024, k_strides=(16388, 2048, 128)), cf.CF_ERR_UNSUPPORTED),  # 16-byte rule
        (cf.make_desc(32, 8, 128, 16, 1024, v_strides=(16384, 2048, 64)), cf.CF_ERR_INVALID_ARG),
        (cf.make_desc(32, 8, 128, 16, 1024, softmax_scale=-1.0), cf.CF_ERR_INVALID_ARG),
    ]:
        assert _plan(bad, [5], [1], check=False)[0] == want


def test_length_validation():
    d = cf.make_desc(8, 2, 64, 16, 64)
    assert _plan(d, [5], [6], check=False)[0] == cf.CF_ERR_INVALID_ARG        # Lq > Lc
    assert _plan(d, [5], [-1], check=False)[0] == cf.CF_ERR_INVALID_ARG
    assert _plan(d, [65], [1], max_blocks=4, check=False)[0] == cf.CF_ERR_OUT_OF_RANGE
    assert _plan(d, [64], [1], max_blocks=4, check=False)[0] == cf.CF_OK
    st, dec, comb, pre, parts = _plan(d, [0, 7], [0, 0])                      # nothing to do
    assert st == cf.CF_OK and len(dec) == len(comb) == len(pre) == 0 and parts == 0


def _check_plan(geom, lc, lq, sms=148):
    d = cf.make_desc(geom.num_q_heads, geom.num_kv_heads, geom.head_dim, geom.block_size, geom.num_blocks)
    lc, lq = np.asarray(lc, dtype=np.int32), np.asarray(lq, dtype=np.int32)
    st, dec, comb, pre, parts = _plan(d, lc, lq, max_blocks=1 << 20, sms=sms)
    qs = np.concatenate([[0], np.cumsum(lq)])
    # decode: chunks of each Lq == 1 sequence tile [0, Lc) exactly, in page multiples, none empty
    slots_seen = set()
    for s in np.nonzero(lq == 1)[0]:
        mine = dec[dec[:, 0] == s]
        mine = mine[np.argsort(mine[:, 5])]
        assert len(mine) >= 1 and mine[0, 2] == 0 and mine[-1, 3] == lc[s]
        assert (mine[:, 1] == qs[s]).all()
        assert (mine[1:, 2] == mine[:-1, 3]).all() and (mine[:, 2] % 16 == 0).all() and (mine[:, 3] > mine[:, 2]).all()
        assert list(mine[:, 5]) == list(range(len(mine)))
        if len(mine) == 1:
            assert mine[0, 4] == -1
        else:
            c = comb[comb[:, 0] == qs[s]]
            assert len(c) == 1 and c[0, 2] == len(mine)
            assert list(mine[:, 4]) == list(range(c[0, 1], c[0, 1] + len(mine)))
            slots_seen.update(int(x) for x in mine[:, 4])
    assert set(int(s) for s in dec[:, 0]) == set(int(s) for s in np.nonzero(lq == 1)[0])
    assert slots_seen == set(range(parts))
    lens = dec[:, 3] - dec[:, 2]
    assert (np.diff(lens) <= 0).all()                                      # longest first
    # prefill: every (row, query head) of each Lq > 1 sequence is covered exactly once, by an entry whose
    # kv head serves that query head
    G = geom.num_q_heads // geom.num_kv_heads
    for s in np.nonzero(lq > 1)[0]:
        mine = pre[pre[:, 0] == s]
        cover = np.zeros((lq[s], geom.num_q_heads), dtype=np.int32)
        tiles_seen = {}
        for _, q_row0, row0, n_rows, head, kvh, j0, j1 in mine:
            assert q_row0 == qs[s] + row0 and n_rows >= 1 and kvh == head // G and 0 <= j0 < j1
            tiles_seen.setdefault((row0, n_rows, head), []).append((j0, j1))
            if j0 == 0:
                cover[row0:row0 + n_rows, head] += 1
        assert (cover == 1).all()
        for (row0, n_rows, head), ranges in tiles_seen.items():
            # the KV ranges of a q tile tile [0, its number of visible KV tiles) without gap or overlap
            ranges.sort()
            assert ranges[0][0] == 0 and ranges[-1][1] == ((lc[s] - lq[s]) + row0 + n_rows + 127) // 128
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    assert set(int(s) for s in pre[:, 0]) == set(int(s) for s in np.nonzero(lq > 1)[0])
    ext = (lc - lq)[pre[:, 0]] + pre[:, 2] + pre[:, 3]
    if len(ext):
        assert ext[0] == ext.max()                                         # longest KV extent first
    return dec, comb, pre, parts


def test_plan_covers_the_five_configs():
    g4, g8 = syn.GEOM_G4, syn.GEOM_G8
    _check_plan(syn.GEOM_TINY, [256] * 5, [128, 1, 1, 1, 1])
    dec, *_ = _check_plan(g4, syn.config2_lengths(), [1] * 64)
    assert 148 * 2 <= len(dec) * 8 <= 148 * 2 * 8          # a few waves of CTAs, not thousands
    _check_plan(g4, [6144 + 512, 6144 + 512] + list(syn.config3_lengths()), [512, 512] + [1] * 48)
    dec, *_ = _check_plan(g4, [24576 + 2048] + list(syn.config4_lengths()), [2048] + [1] * 16)
    assert len(dec) * 8 >= 148 * 2                          # 16 x 8 pairs alone would leave SMs idle
    _check_plan(g8, [4096 + 8192] + list(syn.config5_lengths()), [8192] + [1] * 256)


def test_plan_random_batches():
    rng = np.random.default_rng(0)
    for _ in range(50):
        S = int(rng.integers(1, 40))
        lq = rng.choice([0, 1, 1, 1, 2, 17, 64, 65, 300], size=S)
        lc = lq + rng.integers(0, 5000, size=S)
        _check_plan(syn.GEOM_G4, lc, lq, sms=int(rng.choice([1, 4, 148])))
        _check_plan(syn.Geometry(4, 4, 128, 16, 1 << 16), lc, lq)          # group size 1: row-tile pairs
        _check_plan(syn.Geometry(8, 2, 64, 16, 1 << 16), lc, lq)           # head_dim 64


def test_calls_without_a_device_fail_with_a_status():
    """On a machine with no GPU the entry points report an error code; nothing falls back to the CPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    ctx = ctypes.c_void_p()
    st = cf.load_library().cf_create(ctypes.byref(ctx), 0, 0)
    assert st in (cf.CF_ERR_CUDA, cf.CF_ERR_INVALID_ARG) and not ctx.value
    with pytest.raises(cf.CfError):
        cf.cf_create(0)


def test_cost_model_is_sane_on_the_host():
    d = cf.make_desc(32, 8, 128, 16, 65536)
    dec, comb, pre = cf.cf_estimate_us(d, [4096] * 64, [1] * 64, 4096)
    assert pre == 0 and dec > 0
    dec2, _, _ = cf.cf_estimate_us(d, [8192] * 64, [1] * 64, 4096)
    assert dec2 > dec * 1.5                                       # decode time follows the K/V bytes
    _, _, p1 = cf.cf_estimate_us(d, [6144 + 512], [512], 4096)
    _, _, p2 = cf.cf_estimate_us(d, [24576 + 2048], [2048], 4096)
    assert 0 < p1 < p2
    _, _, p3 = cf.cf_estimate_us(d, [24576 + 2048], [2048], 4096, num_sms=74)
    assert p3 > 1.5 * p2                                          # half the SMs, about twice the waves
    assert cf.cf_estimate_us(d, [7], [0], 4096) == (0.0, 0.0, 0.0)


def test_spatial_share_follows_what_decode_needs():
    """The first prefill grid's share of the SMs: none without a mixed batch; 3/5 of the machine when decode needs
    most of the call's time; more, up to 7/8, as the prefill grows against a fixed decode batch; less for a group
    size of 8 (decode needs more SMs to saturate HBM) than for 4 on the same lengths."""
    g4, g8 = cf.make_desc(32, 8, 128, 16, 65536), cf.make_desc(64, 8, 128, 16, 65536)
    dec = [4096] * 48
    assert cf.cf_spatial_share(g4, dec, [1] * 48) == 0
    assert cf.cf_spatial_share(g4, [6656], [512]) == 0
    assert cf.cf_spatial_share(g4, [], []) == 0
    chat = cf.cf_spatial_share(g4, [6656, 6656] + dec, [512, 512] + [1] * 48)
    assert chat == 148 * 3 // 5
    shares = [cf.cf_spatial_share(g4, [p + 2048] + [20000] * 16, [2048] + [1] * 16) for p in (0, 4096, 12288, 24576, 65536)]
    assert shares == sorted(shares) and shares[0] == 88 and shares[-1] == 129
    assert all(88 <= s <= 129 for s in shares)
    mid4 = cf.cf_spatial_share(g4, [8192 + 8192] + [2048] * 256, [8192] + [1] * 256)
    mid8 = cf.cf_spatial_share(g8, [8192 + 8192] + [2048] * 256, [8192] + [1] * 256)
    assert 88 <= mid8 <= mid4 <= 129
    assert cf.cf_spatial_share(g4, [26624] + [20000] * 16, [2048] + [1] * 16, num_sms=74) <= 74 * 7 // 8


def test_kv_split_of_the_last_prefill_wave():
    """256 equal items on 148 SMs leave a last wave of 108: the planner cuts those into KV ranges that
    tile each item's extent, never start inside the diagonal band, and fill the machine."""
    d = cf.make_desc(32, 8, 128, 16, 65536)
    lc, lq = [24576 + 2048], [2048]
    st, dec, comb, pre, parts, counts = cf.cf_plan_inspect(d, lc, lq, 4096, 148, want_counts=True)
    n_items = 16 * 16                                   # 16 q tiles x 16 head pairs
    assert counts[5] == n_items % 148                   # the 108 items of the last wave are split
    k = (counts[4] - (n_items - counts[5])) // counts[5]
    assert k >= 2 and counts[4] == (n_items - counts[5]) + counts[5] * k
    cover = np.zeros((2048, 32), dtype=np.int32)        # every (row, head) has exactly one range that starts at tile 0
    for _, q_row0, row0, n_rows, head, kvh, j0, j1 in pre:
        if j0 == 0:
            cover[row0:row0 + n_rows, head] += 1
    assert (cover == 1).all()
    # 128 equal items on 148 SMs: splitting would not pay for its partial traffic
    counts = cf.cf_plan_inspect(d, [6656, 6656], [512, 512], 4096, 148, want_counts=True)[5]
    assert counts[5] == 0 and counts[4] == 128
    # on pairs of SMs: 128 four-head items on 74 pairs leave a last wave of 54, cut into KV ranges; two combine
    # items (one per CTA of the pair) per split item; every (row, head) still has exactly one range from tile 0
    st, dec, comb, pre, parts, counts = cf.cf_plan_inspect(d, lc, lq, 4096, 148, want_counts=True, prefill_pairs=1)
    assert counts[5] == 2 * (128 % 74)
    k = (counts[4] - (128 - 54)) // 54
    assert k >= 2 and counts[4] == (128 - 54) + 54 * k
    cover = np.zeros((2048, 32), dtype=np.int32)
    for _, q_row0, row0, n_rows, head, kvh, j0, j1 in pre:
        assert kvh == head // 4
        if j0 == 0:
            cover[row0:row0 + n_rows, head] += 1
    assert (cover == 1).all()


def test_few_items_are_cut_into_kv_ranges():
    """A 512-token chunk over an 8K prefix on one TP4 rank (16 query heads, 2 KV heads) is only 32 tile
    pairs for 148 SMs: the planner cuts them into KV ranges until the machine is about full."""
    d = cf.make_desc(16, 2, 128, 16, 65536)
    lc, lq = np.array([8192 + 512], np.int32), np.array([512], np.int32)
    counts = cf.cf_plan_inspect(d, lc, lq, 8192, 148, want_counts=True)[5]
    assert counts[5] > 0 and 96 <= counts[4] <= 148
    counts = cf.cf_plan_inspect(d, lc, lq, 8192, 148, want_counts=True, prefill_pairs=1)[5]          # pairs: 8 four-head items for 74 pairs
    assert counts[5] > 0 and 48 <= counts[4] <= 74
    _, _, whole = cf.cf_estimate_us(d, lc, lq, 8192, num_sms=148)
    assert whole < 0.6 * (8 + 1.9 * 68)                 # well under the time of one unsplit item


def test_forced_kv_split_tiles_every_item():
    """prefill_force_split = k cuts every item that is long enough into KV ranges; the ranges of every q tile
    still tile its visible KV tiles (checked inside _check_plan for the default plan; here with the option)."""
    d = cf.make_desc(32, 8, 128, 16, 65536)
    lc, lq = [3100 + 700, 50], [700, 1]
    for k in (2, 3, 8):
        st, dec, comb, pre, parts, counts = cf.cf_plan_inspect(d, lc, lq, 4096, 148, prefill_force_split=k, want_counts=True)
        assert counts[5] > 0 and counts[4] >= counts[5]       # (pairs of SMs: two combine items per split item)
        by_tile = {}
        for _, q_row0, row0, n_rows, head, kvh, j0, j1 in pre:
            by_tile.setdefault((row0, head), []).append((j0, j1))
        for (row0, head), ranges in by_tile.items():
            ranges.sort()
            n_rows = min(128, 700 - row0)
            assert ranges[0][0] == 0 and ranges[-1][1] == (3100 + row0 + n_rows + 127) // 128
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            assert len(ranges) <= k


def test_windowed_plan_skips_what_no_query_can_see():
    """Sliding window W: decode chunks tile [page of (Lc - W), Lc) and prefill KV ranges tile the tiles from the one
    that holds the first row's left edge up to the diagonal; nothing left of that is planned."""
    rng = np.random.default_rng(3)
    for W in (1, 16, 100, 128, 1000, 4096):
        d = cf.make_desc(32, 8, 128, 16, 1 << 16, window_size=W)
        S = 12
        lq = rng.choice([1, 1, 1, 64, 300, 700], size=S)
        lc = lq + rng.integers(0, 9000, size=S)
        for split in (0, 2):
            st, dec, comb, pre, parts = cf.cf_plan_inspect(d, lc, lq, 1 << 16, 148, prefill_force_split=split)
            for s in np.nonzero(lq == 1)[0]:
                mine = dec[dec[:, 0] == s]
                mine = mine[np.argsort(mine[:, 5])]
                lo = max(0, lc[s] - W)
                assert mine[0, 2] == (lo // 16) * 16 and mine[-1, 3] == lc[s]
                assert (mine[1:, 2] == mine[:-1, 3]).all() and (mine[:, 3] > mine[:, 2]).all()
            by_tile = {}
            for s_, q_row0, row0, n_rows, head, kvh, j0, j1 in pre:
                by_tile.setdefault((s_, row0, n_rows, head), []).append((j0, j1))
            assert len(by_tile) == sum(((n + 127) // 128) * 32 for n in lq if n > 1)
            for (s_, row0, n_rows, head), ranges in by_tile.items():
                ranges.sort()
                P = lc[s_] - lq[s_]
                assert ranges[0][0] == max(0, P + row0 - W + 1) // 128
                assert ranges[-1][1] == (P + row0 + n_rows + 127) // 128
                assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    assert cf.cf_plan_inspect(cf.make_desc(32, 8, 128, 16, 64, window_size=-1), [5], [1], 8, check=False)[0] == cf.CF_ERR_INVALID_ARG


def test_shared_prefix_argument_check_needs_no_device():
    """share_group and shared_len come together or not at all (checked before anything else is touched)."""
    lib = cf.load_library()
    d = cf.make_desc(32, 8, 128, 16, 64)
    arr = np.zeros(2, dtype=np.int32)
    fake_ctx = ctypes.c_void_p(1)                      # never dereferenced: the pairing check comes first
    st = lib.cf_mixed_attention_shared(fake_ctx, ctypes.byref(d), None, None, None, None, 4, arr.ctypes.data, arr.ctypes.data,
                                       arr.ctypes.data, None, 2, None, None, None)
    assert st == cf.CF_ERR_INVALID_ARG
