"""The seeded input generators: shapes, length distributions and stored length draws."""
import os

import numpy as np

import cf_synth as syn

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_length_draws_match_stored_files():
    for name, fn in (("cfg2", syn.config2_lengths), ("cfg3", syn.config3_lengths),
                     ("cfg4", syn.config4_lengths), ("cfg5", syn.config5_lengths)):
        want = np.loadtxt(os.path.join(GOLD, f"lengths_{name}.txt"), dtype=np.int64)
        assert np.array_equal(fn(0), want), name


def test_length_ranges():
    for k in range(3):
        a = syn.config2_lengths(k); assert a.shape == (64,) and a.min() >= 1024 and a.max() <= 8192
        a = syn.config3_lengths(k); assert a.shape == (48,) and a.min() >= 128 and a.max() <= 16384
        a = syn.config4_lengths(k); assert a.shape == (16,) and a.min() >= 8192 and a.max() <= 32768
        a = syn.config5_lengths(k); assert a.shape == (256,) and a.min() >= 64 and a.max() <= 32768
    # "mean 2048, sigma 1": the unclipped lognormal mean is exp(mu + 1/2) = 2048
    big = syn.lognormal_clipped(np.random.default_rng(1), 400000, np.log(2048.0) - 0.5, 1.0, 0, 10**9)
    assert abs(big.mean() / 2048.0 - 1.0) < 0.02
    med = syn.lognormal_clipped(np.random.default_rng(2), 400000, np.log(4096.0), 0.8, 0, 10**9)
    assert abs(np.median(med) / 4096.0 - 1.0) < 0.02


def test_config1_layout():
    sc = syn.config1_tiny()
    b = sc.batches[0]
    assert list(b.query_len) == [128, 1, 1, 1, 1] and list(b.context_len) == [256] * 5
    assert b.q.shape == (132, 8, 64) and b.k_new.shape == (132, 2, 64)
    assert sc.k_pool.shape == (256, 2, 16, 64)
    used = b.block_table[b.block_table >= 0]
    assert used.size == np.unique(used).size == 5 * 16          # disjoint pages
    # prefix slots are finite, new-token slots and unused pages are NaN before the append
    kf = syn.bf16_bits_to_f32(sc.k_pool)
    assert np.isfinite(kf[b.block_table[0, :8]]).all() and np.isnan(kf[b.block_table[0, 8:16]]).all()
    assert np.isnan(kf[b.block_table[1, 15], :, 15]).all() and np.isfinite(kf[b.block_table[1, 15], :, :15]).all()


def test_bf16_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38], dtype=np.float32)   # ties: 1+2^-8 -> 1, 1+3*2^-8 -> 1+2^-6
    bits = syn.f32_to_bf16_bits(x)
    back = syn.bf16_bits_to_f32(bits)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.015625 and back[3] == -2.5
    assert syn.f32_to_bf16_bits(np.float32(64.0)).shape == ()


def test_config5_points_and_split():
    assert len(syn.CONFIG5_POINTS) == 13
    q = syn.config5_sweep_point  # only lengths are checked here (pools are large): reuse its arithmetic
    base, rem = divmod(2048, 3)
    assert [base + (1 if i < rem else 0) for i in range(3)] == [683, 683, 682]
    del q


def test_sample_rows_keeps_decode_rows_and_tile_edges():
    sc = syn.scenario_from_lengths("t", syn.Geometry(4, 2, 32, 16, 128), 1, [0, 9], [[600, 1]])
    rows = syn.sample_rows(sc.batches[0], max_prefill_rows_per_seq=64)
    assert 600 in rows and 0 in rows and 599 in rows and rows.size <= 65
