"""Seeded synthetic batches for the mixed decode + chunked-prefill paged-attention path.

This module only *draws inputs*: sequence lengths, block tables, bf16 bit patterns
for Q / K / V.  It holds none of the attention arithmetic and imports neither the
CPU oracle nor the CUDA library; both are handed the arrays produced here.

A decode node under the paper's lending mechanism builds "a mixed prefill/decode
batch" from its resident decode sequences plus locally queued prefill that reuses
a resident prefix (Section 5), and issues the prefill in bounded units (Section
4.4).  The paper's traces are not public, so the batches below are synthetic
stand-ins with the shapes of its chat and agentic workloads: many one-token
decode sequences with long, uneven contexts, plus a few prefill chunks that sit
on top of an already-cached prefix.

All tensors are numpy arrays; bf16 values are carried as ``uint16`` bit patterns.

Notation (per sequence ``s``): ``Lq`` = query_len (new tokens this iteration),
``Lc`` = context_len (visible KV length *including* the new tokens),
``P = Lc - Lq`` (cached prefix).  Pools are laid out ``[NB, Hkv, B, D]``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Iterator, List, Optional, Sequence, Tuple

import numpy as np

BF16_NAN_BITS = np.uint16(0x7FC0)


# --------------------------------------------------------------------------- bf16 bit helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    shape = np.shape(x)
    u = np.ascontiguousarray(x, dtype=np.float32).reshape(-1).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16).reshape(shape)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


def normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    """~N(0,1) values rounded to bf16, as uint16 bit patterns."""
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


# --------------------------------------------------------------------------- containers
@dataclass(frozen=True)
class Geometry:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    num_blocks: int

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    def pool_shape(self) -> Tuple[int, int, int, int]:
        return (self.num_blocks, self.num_kv_heads, self.block_size, self.head_dim)

    def kv_bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2


@dataclass
class Batch:
    """One iteration's call arguments (host side)."""
    geom: Geometry
    context_len: np.ndarray          # int32 [S], includes this iteration's new tokens
    query_len: np.ndarray            # int32 [S]
    block_table: np.ndarray          # int32 [S, max_blocks], unused tail = -1
    q: np.ndarray                    # uint16 [T, Hq, D]
    k_new: np.ndarray                # uint16 [T, Hkv, D]
    v_new: np.ndarray                # uint16 [T, Hkv, D]
    label: str = ""

    @property
    def num_seqs(self) -> int:
        return int(self.context_len.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.query_len.sum())

    @property
    def max_blocks(self) -> int:
        return int(self.block_table.shape[1])

    def q_start(self) -> np.ndarray:
        out = np.zeros(self.num_seqs + 1, dtype=np.int64)
        np.cumsum(self.query_len, out=out[1:])
        return out


@dataclass
class Scenario:
    """A pool pre-filled with every sequence's cached prefix, plus the iterations to run on it.

    ``k_pool`` / ``v_pool`` hold the cache *before* iteration 0's append: visible prefix
    slots carry N(0,1) bf16 values, every other slot carries a bf16 NaN so that any read
    outside the visible range poisons the result.
    """
    name: str
    geom: Geometry
    k_pool: np.ndarray               # uint16 [NB, Hkv, B, D]
    v_pool: np.ndarray
    batches: List[Batch] = field(default_factory=list)


# --------------------------------------------------------------------------- building blocks
def deal_block_tables(rng: np.random.Generator, geom: Geometry, capacity_tokens: Sequence[int],
                      max_blocks: Optional[int] = None) -> np.ndarray:
    """Deal disjoint physical blocks to sequences from a seeded random permutation of the pool."""
    B = geom.block_size
    need = [(int(c) + B - 1) // B for c in capacity_tokens]
    total = int(sum(need))
    if total > geom.num_blocks:
        raise ValueError(f"pool of {geom.num_blocks} blocks cannot hold {total}")
    perm = rng.permutation(geom.num_blocks).astype(np.int32)
    width = max(need + [1]) if max_blocks is None else max_blocks
    table = np.full((len(need), width), -1, dtype=np.int32)
    at = 0
    for s, n in enumerate(need):
        table[s, :n] = perm[at:at + n]
        at += n
    return table


def empty_pools(geom: Geometry) -> Tuple[np.ndarray, np.ndarray]:
    k = np.full(geom.pool_shape(), BF16_NAN_BITS, dtype=np.uint16)
    v = np.full(geom.pool_shape(), BF16_NAN_BITS, dtype=np.uint16)
    return k, v


def fill_prefix(rng: np.random.Generator, geom: Geometry, pool: np.ndarray,
                block_row: np.ndarray, n_tokens: int) -> None:
    """Write n_tokens N(0,1) bf16 rows into the pages listed in block_row (in order)."""
    if n_tokens <= 0:
        return
    B, H, D = geom.block_size, geom.num_kv_heads, geom.head_dim
    nb = (n_tokens + B - 1) // B
    vals = np.full((nb * B, H, D), BF16_NAN_BITS, dtype=np.uint16)
    vals[:n_tokens] = normal_bf16(rng, (n_tokens, H, D))
    # [nb*B, H, D] -> [nb, B, H, D] -> [nb, H, B, D]
    pool[block_row[:nb]] = vals.reshape(nb, B, H, D).transpose(0, 2, 1, 3)


def make_batch(rng: np.random.Generator, geom: Geometry, context_len, query_len,
               block_table: np.ndarray, label: str = "") -> Batch:
    context_len = np.asarray(context_len, dtype=np.int32)
    query_len = np.asarray(query_len, dtype=np.int32)
    T = int(query_len.sum())
    return Batch(
        geom=geom, context_len=context_len, query_len=query_len,
        block_table=np.ascontiguousarray(block_table, dtype=np.int32),
        q=normal_bf16(rng, (T, geom.num_q_heads, geom.head_dim)),
        k_new=normal_bf16(rng, (T, geom.num_kv_heads, geom.head_dim)),
        v_new=normal_bf16(rng, (T, geom.num_kv_heads, geom.head_dim)),
        label=label)


def scenario_from_lengths(name: str, geom: Geometry, seed: int,
                          prefix_len: Sequence[int], query_lens_per_iter: Sequence[Sequence[int]],
                          shuffle_seqs: bool = False) -> Scenario:
    """Generic builder: sequence s starts with prefix_len[s] cached tokens and receives
    query_lens_per_iter[t][s] new tokens in iteration t."""
    rng = np.random.default_rng(seed)
    prefix = np.asarray(prefix_len, dtype=np.int64)
    qiters = np.asarray(query_lens_per_iter, dtype=np.int64).reshape(len(query_lens_per_iter), -1)
    S = prefix.shape[0]
    order = np.arange(S)
    if shuffle_seqs:
        order = rng.permutation(S)
        prefix = prefix[order]
        qiters = qiters[:, order]
    capacity = prefix + qiters.sum(axis=0)
    table = deal_block_tables(rng, geom, capacity)
    k_pool, v_pool = empty_pools(geom)
    for s in range(S):
        fill_prefix(rng, geom, k_pool, table[s], int(prefix[s]))
        fill_prefix(rng, geom, v_pool, table[s], int(prefix[s]))
    sc = Scenario(name=name, geom=geom, k_pool=k_pool, v_pool=v_pool)
    have = prefix.copy()
    for t in range(qiters.shape[0]):
        lq = qiters[t]
        have = have + lq
        sc.batches.append(make_batch(rng, geom, have, lq, table, label=f"{name}/it{t}"))
    return sc


# --------------------------------------------------------------------------- length draws
def lognormal_clipped(rng: np.random.Generator, n: int, mu: float, sigma: float, lo: int, hi: int) -> np.ndarray:
    z = rng.standard_normal(n)
    return np.clip(np.rint(np.exp(mu + sigma * z)), lo, hi).astype(np.int64)


def uniform_int(rng: np.random.Generator, n: int, lo: int, hi: int) -> np.ndarray:
    return rng.integers(lo, hi + 1, size=n, dtype=np.int64)


# --------------------------------------------------------------------------- the five configs
GEOM_TINY = Geometry(num_q_heads=8, num_kv_heads=2, head_dim=64, block_size=16, num_blocks=256)
GEOM_G4 = Geometry(num_q_heads=32, num_kv_heads=8, head_dim=128, block_size=16, num_blocks=65536)
GEOM_G8 = Geometry(num_q_heads=64, num_kv_heads=8, head_dim=128, block_size=16, num_blocks=65536)


def _seed(config: int, k: int) -> int:
    return 1000 * config + k


def config1_tiny(k: int = 0) -> Scenario:
    """4 decode seqs with context 256 plus one 128-token prefill chunk over a 128-token prefix."""
    prefix = [128] + [255] * 4
    qlen = [[128] + [1] * 4]
    return scenario_from_lengths("cfg1_tiny", GEOM_TINY, _seed(1, k), prefix, qlen)


def config2_lengths(k: int = 0) -> np.ndarray:
    rng = np.random.default_rng(_seed(2, k) + 500)
    return uniform_int(rng, 64, 1024, 8192)


def config2_decode_only(k: int = 0) -> Scenario:
    lc = config2_lengths(k)
    return scenario_from_lengths("cfg2_decode", GEOM_G4, _seed(2, k), lc - 1, [[1] * 64])


def config3_lengths(k: int = 0) -> np.ndarray:
    rng = np.random.default_rng(_seed(3, k) + 500)
    return lognormal_clipped(rng, 48, np.log(4096.0), 0.8, 128, 16384)


def config3_chat(k: int = 0, iterations: Sequence[int] = (0, 1, 2, 3)) -> Scenario:
    """48 decode seqs (lognormal contexts) + 2 lent prefills of 2048 new tokens over 6144 cached,
    in 512-token chunks; iteration t carries chunk t and every decode seq grown by one token."""
    lc = config3_lengths(k)
    n_it = max(iterations) + 1
    prefix = [6144, 6144] + list(lc - 1)
    qlen = [[512, 512] + [1] * 48 for _ in range(n_it)]
    sc = scenario_from_lengths("cfg3_chat", GEOM_G4, _seed(3, k), prefix, qlen)
    return sc


def config3_chat_tp4_shard(k: int = 0, iterations: Sequence[int] = (0, 1, 2, 3)) -> Scenario:
    """One tensor-parallel rank's share of the chat-like batch under the paper's TP4 deployment
    (Section 6.1): the same sequences, a quarter of the heads (8 query heads, 2 KV heads)."""
    lc = config3_lengths(k)
    n_it = max(iterations) + 1
    prefix = [6144, 6144] + list(lc - 1)
    qlen = [[512, 512] + [1] * 48 for _ in range(n_it)]
    geom = Geometry(num_q_heads=8, num_kv_heads=2, head_dim=128, block_size=16, num_blocks=65536)
    return scenario_from_lengths("cfg3_chat_tp4", geom, _seed(3, k) + 40, prefix, qlen)


def config4_lengths(k: int = 0) -> np.ndarray:
    rng = np.random.default_rng(_seed(4, k) + 500)
    return uniform_int(rng, 16, 8192, 32768)


def config4_agentic(k: int = 0, iterations: Sequence[int] = (0, 1, 2, 3)) -> Scenario:
    """16 decode seqs (contexts 8K..32K) + 1 lent prefill of 8192 new tokens over 24,576 cached,
    in 2048-token chunks."""
    lc = config4_lengths(k)
    n_it = max(iterations) + 1
    prefix = [24576] + list(lc - 1)
    qlen = [[2048] + [1] * 16 for _ in range(n_it)]
    return scenario_from_lengths("cfg4_agentic", GEOM_G4, _seed(4, k), prefix, qlen)


def config5_lengths(k: int = 0) -> np.ndarray:
    """Lognormal whose *unclipped mean* is 2048 with sigma 1: mu = ln 2048 - sigma^2/2."""
    rng = np.random.default_rng(_seed(5, k) + 500)
    return lognormal_clipped(rng, 256, np.log(2048.0) - 0.5, 1.0, 64, 32768)


CONFIG5_POINTS: List[Tuple[int, int]] = [(0, 0)] + [(b, n) for b in (512, 2048, 8192) for n in (1, 2, 3, 4)]


def config5_sweep_point(budget: int, n_prompts: int, k: int = 0) -> Scenario:
    """256 decode seqs + a prefill token budget split over n_prompts prompts with prefixes U{0..8192}."""
    lc = config5_lengths(k)
    rng = np.random.default_rng(_seed(5, k) + 700 + 13 * budget + n_prompts)
    prefix: List[int] = []
    qlen: List[int] = []
    if budget > 0:
        base, rem = divmod(budget, n_prompts)
        for i in range(n_prompts):
            qlen.append(base + (1 if i < rem else 0))
            prefix.append(int(rng.integers(0, 8193)))
    prefix += list(lc - 1)
    qlen += [1] * 256
    return scenario_from_lengths(f"cfg5_b{budget}_n{n_prompts}", GEOM_G8, _seed(5, k) + budget + n_prompts,
                                 prefix, [qlen])


# --------------------------------------------------------------------------- accounting (sizes only)
def decode_algorithmic_bytes(geom: Geometry, context_len: np.ndarray, query_len: np.ndarray, window: int = 0,
                            kv_elem_bytes: int = 2) -> int:
    """Bytes a decode pass must move: K and V of every visible token once per KV head (the last `window` tokens
    with a sliding window; one byte per element for an fp8 cache), the q row in and the o row out, and the
    block-table entries."""
    m = np.asarray(query_len) == 1
    lc = np.asarray(context_len, dtype=np.int64)[m]
    vis = np.minimum(lc, window) if window > 0 else lc
    per_tok = 2 * geom.num_kv_heads * geom.head_dim * kv_elem_bytes
    return int((vis * per_tok).sum() + m.sum() * 2 * geom.num_q_heads * geom.head_dim * 2
               + 4 * ((vis + geom.block_size - 1) // geom.block_size).sum())


def _visible_pairs(lc: np.ndarray, lq: np.ndarray, window: int) -> int:
    """Number of (query row, visible key) pairs of the chunks: row i of a chunk sees min(P + i + 1, window) keys."""
    total = 0
    for c, q in zip(lc, lq):
        rows = np.arange(int(c - q) + 1, int(c) + 1, dtype=np.int64)
        total += int((np.minimum(rows, window) if window > 0 else rows).sum())
    return total


def prefill_flops(geom: Geometry, context_len: np.ndarray, query_len: np.ndarray, window: int = 0) -> int:
    """4*D*Hq * (number of visible (query, key) pairs) over the sequences with Lq > 1."""
    lq = np.asarray(query_len, dtype=np.int64)
    lc = np.asarray(context_len, dtype=np.int64)
    m = lq > 1
    return int(4 * geom.head_dim * geom.num_q_heads * _visible_pairs(lc[m], lq[m], window))


def prefill_algorithmic_bytes(geom: Geometry, context_len: np.ndarray, query_len: np.ndarray, window: int = 0,
                              kv_elem_bytes: int = 2) -> int:
    """Bytes a prefill pass must move: K and V of every token some row of the chunk can see, once per KV head, the
    chunk's q rows in and o rows out."""
    lq = np.asarray(query_len, dtype=np.int64)
    lc = np.asarray(context_len, dtype=np.int64)
    m = lq > 1
    vis = lc[m] if window <= 0 else np.minimum(lc[m], lq[m] + window - 1)
    per_tok = 2 * geom.num_kv_heads * geom.head_dim * kv_elem_bytes
    return int((vis * per_tok).sum() + (lq[m] * 2 * geom.num_q_heads * geom.head_dim * 2).sum())


def decode_flops(geom: Geometry, context_len: np.ndarray, query_len: np.ndarray, window: int = 0) -> int:
    m = np.asarray(query_len) == 1
    lc = np.asarray(context_len, dtype=np.int64)[m]
    vis = np.minimum(lc, window) if window > 0 else lc
    return int(4 * geom.head_dim * geom.num_q_heads * vis.sum())


def tile_edge_rows(batch: Batch, tile: int = 128, stride: int = 41) -> np.ndarray:
    """Packed q-row indices to check at full size: every decode row; for a prefill sequence the first and
    last row of every `tile`-row q tile (so that no q tile, and with all heads checked no work item, goes
    unchecked), the chunk's last row, and every `stride`-th row."""
    qs = batch.q_start()
    rows: List[np.ndarray] = []
    for s in range(batch.num_seqs):
        n = int(batch.query_len[s])
        if n == 0:
            continue
        idx = np.arange(n)
        if n > 1:
            idx = idx[(idx % tile == 0) | (idx % tile == tile - 1) | (idx % stride == 0) | (idx == n - 1)]
        rows.append(qs[s] + idx)
    return np.concatenate(rows).astype(np.int64) if rows else np.zeros(0, dtype=np.int64)


def sample_rows(batch: Batch, max_prefill_rows_per_seq: int = 0) -> np.ndarray:
    """Packed q-row indices to check: every decode row; for prefill sequences either all rows or
    a deterministic subsample (first and last row of every 128-row tile plus every 7th row,
    thinned evenly to the cap)."""
    qs = batch.q_start()
    rows: List[np.ndarray] = []
    for s in range(batch.num_seqs):
        n = int(batch.query_len[s])
        if n == 0:
            continue
        idx = np.arange(n)
        if max_prefill_rows_per_seq and n > max_prefill_rows_per_seq:
            keep = (idx % 128 == 0) | (idx % 128 == 127) | (idx % 7 == 0) | (idx == n - 1)
            idx = idx[keep]
            if idx.size > max_prefill_rows_per_seq:
                pick = np.unique(np.linspace(0, idx.size - 1, max_prefill_rows_per_seq).astype(np.int64))
                idx = idx[pick]
        rows.append(qs[s] + idx)
    return np.concatenate(rows).astype(np.int64) if rows else np.zeros(0, dtype=np.int64)


def shared_prefix_scenario(name: str, geom: Geometry, seed: int, shared_tokens: int, own_prefix: Sequence[int],
                           query_len: Sequence[int], group: Optional[Sequence[int]] = None):
    """Sequences whose block tables alias the same pages for a common prefix (radix-cache reuse: turns of one
    agent session, sub-agents forked from one context).  Sequence s with group[s] >= 0 starts with the
    `shared_tokens` tokens of its group's prefix (a multiple of the block size, the same physical pages for every
    member), followed by own_prefix[s] cached tokens of its own and query_len[s] new ones; group[s] < 0: no
    shared part.  Returns (scenario with one batch, share_group int32 [S], shared_len int32 [S])."""
    B = geom.block_size
    assert shared_tokens % B == 0
    S = len(own_prefix)
    group = np.zeros(S, dtype=np.int32) if group is None else np.asarray(group, dtype=np.int32)
    rng = np.random.default_rng(seed)
    k_pool, v_pool = empty_pools(geom)
    perm = rng.permutation(geom.num_blocks).astype(np.int32)
    at = 0
    n_shared_pages = shared_tokens // B
    group_pages = {}
    for gid in sorted(set(int(x) for x in group if x >= 0)):
        pages = perm[at:at + n_shared_pages]
        at += n_shared_pages
        fill_prefix(rng, geom, k_pool, pages, shared_tokens)
        fill_prefix(rng, geom, v_pool, pages, shared_tokens)
        group_pages[gid] = pages
    lens = []
    rows = []
    for s in range(S):
        sh = shared_tokens if group[s] >= 0 else 0
        total = sh + int(own_prefix[s]) + int(query_len[s])
        n_own_pages = (total + B - 1) // B - sh // B
        own = perm[at:at + n_own_pages]
        at += n_own_pages
        assert at <= geom.num_blocks, "pool too small"
        row = np.concatenate([group_pages[int(group[s])], own]) if group[s] >= 0 else own
        fill_prefix(rng, geom, k_pool, own, int(own_prefix[s]))
        fill_prefix(rng, geom, v_pool, own, int(own_prefix[s]))
        rows.append(row)
        lens.append(total)
    width = max(len(r) for r in rows)
    table = np.full((S, width), -1, dtype=np.int32)
    for s, r in enumerate(rows):
        table[s, :len(r)] = r
    b = make_batch(rng, geom, lens, query_len, table, label=name)
    sc = Scenario(name, geom, k_pool, v_pool, [b])
    shared_len = np.where(group >= 0, shared_tokens, 0).astype(np.int32)
    return sc, group.astype(np.int32), shared_len
