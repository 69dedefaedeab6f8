"""The N > 1 path of the benchmark on CPU: two gloo ranks, each an independent replica (the attention
path has no exchange step), the only collective being the max-over-ranks of the step time."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    import cf_synth as syn
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        ms = [3.0, 5.5][rank]                                   # each replica's own step time
        slowest = bench.reduce_max(ms, dist, torch.device("cpu"))
        lens = syn.config3_lengths(rank % 3)                    # replicas draw different seeds, same shapes
        tokens = 1072 * 10
        value = world * tokens / (slowest * 1e-3)               # whole-job rate over the slowest rank
        out.put((rank, slowest, int(lens.sum()), value))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_whole_job_rate_over_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == 5.5                        # max over ranks, seen by both
    assert res[0][2] != res[1][2]                               # different replicas, different draws
    assert abs(res[0][3] - 2 * 10720 / 5.5e-3) < 1e-6


def test_reduce_max_is_identity_without_a_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(1.25, None, torch.device("cpu")) == 1.25


def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    import cf_synth as syn
    import paper_2609_27085_b200 as cf
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        # every rank plans the same sequences for ITS quarter of the heads (tensor parallelism by KV-head group)
        Hq, Hkv = 32, 8
        lc = np.array([6144 + 512, 6144 + 512] + list(syn.config3_lengths()), dtype=np.int32)
        lq = np.array([512, 512] + [1] * 48, dtype=np.int32)
        d = cf.make_desc(Hq // world, Hkv // world, 128, 16, 65536)
        st, dec, comb, pre, parts = cf.cf_plan_inspect(d, lc, lq, 4096, 148)
        mine = {"decode": [(int(s), rank * (Hkv // world) + kvh, int(b), int(e)) for s, _, b, e, _, _ in dec for kvh in range(Hkv // world)],
                "prefill": [(int(s), int(row0), int(n), rank * (Hq // world) + int(h), int(j0), int(j1))
                            for s, _, row0, n, h, _, j0, j1 in pre]}
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        if rank == 0:
            out.put(gathered)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_four_head_sharded_ranks_cover_every_row_and_head_once():
    """Four gloo ranks, each planning its (Hq/4, Hkv/4) shard of the chat-like batch: the union of the shards'
    work covers every (decode sequence, KV head, key) and every (prefill row, query head) exactly once."""
    import numpy as np
    sys.path.insert(0, ROOT)
    import cf_synth as syn
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 4, port, q)) for r in range(4)]
    for p in procs:
        p.start()
    gathered = q.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    lc = np.array([6144 + 512, 6144 + 512] + list(syn.config3_lengths()), dtype=np.int64)
    lq = np.array([512, 512] + [1] * 48)
    dec_cover = {(s, kvh): np.zeros(lc[s], dtype=np.int32) for s in range(2, 50) for kvh in range(8)}
    pre_cover = {s: np.zeros((512, 32), dtype=np.int32) for s in (0, 1)}
    for shard in gathered:
        for s, kvh, b, e in shard["decode"]:
            dec_cover[(s, kvh)][b:e] += 1
        for s, row0, n, head, j0, j1 in shard["prefill"]:
            if j0 == 0:                                   # a KV-split item lists one entry per range; count the tile once
                pre_cover[s][row0:row0 + n, head] += 1
    assert all((c == 1).all() for c in dec_cover.values())
    assert all((c == 1).all() for c in pre_cover.values())
