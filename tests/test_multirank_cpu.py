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
