"""The N > 1 bookkeeping of bench.py on CPU: two gloo ranks, each with its own timing; every rank
must get the slowest rank's time back, and the whole-job throughput must be what all ranks
processed divided by that time (token shards, no data-path collective)."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e = bench.max_over_ranks([10.0 + rank, 100.0 - rank])
    dist.barrier()
    out.put((rank, ms, e2e, bench.aggregate_tokens_per_s(world, 2048, 5, ms)))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_throughput_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, value in got:
        assert ms == 11.0 and e2e == 100.0                      # slowest rank of each timing
        assert abs(value - 2 * 2048 * 5 / 11e-3) < 1e-6 * value   # all ranks' tokens / slowest time


def test_max_over_ranks_without_a_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
