"""The N > 1 path of bench.py on CPU: two gloo ranks with different device times agree on the slowest
one, and the whole-job rate counts every rank's shard over that time (weak scaling, no data-path
collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e, attn = bench.max_over_ranks([10.0 + 5.0 * rank, 20.0 - 3.0 * rank, 1.0 + rank], dist, "cpu")
    q.put((rank, ms, e2e, attn, bench.whole_job_rate(1000, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, attn, rate in got:
        assert (ms, e2e, attn) == (15.0, 20.0, 2.0)
        assert abs(rate - 2 * 1000 / 15e-3) < 1e-6


def test_single_rank_passthrough():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, "cpu") == [1.5, 2.5]
    assert bench.whole_job_rate(10, 1, 1000.0) == 10.0
